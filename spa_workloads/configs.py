"""The five workload shapes.

Shapes follow the settings the paper evaluates on: ViT-style 16x16 patches on
224^2 / 384^2 images (Sec. 2, Sec. 4.1), a detection-sized 1280x800-like input at
stride 16 (Sec. 4.2), and per-image select ratios in the range its Tables 4-7
report (about 13 % to 99 %).  Object "blobs" stand in for the box / mask labels of
Sec. 3.2 that decide which tokens are informative.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class SpaConfig:
    name: str
    B: int                 # images in the batch
    grid: Tuple[int, int]  # token grid (rows, cols); N = rows * cols
    C: int                 # channels
    H: int                 # attention heads; d = C // H
    dtype: str             # "f32" or "bf16": storage type of x, weights, dY
    seed: int
    blobs: Tuple[int, int]         # min / max number of circular blobs per image
    keep: Tuple[float, float]      # per-image target keep fraction ~ U(lo, hi)
    keep_mode: str = "uniform"     # "uniform" or "alternate" (lo, hi, lo, hi, ...)
    offset: float = 6.0            # blob tokens get +offset * w_g/|w_g|
    tau: float = 0.0               # gate threshold on the logit
    backward: bool = False         # config also exercises the backward pass

    @property
    def N(self) -> int:
        return self.grid[0] * self.grid[1]

    @property
    def d(self) -> int:
        return self.C // self.H

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS = (
    SpaConfig("tiny_f32", B=4, grid=(14, 14), C=96, H=3, dtype="f32", seed=0,
              blobs=(1, 3), keep=(0.10, 0.50), offset=3.0, backward=True),
    SpaConfig("vit_s16_bf16", B=64, grid=(14, 14), C=384, H=6, dtype="bf16", seed=1,
              blobs=(1, 4), keep=(0.20, 0.80), backward=True),
    SpaConfig("detection_bf16", B=16, grid=(50, 84), C=256, H=8, dtype="bf16", seed=2,
              blobs=(1, 6), keep=(0.05, 0.40), backward=True),
    SpaConfig("vit_b16_384_bf16", B=32, grid=(24, 24), C=768, H=12, dtype="bf16", seed=3,
              blobs=(1, 4), keep=(0.10, 0.90), keep_mode="alternate", backward=True),
    SpaConfig("train_vit_b_bf16", B=128, grid=(14, 14), C=768, H=12, dtype="bf16", seed=4,
              blobs=(1, 4), keep=(0.01, 0.60), backward=True),
)


def get_config(i: int) -> SpaConfig:
    """Config by 1-based index (1..5), as the workloads are numbered."""
    return CONFIGS[i - 1]


def scaled_config(cfg: SpaConfig, B: int | None = None, **kw) -> SpaConfig:
    """A copy of `cfg` with a different batch size or other fields (reduced test cases)."""
    if B is not None:
        kw["B"] = B
    return replace(cfg, **kw)
