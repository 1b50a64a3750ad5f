"""Seeded input generator for one SPA block.

Every tensor is drawn once from a counter-based generator (numpy Philox), rounded
once to the storage dtype of the workload (fp32 or bf16), and handed out as fp64
arrays holding exactly those rounded values.  The CPU oracle consumes the fp64
arrays; the CUDA path consumes the same values re-encoded in the storage dtype, so
both sides read identical bits.

Recipe (per workload):
  * w_g ~ N(0, 1/C); u = w_g / |w_g|.
  * per image: a target keep fraction f_b, 1..k circular blobs with uniform centres
    and relative radii in [0.5, 1]; one common radius scale is bisected until the
    fraction of grid cells covered by the union is closest to f_b.
  * x ~ N(0, 1), plus `offset * u` on blob tokens; b_g = -(offset/2) * |w_g|, so the
    threshold tau = 0 sits midway between the background and the blob logit means.
  * W_qkv, W_o ~ N(0, 1/C); b_qkv, b_o ~ N(0, 0.02^2); dY ~ N(0, 1).
  * input validity: after rounding, any token whose gate logit (fp64, rounded
    inputs) lies within `margin` of tau is moved away from it by changing one
    element of its row, so the keep decision never depends on rounding order.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

from .configs import SpaConfig

MARGIN = 2e-3   # enforced |logit - tau|; the parity contract only needs 1e-3


# --------------------------------------------------------------------------- bf16
def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp values to bfloat16 (round-to-nearest-even) and return uint16 bit patterns."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def from_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float32 values."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """fp64 array rounded to the nearest bfloat16 value, returned as fp64."""
    return from_bf16_bits(to_bf16_bits(a)).astype(np.float64).reshape(np.shape(a))


def _round(a: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return bf16_round(a)
    return np.asarray(a, dtype=np.float32).astype(np.float64)


# --------------------------------------------------------------------------- blobs
def _blob_mask(rng: np.random.Generator, grid, n_blobs: int, target: float) -> np.ndarray:
    """Boolean [rows*cols] mask of the union of `n_blobs` discs covering ~`target` of the grid."""
    rows, cols = grid
    cy = rng.uniform(0.0, rows, size=n_blobs)
    cx = rng.uniform(0.0, cols, size=n_blobs)
    rel = rng.uniform(0.5, 1.0, size=n_blobs)
    yy, xx = np.meshgrid(np.arange(rows) + 0.5, np.arange(cols) + 0.5, indexing="ij")
    d2 = (yy[None] - cy[:, None, None]) ** 2 + (xx[None] - cx[:, None, None]) ** 2  # [k, rows, cols]

    def cover(scale: float) -> np.ndarray:
        return (d2 <= (rel[:, None, None] * scale) ** 2).any(axis=0)

    lo, hi = 0.0, float(2 * (rows + cols))
    best, best_err = cover(hi), 2.0
    for _ in range(40):
        mid = 0.5 * (lo + hi)
        m = cover(mid)
        frac = m.mean()
        err = abs(frac - target)
        if err < best_err:
            best, best_err = m, err
        if frac < target:
            lo = mid
        else:
            hi = mid
    return best.reshape(-1)


# --------------------------------------------------------------------------- inputs
@dataclass
class SpaInputs:
    cfg: SpaConfig
    x: np.ndarray          # [B, N, C] fp64, values representable in cfg.dtype
    w_g: np.ndarray        # [C]
    b_g: float             # representable in fp32
    tau: float
    W_qkv: np.ndarray      # [3C, C]  (out x in)
    b_qkv: np.ndarray      # [3C]
    W_o: np.ndarray        # [C, C]
    b_o: np.ndarray        # [C]
    dY: np.ndarray         # [B, N, C]
    blob_mask: np.ndarray  # [B, N] bool: tokens that received the blob offset
    keep_target: np.ndarray  # [B] target keep fractions
    extra: Dict[str, np.ndarray] = field(default_factory=dict)

    def torch(self, name: str, device="cpu"):
        """Tensor `name` in the workload's storage dtype (exact re-encoding of the fp64 values)."""
        import torch
        a = getattr(self, name)
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        if self.cfg.dtype == "bf16":
            t = t.to(torch.bfloat16)
        return t.to(device)


def _logits(x2d: np.ndarray, w: np.ndarray, b: float) -> np.ndarray:
    # input-validity check only: the generator must know which tokens sit near tau
    return x2d @ w + b


def make_inputs(cfg: SpaConfig, keep_override: Optional[np.ndarray] = None,
                margin: float = MARGIN) -> SpaInputs:
    """Draw every tensor of workload `cfg`.  `keep_override` ([B] fractions, 0 or 1 allowed)
    replaces the per-image keep targets (edge cases: empty or fully selected images)."""
    rng = np.random.Generator(np.random.Philox(key=cfg.seed))
    B, N, C = cfg.B, cfg.N, cfg.C

    w_g = _round(rng.normal(0.0, 1.0 / np.sqrt(C), size=C), cfg.dtype)
    wn = float(np.linalg.norm(w_g))
    u = w_g / wn
    b_g = float(np.float32(-(cfg.offset / 2.0) * wn))

    if keep_override is not None:
        keep = np.asarray(keep_override, dtype=np.float64).reshape(B)
        rng.uniform(size=B)  # keep the stream position independent of the override
    elif cfg.keep_mode == "alternate":
        keep = np.where(np.arange(B) % 2 == 0, cfg.keep[0], cfg.keep[1]).astype(np.float64)
        rng.uniform(size=B)
    else:
        keep = rng.uniform(cfg.keep[0], cfg.keep[1], size=B)

    blob = np.zeros((B, N), dtype=bool)
    for b in range(B):
        k = int(rng.integers(cfg.blobs[0], cfg.blobs[1] + 1))
        m = _blob_mask(rng, cfg.grid, k, float(keep[b]))
        if keep[b] <= 0.0:
            m[:] = False
        elif keep[b] >= 1.0:
            m[:] = True
        blob[b] = m

    x = rng.normal(0.0, 1.0, size=(B, N, C))
    x += (cfg.offset * blob)[:, :, None] * u[None, None, :]
    x = _round(x, cfg.dtype)

    # keep every logit at least `margin` from tau (on the rounded values, in fp64)
    x2 = x.reshape(B * N, C)
    c_star = int(np.argmax(np.abs(w_g)))
    step = 4.0 * margin / abs(w_g[c_star])
    for _ in range(60):
        s = _logits(x2, w_g, b_g)
        bad = np.nonzero(np.abs(s - cfg.tau) < margin)[0]
        if bad.size == 0:
            break
        direction = np.where(s[bad] >= cfg.tau, 1.0, -1.0) * np.sign(w_g[c_star])
        x2[bad, c_star] = _round(x2[bad, c_star] + direction * step, cfg.dtype)
        step *= 1.5
    else:  # pragma: no cover
        raise RuntimeError("could not enforce the gate margin")
    x = x2.reshape(B, N, C)

    W_qkv = _round(rng.normal(0.0, 1.0 / np.sqrt(C), size=(3 * C, C)), cfg.dtype)
    b_qkv = _round(rng.normal(0.0, 0.02, size=3 * C), cfg.dtype)
    W_o = _round(rng.normal(0.0, 1.0 / np.sqrt(C), size=(C, C)), cfg.dtype)
    b_o = _round(rng.normal(0.0, 0.02, size=C), cfg.dtype)
    dY = _round(rng.normal(0.0, 1.0, size=(B, N, C)), cfg.dtype)

    return SpaInputs(cfg=cfg, x=x, w_g=w_g, b_g=b_g, tau=float(cfg.tau), W_qkv=W_qkv, b_qkv=b_qkv,
                     W_o=W_o, b_o=b_o, dY=dY, blob_mask=blob, keep_target=keep)
