"""One pre-norm transformer block around SPA as a sequence of library calls.

out = y1 + FFN(LN2(y1)),  y1 = x + scatter(SPA(LN1(x)))  (paper Sec. 3.2: selected tokens go through attention,
the others are passed straight on to the feed-forward network).  `SpaLayer` owns the buffers and issues the
C-ABI calls; every step runs in the CUDA library.
"""
from __future__ import annotations

import torch

from . import binding as L
from .block import SpaBlock


class SpaLayer:
    def __init__(self, B: int, N: int, C: int, H: int, dtype: str, hidden: int | None = None, tau: float = 0.0,
                 eps: float = 1e-5, flags: int = 0, device: str = "cuda"):
        self.B, self.N, self.C, self.H = B, N, C, H
        self.hidden = 4 * C if hidden is None else hidden
        self.eps = eps
        # the attention part adds its result to the residual stream: SPA_FLAG_RESIDUAL
        self.blk = SpaBlock(B, N, C, H, dtype, tau=tau, flags=flags | L.SPA_FLAG_RESIDUAL, device=device)
        self.p = self.blk.p
        # same problem without the residual flag (plain row scatter in the backward pass)
        self.p_plain = L.make_params(B, N, C, H, dtype, self.blk.cap, flags & ~L.SPA_FLAG_RESIDUAL, tau)
        dev = torch.device(device)
        T = self.blk.tdtype
        rows = max(B * N, 1)
        e = lambda *s, dt=T: torch.empty(*s, dtype=dt, device=dev)
        self.cu_all = (torch.arange(B + 1, dtype=torch.int32, device=dev) * N).contiguous()  # every token is a row
        self.z, self.y1, self.t, self.out = e(B, N, C), e(B, N, C), e(B, N, C), e(B, N, C)
        self.u, self.h = e(rows, self.hidden), e(rows, self.hidden)
        self.m1, self.r1, self.m2, self.r2 = (e(rows, dt=torch.float32) for _ in range(4))
        self.dh, self.dt, self.dy1, self.dZ, self.dX = e(rows, self.hidden), e(B, N, C), e(B, N, C), e(B, N, C), e(B, N, C)
        f = lambda *s: torch.empty(*s, dtype=torch.float32, device=dev)
        self.dW1, self.db1, self.dW2, self.db2 = f(self.hidden, C), f(self.hidden), f(C, self.hidden), f(C)
        self.dg1, self.dbe1, self.dg2, self.dbe2 = f(C), f(C), f(C), f(C)
        # split-K partials of the widest weight gradient (at most 32 splits) and the per-CTA sums of the LayerNorm backward
        ws = max(L.spa_workspace_bytes(self.p), 32 * self.hidden * C * 4 + 32 * max(self.hidden, C) * 4 + 1024,
                 L.spa_train_workspace_bytes(self.p))
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
        self._saved = None

    def forward(self, x, prm):
        """prm: dict of device tensors g1, be1, w_g, W_qkv, b_qkv, W_o, b_o, g2, be2, W1, b1, W2, b2 and float b_g."""
        p, blk, C, Hd = self.p, self.blk, self.C, self.hidden
        st = blk.status
        L.spa_layer_norm(p, x, prm["g1"], prm["be1"], self.eps, self.z, self.m1, self.r1)
        L.spa_gate(p, self.z, prm["w_g"], prm["b_g"], None, blk.scores, blk.mask)
        L.spa_select_pack(p, self.z, blk.mask, blk.scores, blk.xp, blk.idx, blk.inv, blk.cu, st)
        L.spa_packed_qkv(p, blk.xp, prm["W_qkv"], prm["b_qkv"], blk.cu, blk.qkv, st)
        L.spa_packed_attention_fwd(p, blk.qkv, blk.cu, self.B, blk.ao, blk.lse, st)
        if blk.fused:
            L.spa_unpack_prefill(p, x, self.y1)                       # residual stream; selected rows get += below
            L.spa_packed_proj_scatter(p, blk.ao, prm["W_o"], prm["b_o"], blk.idx, blk.cu, self.y1, st)
        else:
            L.spa_packed_proj(p, blk.ao, prm["W_o"], prm["b_o"], blk.cu, blk.z, st)
            L.spa_unpack_scatter(p, blk.z, x, blk.idx, blk.inv, blk.cu, self.y1, st)
        L.spa_layer_norm(p, self.y1, prm["g2"], prm["be2"], self.eps, self.t, self.m2, self.r2)
        L.spa_packed_linear(p, self.t, prm["W1"], prm["b1"], C, Hd, self.cu_all, self.u, False, st)
        L.spa_gelu(p, self.u, Hd, self.h)
        L.spa_unpack_prefill(p, self.y1, self.out)
        L.spa_packed_linear(p, self.h, prm["W2"], prm["b2"], Hd, C, self.cu_all, self.out, True, st)
        self._saved = (x, prm)
        return self.out

    def backward(self, d_out):
        """Gradient to x (returned) and to every parameter but the gate's (dW*, db*, dg*, dbe*, and the SPA block's)."""
        p, blk, C, Hd, ws = self.p, self.blk, self.C, self.hidden, self.workspace
        x, prm = self._saved
        st = blk.status
        L.spa_packed_linear_bwd(p, self.h, prm["W2"], d_out, Hd, C, self.cu_all, self.dh, self.dW2, self.db2, ws, st)
        L.spa_gelu_bwd(p, self.dh, self.u, Hd, self.dh)
        L.spa_packed_linear_bwd(p, self.t, prm["W1"], self.dh, C, Hd, self.cu_all, self.dt, self.dW1, self.db1, ws, st)
        L.spa_layer_norm_bwd(p, self.dt, self.y1, prm["g2"], self.m2, self.r2, d_out, self.dy1, self.dg2, self.dbe2, ws)
        # attention branch: its input gradient reaches LN1's output on the selected rows only
        L.spa_unpack_scatter_bwd(p, self.dy1, blk.idx, blk.inv, blk.cu, blk.dz, None)
        L.spa_packed_linear_bwd(p, blk.ao, prm["W_o"], blk.dz, C, C, blk.cu, blk.dao, blk.dW_o, blk.db_o, ws, st)
        L.spa_packed_attention_bwd(p, blk.qkv, blk.ao, blk.lse, blk.dao, blk.cu, self.B, blk.dqkv, ws, st)
        L.spa_packed_linear_bwd(p, blk.xp, prm["W_qkv"], blk.dqkv, C, 3 * C, blk.cu, blk.dxp, blk.dW_qkv, blk.db_qkv, ws, st)
        self.dZ.zero_()
        L.spa_select_pack_bwd(self.p_plain, blk.dxp, None, blk.idx, blk.cu, self.dZ)
        L.spa_layer_norm_bwd(p, self.dZ, x, prm["g1"], self.m1, self.r1, self.dy1, self.dX, self.dg1, self.dbe1, ws)
        return self.dX

    def read_status(self) -> int:
        return self.blk.read_status()
