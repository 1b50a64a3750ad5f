"""One SPA block as a sequence of library calls.

`SpaBlock` owns the device buffers of one block (allocated once through PyTorch) and issues the
C-ABI calls in order on the current stream.  It computes nothing itself: every step runs in the
CUDA library.  Nothing here synchronises; N_p stays on the device.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as L


class SpaBlock:
    """Buffers + call sequence for gate -> select/pack -> QKV -> attention -> projection -> unpack
    (paper Sec. 3.2) and the matching backward pass."""

    def __init__(self, B: int, N: int, C: int, H: int, dtype: str, tau: float = 0.0, flags: int = 0,
                 capacity: Optional[int] = None, backward: bool = True, device: str = "cuda",
                 fused: Optional[bool] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("SpaBlock needs a CUDA device; there is no CPU path")
        L.lib()
        self.B, self.N, self.C, self.H = B, N, C, H
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        cap = capacity if capacity is not None else max(B * N, 1)
        self.p = L.make_params(B, N, C, H, dtype, cap, flags, tau)
        self.cap = cap
        # fused unpack: the projection and the QKV input gradient scatter their rows to the tokens themselves
        # (tensor-core problems only); None = use it where the library offers it
        can_fuse = L.spa_fused_scatter_supported(self.p)
        if fused and not can_fuse:
            raise ValueError("the fused scatter calls do not apply to this problem (needs bf16 tensor-core sizes)")
        self.fused = can_fuse if fused is None else bool(fused)
        dev = torch.device(device)
        T = self.tdtype
        e = lambda *s, dt=T: torch.empty(*s, dtype=dt, device=dev)
        self.scores = e(max(B * N, 1), dt=torch.float32)
        self.mask = e(max(B * N, 1), dt=torch.uint8)
        self.cu = torch.zeros(B + 1, dtype=torch.int32, device=dev)
        self.idx = e(cap, dt=torch.int32)
        self.inv = e(max(B * N, 1), dt=torch.int32)
        self.xp = e(cap, C)
        self.qkv = e(cap, 3 * C)
        self.ao = e(cap, C)
        self.lse = e(H, cap, dt=torch.float32)
        self.z = e(cap, C)
        self.y = e(B, N, C)
        self.status = torch.zeros(4, dtype=torch.int32, device=dev)
        ws = L.spa_workspace_bytes(self.p)
        self.workspace = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev) if ws > 0 else None
        # the weight gradients do not feed the rest of the backward chain: they run on a second stream,
        # with a scratch area of their own, beside the attention backward and the input gradients
        self.side_stream = torch.cuda.Stream(device=dev) if backward else None
        self.workspace_side = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev) if (ws > 0 and backward) else None
        if backward:
            self.dz = e(cap, C)
            self.dao = e(cap, C)
            self.dqkv = e(cap, 3 * C)
            self.dxp = e(cap, C)
            self.dX = e(B, N, C)
            self.dW_qkv = e(3 * C, C, dt=torch.float32)
            self.db_qkv = e(3 * C, dt=torch.float32)
            self.dW_o = e(C, C, dt=torch.float32)
            self.db_o = e(C, dt=torch.float32)
        self._saved = None
        self._seg = (self.cu, B)   # attention segments: the images, unless forward() is given others

    # ------------------------------------------------------------------ forward
    def forward(self, x, w_g, b_g: float, W_qkv, b_qkv, W_o, b_o, s_up=None, y=None, order=None, seg_offsets=None):
        """`order` (int32 [N] on the device): visiting order of each image's tokens for the packing (a shifted
        feature map); `seg_offsets` (int32, ascending, ending at N_p): attention segments other than the images,
        e.g. the container cut; the backward pass uses the same segments."""
        p = self.p
        y = self.y if y is None else y
        inplace = bool(p.flags & L.SPA_FLAG_INPLACE)
        if self.fused and not inplace:
            # the pass-through rows y = x are written by the gate, which reads all of x anyway
            L.spa_gate_prefill(p, x, w_g, b_g, s_up, self.scores, self.mask, y)
        else:
            L.spa_gate(p, x, w_g, b_g, s_up, self.scores, self.mask)
        if order is None:
            L.spa_select_pack(p, x, self.mask, self.scores, self.xp, self.idx, self.inv, self.cu, self.status)
        else:
            L.spa_select_pack_ordered(p, x, self.mask, self.scores, order, self.xp, self.idx, self.inv, self.cu,
                                      self.status)
        L.spa_packed_qkv(p, self.xp, W_qkv, b_qkv, self.cu, self.qkv, self.status)
        self._seg = (self.cu, self.B) if seg_offsets is None else (seg_offsets, int(seg_offsets.numel()) - 1)
        L.spa_packed_attention_fwd(p, self.qkv, self._seg[0], self._seg[1], self.ao, self.lse, self.status)
        if self.fused:
            if inplace:
                y = x
            L.spa_packed_proj_scatter(p, self.ao, W_o, b_o, self.idx, self.cu, y, self.status)
        else:
            L.spa_packed_proj(p, self.ao, W_o, b_o, self.cu, self.z, self.status)
            if inplace:
                L.spa_unpack_scatter(p, self.z, None, self.idx, self.inv, self.cu, x, self.status)
                y = x
            else:
                L.spa_unpack_scatter(p, self.z, x, self.idx, self.inv, self.cu, y, self.status)
        self._saved = (W_qkv, W_o)
        return y

    # ------------------------------------------------------------------ backward
    def backward(self, dY, dX=None, overlap=True):
        """Gradients for the last forward(): returns dX; parameter gradients land in dW_qkv, db_qkv,
        dW_o, db_o (fp32).  No gradient reaches the gate (hard threshold).  With overlap=True the two
        weight-gradient calls are issued on a second stream and joined before returning."""
        p = self.p
        W_qkv, W_o = self._saved
        dX = self.dX if dX is None else dX
        C = self.C
        main = torch.cuda.current_stream()
        side = self.side_stream if (overlap and self.side_stream is not None) else None
        # dz = gather of dY; dX = dY on the tokens that passed through (fused path: the QKV input gradient
        # scatters its rows to the selected tokens itself, so no packed dx and no scatter kernel follow)
        L.spa_unpack_scatter_bwd(p, dY, self.idx, self.inv, self.cu, self.dz, dX)
        if side is None:
            L.spa_packed_linear_bwd(p, self.ao, W_o, self.dz, C, C, self.cu, self.dao, self.dW_o, self.db_o,
                                    self.workspace, self.status)
        else:
            side.wait_stream(main)
            L.spa_packed_linear_bwd(p, self.ao, W_o, self.dz, C, C, self.cu, None, self.dW_o, self.db_o,
                                    self.workspace_side, self.status, stream=side)
            L.spa_packed_linear_bwd(p, self.ao, W_o, self.dz, C, C, self.cu, self.dao, None, None,
                                    self.workspace, self.status)
        L.spa_packed_attention_bwd(p, self.qkv, self.ao, self.lse, self.dao, self._seg[0], self._seg[1], self.dqkv,
                                   self.workspace, self.status)
        if self.fused:
            if side is None:
                L.spa_packed_linear_bwd_scatter(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.idx, self.cu, dX,
                                                self.dW_qkv, self.db_qkv, self.workspace, self.status)
            else:
                side.wait_stream(main)
                L.spa_packed_linear_bwd(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.cu, None, self.dW_qkv,
                                        self.db_qkv, self.workspace_side, self.status, stream=side)
                L.spa_packed_linear_bwd_scatter(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.idx, self.cu, dX,
                                                None, None, None, self.status)
                main.wait_stream(side)
            return dX
        if side is None:
            L.spa_packed_linear_bwd(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.cu, self.dxp, self.dW_qkv,
                                    self.db_qkv, self.workspace, self.status)
        else:
            side.wait_stream(main)
            L.spa_packed_linear_bwd(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.cu, None, self.dW_qkv, self.db_qkv,
                                    self.workspace_side, self.status, stream=side)
            L.spa_packed_linear_bwd(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.cu, self.dxp, None, None,
                                    self.workspace, self.status)
        L.spa_select_pack_bwd(p, self.dxp, dY, self.idx, self.cu, dX)
        if side is not None:
            main.wait_stream(side)
        return dX

    def backward_trainable(self, dY, x, w_g, labels=None, alpha: float = 1.0, s_up=None, dX=None):
        """backward() extended by the gradient that reaches the gate (Sec. 3.2 Eq. 4-5, Sec. 3.3 Eq. 10): the
        selection loss alpha * BCE(Sigmoid(scores), labels) when `labels` (uint8 [B, N]) is given, and, under
        SPA_FLAG_GATE_SCALE, the path through the sigmoid scaling of the packed rows.  `s_up` must be the
        tensor given to forward().  Returns dX; also fills dw_g, db_g, ds_up (fp32), ds and loss."""
        p, C = self.p, self.C
        W_qkv, W_o = self._saved
        dX = self.dX if dX is None else dX
        if not hasattr(self, "ds"):
            dev = self.scores.device
            n = max(self.B * self.N, 1)
            self.ds = torch.empty(n, dtype=torch.float32, device=dev)
            self.ds_up = torch.empty(n, dtype=torch.float32, device=dev)
            self.dw_g = torch.empty(C, dtype=torch.float32, device=dev)
            self.db_g = torch.empty(1, dtype=torch.float32, device=dev)
            self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
            self.train_ws = torch.empty(max(L.spa_train_workspace_bytes(p), 256), dtype=torch.uint8, device=dev)
        L.spa_select_loss(p, self.scores, labels, alpha, self.ds, self.loss, self.train_ws)
        L.spa_unpack_scatter_bwd(p, dY, self.idx, self.inv, self.cu, self.dz, dX)
        L.spa_packed_linear_bwd(p, self.ao, W_o, self.dz, C, C, self.cu, self.dao, self.dW_o, self.db_o,
                                self.workspace, self.status)
        L.spa_packed_attention_bwd(p, self.qkv, self.ao, self.lse, self.dao, self._seg[0], self._seg[1], self.dqkv,
                                   self.workspace, self.status)
        L.spa_packed_linear_bwd(p, self.xp, W_qkv, self.dqkv, C, 3 * C, self.cu, self.dxp, self.dW_qkv,
                                self.db_qkv, self.workspace, self.status)
        if p.flags & L.SPA_FLAG_GATE_SCALE:
            L.spa_select_pack_bwd_gated(p, self.dxp, x, self.scores, dY, self.idx, self.cu, dX, self.ds)
        else:
            L.spa_select_pack_bwd(p, self.dxp, dY, self.idx, self.cu, dX)
        L.spa_gate_bwd(p, x, w_g, self.scores, s_up, self.ds, dX, self.dw_g, self.db_g, self.ds_up, self.train_ws)
        return dX

    def read_status(self) -> int:
        """Blocking: the device status word (0 = ok)."""
        return L.spa_read_status(self.status)
