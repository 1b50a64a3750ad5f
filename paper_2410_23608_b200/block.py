"""One SPA block: the device buffers, handed to the library's two block calls.

`SpaBlock` owns the buffers of one block (allocated once through PyTorch) and calls `spa_block_fwd` /
`spa_block_bwd` on the current stream.  The order of the kernels, the choice between fused and separate
scatter calls and the second stream for the weight gradients all live in the library; nothing here
computes or sequences.  Nothing synchronises; N_p stays on the device.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as L


class SpaBlock:
    """Buffers for gate -> select/pack -> QKV -> attention -> projection -> unpack (paper Sec. 3.2) and the
    matching backward pass."""

    def __init__(self, B: int, N: int, C: int, H: int, dtype: str, tau: float = 0.0, flags: int = 0,
                 capacity: Optional[int] = None, backward: bool = True, device: str = "cuda",
                 fused: Optional[bool] = None, one_pass: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("SpaBlock needs a CUDA device; there is no CPU path")
        L.lib()
        self.B, self.N, self.C, self.H = B, N, C, H
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        cap = capacity if capacity is not None else max(B * N, 1)
        # fused unpack: the projection and the QKV input gradient scatter their rows to the tokens themselves
        # (tensor-core problems only); None = use it where the library offers it
        can_fuse = L.spa_fused_scatter_supported(L.make_params(B, N, C, H, dtype, cap, flags, tau))
        if fused and not can_fuse:
            raise ValueError("the fused scatter calls do not apply to this problem (needs bf16 tensor-core sizes)")
        self.fused = can_fuse if fused is None else bool(fused)
        if not self.fused:
            flags |= L.SPA_FLAG_UNFUSED
        self.p = L.make_params(B, N, C, H, dtype, cap, flags, tau)
        self.cap = cap
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
        # the weight gradients run on a second stream (owned by the library handle), with a scratch area of their own
        self.workspace_side = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev) if (ws > 0 and backward) else None
        self._overlap = L.spa_overlap_create() if backward else None
        # one_pass: gate, selection and packing as one kernel (measured slower than the two kernels on the five
        # workloads, so off unless asked for); its scratch is zeroed once here, the kernel leaves it zero
        self.one_pass = one_pass and L.spa_gate_select_pack_supported(self.p)
        self.pack_state = (torch.zeros(max(L.spa_pack_state_bytes(self.p), 256), dtype=torch.uint8, device=dev)
                           if self.one_pass else None)
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
        self._saved = None            # (W_qkv, W_o) of the last forward()
        self._seg = (self.cu, B)      # attention segments: the images, unless forward() is given others
        self._keep = None             # tensors of the last call that the enqueued work still reads
        self._container_len = 0       # > 0: the library builds the container cuts itself (forward(container_len=L))
        self.container_seg = None

    def __del__(self):
        try:
            if getattr(self, "_overlap", None):
                torch.cuda.synchronize()
                L.spa_overlap_destroy(self._overlap)
                self._overlap = None
        except Exception:
            pass

    def _buffers(self, **extra):
        seg, n_seg = self._seg
        f = dict(scores=self.scores, mask=self.mask, cu_seqlens=self.cu, idx=self.idx, inv=self.inv, x_packed=self.xp,
                 qkv=self.qkv, attn_out=self.ao, lse=self.lse, z=self.z, workspace=self.workspace, d_status=self.status,
                 pack_state=self.pack_state, container_len=self._container_len,
                 seg_offsets=None if seg is self.cu else seg, n_seg=n_seg)
        f.update(extra)
        return L.block_buffers(**f)

    # ------------------------------------------------------------------ forward
    def forward(self, x, w_g, b_g: float, W_qkv, b_qkv, W_o, b_o, s_up=None, y=None, order=None, seg_offsets=None,
                container_len: int = 0):
        """`order` (int32 [N] on the device): visiting order of each image's tokens for the packing (a shifted
        feature map); `seg_offsets` (int32, ascending, ending at N_p): attention segments other than the images;
        `container_len` = L > 0: the paper's containers, their cuts built on the device by the library (the segment
        array is owned here).  The backward pass uses the same segments."""
        inplace = bool(self.p.flags & L.SPA_FLAG_INPLACE)
        y = x if inplace else (self.y if y is None else y)
        self._container_len = int(container_len)
        if container_len > 0:
            n_max = L.spa_container_max_segments(self.p, container_len)
            if self.container_seg is None or self.container_seg.numel() != n_max + 1:
                self.container_seg = torch.zeros(n_max + 1, dtype=torch.int32, device=self.cu.device)
            seg_offsets = self.container_seg
        self._seg = (self.cu, self.B) if seg_offsets is None else (seg_offsets, int(seg_offsets.numel()) - 1)
        self._saved = (W_qkv, W_o)
        self._keep = (x, w_g, W_qkv, b_qkv, W_o, b_o, s_up, order, seg_offsets, y)
        L.spa_block_fwd(self.p, self._buffers(x=x, w_g=w_g, b_g=float(b_g), s_up=s_up, W_qkv=W_qkv, b_qkv=b_qkv, W_o=W_o,
                                              b_o=b_o, order=order, y=y))
        return y

    # ------------------------------------------------------------------ backward
    def _backward_fields(self, dY, dX):
        W_qkv, W_o = self._saved
        return dict(W_qkv=W_qkv, W_o=W_o, dY=dY, dz=self.dz, d_attn_out=self.dao, dqkv=self.dqkv, dx_packed=self.dxp,
                    dX=dX, dW_qkv=self.dW_qkv, db_qkv=self.db_qkv, dW_o=self.dW_o, db_o=self.db_o,
                    workspace_side=self.workspace_side)

    def backward(self, dY, dX=None, overlap=True):
        """Gradients for the last forward(): returns dX; parameter gradients land in dW_qkv, db_qkv,
        dW_o, db_o (fp32).  No gradient reaches the gate (hard threshold).  With overlap=True the two
        weight-gradient products run on the library's second stream and are joined before the call returns."""
        dX = self.dX if dX is None else dX
        L.spa_block_bwd(self.p, self._buffers(overlap=self._overlap if overlap else None,
                                              **self._backward_fields(dY, dX)))
        return dX

    def backward_trainable(self, dY, x, w_g, labels=None, alpha: float = 1.0, s_up=None, dX=None):
        """backward() extended by the gradient that reaches the gate (Sec. 3.2 Eq. 4-5, Sec. 3.3 Eq. 10): the
        selection loss alpha * BCE(Sigmoid(scores), labels) when `labels` (uint8 [B, N]) is given, and, under
        SPA_FLAG_GATE_SCALE, the path through the sigmoid scaling of the packed rows.  `s_up` must be the
        tensor given to forward().  Returns dX; also fills dw_g, db_g, ds_up (fp32), ds and loss."""
        dX = self.dX if dX is None else dX
        if not hasattr(self, "ds"):
            dev = self.scores.device
            n = max(self.B * self.N, 1)
            self.ds = torch.empty(n, dtype=torch.float32, device=dev)
            self.ds_up = torch.empty(n, dtype=torch.float32, device=dev)
            self.dw_g = torch.empty(self.C, dtype=torch.float32, device=dev)
            self.db_g = torch.empty(1, dtype=torch.float32, device=dev)
            self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
            self.train_ws = torch.empty(max(L.spa_train_workspace_bytes(self.p), 256), dtype=torch.uint8, device=dev)
        L.spa_block_bwd(self.p, self._buffers(x=x, w_g=w_g, s_up=s_up, trainable=1, labels=labels, alpha=float(alpha),
                                              ds=self.ds, ds_up=self.ds_up, dw_g=self.dw_g, db_g=self.db_g,
                                              loss=self.loss, train_workspace=self.train_ws,
                                              **self._backward_fields(dY, dX)))
        return dX

    def read_status(self) -> int:
        """Blocking: the device status word (0 = ok)."""
        return L.spa_read_status(self.status)
