"""ctypes binding of libspa.so: the same names as include/spa.h, argument marshalling only.

Every function takes torch tensors that already live on the GPU (PyTorch is used for device
memory and streams, nothing else), checks nothing but presence, and raises SpaError when the
library returns a negative status.  There is no fallback: if the library is missing or no CUDA
device is present, calling into it raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspa.so")

SPA_OK, SPA_ERR_INVALID_ARG, SPA_ERR_UNSUPPORTED, SPA_ERR_CAPACITY, SPA_ERR_CUDA, SPA_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
SPA_ERR_SCRATCH = -6
SPA_STATIC_SCRATCH_BYTES = 4 << 20
SPA_F32, SPA_BF16 = 0, 1
SPA_FLAG_RESIDUAL, SPA_FLAG_INPLACE, SPA_FLAG_GATE_SCALE, SPA_FLAG_SIMT_ONLY, SPA_FLAG_NO_CTA_PAIRS = 1, 2, 4, 8, 16
SPA_FLAG_UNFUSED = 32
SPA_FLAG_ONE_PASS_BWD = 64

EXPORTS = (
    "spa_workspace_bytes", "spa_gate", "spa_select_pack", "spa_packed_qkv", "spa_packed_attention_fwd",
    "spa_packed_attention_bwd", "spa_packed_proj", "spa_unpack_scatter", "spa_unpack_scatter_bwd",
    "spa_select_pack_bwd", "spa_packed_linear_bwd", "spa_read_status", "spa_status_string",
    "spa_last_cuda_error", "spa_launch_count", "spa_packed_attention_bwd_static",
    "spa_fused_scatter_supported", "spa_gate_prefill", "spa_unpack_prefill", "spa_packed_proj_scatter", "spa_packed_linear_bwd_scatter",
    "spa_select_pack_ordered", "spa_train_workspace_bytes", "spa_score_pool", "spa_select_loss", "spa_select_pack_bwd_gated", "spa_gate_bwd",
    "spa_packed_linear", "spa_layer_norm", "spa_layer_norm_bwd", "spa_gelu", "spa_gelu_bwd",
    "spa_overlap_create", "spa_overlap_destroy", "spa_block_fwd", "spa_block_bwd",
    "spa_probe_exp2", "spa_probe_wait_expiry", "spa_probe_mma_issue", "spa_pack_state_bytes", "spa_gate_select_pack_supported",
    "spa_gate_select_pack", "spa_container_max_segments", "spa_container_offsets",
)


class SpaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().spa_status_string(status).decode()
        if status == SPA_ERR_CUDA:
            msg += ": " + lib().spa_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})")


class SpaParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("C", C.c_int32), ("H", C.c_int32), ("dtype", C.c_int32),
                ("flags", C.c_int32), ("capacity", C.c_int32), ("tau", C.c_float), ("softmax_scale", C.c_float)]


class SpaBlockBuffers(C.Structure):
    """spa_block_buffers of include/spa.h, field for field."""
    _fields_ = [("x", C.c_void_p), ("w_g", C.c_void_p), ("b_g", C.c_float), ("s_up", C.c_void_p),
                ("W_qkv", C.c_void_p), ("b_qkv", C.c_void_p), ("W_o", C.c_void_p), ("b_o", C.c_void_p),
                ("order", C.c_void_p), ("seg_offsets", C.c_void_p), ("n_seg", C.c_int32),
                ("scores", C.c_void_p), ("mask", C.c_void_p), ("cu_seqlens", C.c_void_p), ("idx", C.c_void_p),
                ("inv", C.c_void_p), ("x_packed", C.c_void_p), ("qkv", C.c_void_p), ("attn_out", C.c_void_p),
                ("lse", C.c_void_p), ("z", C.c_void_p), ("y", C.c_void_p),
                ("dY", C.c_void_p), ("dz", C.c_void_p), ("d_attn_out", C.c_void_p), ("dqkv", C.c_void_p),
                ("dx_packed", C.c_void_p), ("dX", C.c_void_p), ("dW_qkv", C.c_void_p), ("db_qkv", C.c_void_p),
                ("dW_o", C.c_void_p), ("db_o", C.c_void_p), ("workspace", C.c_void_p), ("workspace_side", C.c_void_p),
                ("pack_state", C.c_void_p), ("overlap", C.c_void_p), ("d_status", C.c_void_p),
                ("trainable", C.c_int32), ("labels", C.c_void_p), ("alpha", C.c_float), ("ds", C.c_void_p),
                ("ds_up", C.c_void_p), ("dw_g", C.c_void_p), ("db_g", C.c_void_p), ("loss", C.c_void_p),
                ("train_workspace", C.c_void_p), ("container_len", C.c_int32)]


def make_params(B, N, Cc, H, dtype, capacity=None, flags=0, tau=0.0, softmax_scale=0.0) -> SpaParams:
    dt = {"f32": SPA_F32, "bf16": SPA_BF16, torch.float32: SPA_F32, torch.bfloat16: SPA_BF16}.get(dtype, dtype)
    return SpaParams(B, N, Cc, H, dt, flags, capacity if capacity is not None else max(B * N, 1), tau, softmax_scale)


_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built (run `python -m paper_2410_23608_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2410_23608_b200.build.build()")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        pp = C.POINTER(SpaParams)
        L.spa_workspace_bytes.restype = C.c_size_t
        L.spa_workspace_bytes.argtypes = [pp]
        L.spa_gate.argtypes = [pp, vp, vp, f32, vp, vp, vp, vp]
        L.spa_select_pack.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_packed_qkv.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_packed_attention_fwd.argtypes = [pp, vp, vp, i32, vp, vp, vp, vp]
        L.spa_packed_attention_bwd.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp]
        L.spa_packed_attention_bwd_static.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        L.spa_packed_proj.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_unpack_scatter.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_unpack_scatter_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_select_pack_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp]
        L.spa_packed_linear_bwd.argtypes = [pp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.spa_fused_scatter_supported.argtypes = [pp]
        L.spa_gate_prefill.argtypes = [pp, vp, vp, f32, vp, vp, vp, vp, vp]
        L.spa_unpack_prefill.argtypes = [pp, vp, vp, vp]
        L.spa_packed_proj_scatter.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_packed_linear_bwd_scatter.argtypes = [pp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_select_pack_ordered.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_train_workspace_bytes.restype = C.c_size_t
        L.spa_train_workspace_bytes.argtypes = [pp]
        L.spa_score_pool.argtypes = [vp, i32, i32, i32, vp, vp]
        L.spa_select_loss.argtypes = [pp, vp, vp, f32, vp, vp, vp, vp]
        L.spa_select_pack_bwd_gated.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_gate_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_packed_linear.argtypes = [pp, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp]
        L.spa_layer_norm.argtypes = [pp, vp, vp, vp, f32, vp, vp, vp, vp]
        L.spa_layer_norm_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_gelu.argtypes = [pp, vp, i32, vp, vp]
        L.spa_gelu_bwd.argtypes = [pp, vp, vp, i32, vp, vp]
        L.spa_overlap_create.argtypes = [C.POINTER(vp)]
        L.spa_overlap_destroy.argtypes = [vp]
        L.spa_block_fwd.argtypes = [pp, C.POINTER(SpaBlockBuffers), vp]
        L.spa_block_bwd.argtypes = [pp, C.POINTER(SpaBlockBuffers), vp]
        L.spa_pack_state_bytes.restype = C.c_size_t
        L.spa_pack_state_bytes.argtypes = [pp]
        L.spa_gate_select_pack_supported.argtypes = [pp]
        L.spa_gate_select_pack.argtypes = [pp, vp, vp, f32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.spa_container_max_segments.argtypes = [pp, i32]
        L.spa_container_offsets.argtypes = [pp, vp, i32, vp, vp]
        L.spa_probe_exp2.argtypes = [i32, i32, vp, C.POINTER(C.c_ulonglong), vp]
        L.spa_probe_wait_expiry.argtypes = [i32, vp, vp, vp]
        L.spa_probe_mma_issue.argtypes = [i32, i32, vp, vp, vp]
        L.spa_read_status.argtypes = [vp, vp]
        for name in EXPORTS:
            if name not in ("spa_workspace_bytes", "spa_train_workspace_bytes", "spa_pack_state_bytes", "spa_status_string", "spa_last_cuda_error",
                            "spa_launch_count"):
                getattr(L, name).restype = C.c_int
        L.spa_status_string.restype = C.c_char_p
        L.spa_status_string.argtypes = [C.c_int]
        L.spa_last_cuda_error.restype = C.c_char_p
        L.spa_last_cuda_error.argtypes = []
        L.spa_launch_count.restype = C.c_ulonglong
        L.spa_launch_count.argtypes = []
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("the SPA library takes device tensors only")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _check(rc: int, where: str):
    if rc < 0:
        raise SpaError(rc, where)


def spa_workspace_bytes(p: SpaParams) -> int:
    return int(lib().spa_workspace_bytes(C.byref(p)))


def spa_gate(p, x, w_g, b_g, s_up, scores, mask, stream=None):
    _check(lib().spa_gate(C.byref(p), _ptr(x), _ptr(w_g), float(b_g), _ptr(s_up), _ptr(scores), _ptr(mask),
                          _stream(stream)), "spa_gate")


def spa_pack_state_bytes(p) -> int:
    return int(lib().spa_pack_state_bytes(C.byref(p)))


def spa_gate_select_pack_supported(p) -> bool:
    return bool(lib().spa_gate_select_pack_supported(C.byref(p)))


def spa_gate_select_pack(p, x, w_g, b_g, s_up, scores, mask, y, x_packed, idx, inv, cu_seqlens, pack_state,
                         d_status=None, stream=None):
    _check(lib().spa_gate_select_pack(C.byref(p), _ptr(x), _ptr(w_g), float(b_g), _ptr(s_up), _ptr(scores), _ptr(mask),
                                      _ptr(y), _ptr(x_packed), _ptr(idx), _ptr(inv), _ptr(cu_seqlens), _ptr(pack_state),
                                      _ptr(d_status), _stream(stream)), "spa_gate_select_pack")


def spa_container_max_segments(p, L) -> int:
    return int(lib().spa_container_max_segments(C.byref(p), int(L)))


def spa_container_offsets(p, cu_seqlens, L, seg_offsets, stream=None):
    _check(lib().spa_container_offsets(C.byref(p), _ptr(cu_seqlens), int(L), _ptr(seg_offsets), _stream(stream)),
           "spa_container_offsets")


def spa_select_pack(p, x, mask, scores, x_packed, idx, inv, cu_seqlens, d_status=None, stream=None):
    _check(lib().spa_select_pack(C.byref(p), _ptr(x), _ptr(mask), _ptr(scores), _ptr(x_packed), _ptr(idx), _ptr(inv),
                                 _ptr(cu_seqlens), _ptr(d_status), _stream(stream)), "spa_select_pack")


def spa_packed_qkv(p, x_packed, W_qkv, b_qkv, cu_seqlens, qkv, d_status=None, stream=None):
    _check(lib().spa_packed_qkv(C.byref(p), _ptr(x_packed), _ptr(W_qkv), _ptr(b_qkv), _ptr(cu_seqlens), _ptr(qkv),
                                _ptr(d_status), _stream(stream)), "spa_packed_qkv")


def spa_packed_attention_fwd(p, qkv, seg_offsets, n_seg, attn_out, lse, d_status=None, stream=None):
    _check(lib().spa_packed_attention_fwd(C.byref(p), _ptr(qkv), _ptr(seg_offsets), int(n_seg), _ptr(attn_out),
                                          _ptr(lse), _ptr(d_status), _stream(stream)), "spa_packed_attention_fwd")


def spa_packed_attention_bwd(p, qkv, attn_out, lse, d_attn_out, seg_offsets, n_seg, dqkv, workspace=None,
                             d_status=None, stream=None):
    _check(lib().spa_packed_attention_bwd(C.byref(p), _ptr(qkv), _ptr(attn_out), _ptr(lse), _ptr(d_attn_out),
                                          _ptr(seg_offsets), int(n_seg), _ptr(dqkv), _ptr(workspace), _ptr(d_status),
                                          _stream(stream)), "spa_packed_attention_bwd")


def spa_packed_attention_bwd_static(p, qkv, attn_out, lse, d_attn_out, seg_offsets, n_seg, dqkv, d_status=None,
                                    stream=None):
    """Attention backward for callers that cannot allocate: the scratch is an array inside the library
    (at most SPA_STATIC_SCRATCH_BYTES; all calls on a device share it, so keep them ordered)."""
    _check(lib().spa_packed_attention_bwd_static(C.byref(p), _ptr(qkv), _ptr(attn_out), _ptr(lse), _ptr(d_attn_out),
                                                 _ptr(seg_offsets), int(n_seg), _ptr(dqkv), _ptr(d_status),
                                                 _stream(stream)), "spa_packed_attention_bwd_static")


def spa_packed_proj(p, a, W_o, b_o, cu_seqlens, z, d_status=None, stream=None):
    _check(lib().spa_packed_proj(C.byref(p), _ptr(a), _ptr(W_o), _ptr(b_o), _ptr(cu_seqlens), _ptr(z),
                                 _ptr(d_status), _stream(stream)), "spa_packed_proj")


def spa_unpack_scatter(p, z_packed, x, idx, inv, cu_seqlens, y, d_status=None, stream=None):
    _check(lib().spa_unpack_scatter(C.byref(p), _ptr(z_packed), _ptr(x), _ptr(idx), _ptr(inv), _ptr(cu_seqlens),
                                    _ptr(y), _ptr(d_status), _stream(stream)), "spa_unpack_scatter")


def spa_unpack_scatter_bwd(p, dY, idx, inv, cu_seqlens, dz_packed, dX, stream=None):
    _check(lib().spa_unpack_scatter_bwd(C.byref(p), _ptr(dY), _ptr(idx), _ptr(inv), _ptr(cu_seqlens),
                                        _ptr(dz_packed), _ptr(dX), _stream(stream)), "spa_unpack_scatter_bwd")


def spa_select_pack_bwd(p, dx_packed, dY, idx, cu_seqlens, dX, stream=None):
    _check(lib().spa_select_pack_bwd(C.byref(p), _ptr(dx_packed), _ptr(dY), _ptr(idx), _ptr(cu_seqlens), _ptr(dX),
                                     _stream(stream)), "spa_select_pack_bwd")


def spa_packed_linear_bwd(p, a, W, dout, n_in, n_out, cu_seqlens, da, dW, db, workspace=None, d_status=None,
                          stream=None):
    _check(lib().spa_packed_linear_bwd(C.byref(p), _ptr(a), _ptr(W), _ptr(dout), int(n_in), int(n_out),
                                       _ptr(cu_seqlens), _ptr(da), _ptr(dW), _ptr(db), _ptr(workspace),
                                       _ptr(d_status), _stream(stream)), "spa_packed_linear_bwd")


def spa_fused_scatter_supported(p) -> bool:
    return bool(lib().spa_fused_scatter_supported(C.byref(p)))


def spa_gate_prefill(p, x, w_g, b_g, s_up, scores, mask, y, stream=None):
    _check(lib().spa_gate_prefill(C.byref(p), _ptr(x), _ptr(w_g), float(b_g), _ptr(s_up), _ptr(scores), _ptr(mask),
                                  _ptr(y), _stream(stream)), "spa_gate_prefill")


def spa_unpack_prefill(p, src, dst, stream=None):
    _check(lib().spa_unpack_prefill(C.byref(p), _ptr(src), _ptr(dst), _stream(stream)), "spa_unpack_prefill")


def spa_packed_proj_scatter(p, a, W_o, b_o, idx, cu_seqlens, y, d_status=None, stream=None):
    _check(lib().spa_packed_proj_scatter(C.byref(p), _ptr(a), _ptr(W_o), _ptr(b_o), _ptr(idx), _ptr(cu_seqlens),
                                         _ptr(y), _ptr(d_status), _stream(stream)), "spa_packed_proj_scatter")


def spa_packed_linear_bwd_scatter(p, a, W, dout, n_in, n_out, idx, cu_seqlens, dX, dW, db, workspace=None,
                                  d_status=None, stream=None):
    _check(lib().spa_packed_linear_bwd_scatter(C.byref(p), _ptr(a), _ptr(W), _ptr(dout), int(n_in), int(n_out),
                                               _ptr(idx), _ptr(cu_seqlens), _ptr(dX), _ptr(dW), _ptr(db),
                                               _ptr(workspace), _ptr(d_status), _stream(stream)),
           "spa_packed_linear_bwd_scatter")


def spa_select_pack_ordered(p, x, mask, scores, order, x_packed, idx, inv, cu_seqlens, d_status=None, stream=None):
    _check(lib().spa_select_pack_ordered(C.byref(p), _ptr(x), _ptr(mask), _ptr(scores), _ptr(order), _ptr(x_packed),
                                         _ptr(idx), _ptr(inv), _ptr(cu_seqlens), _ptr(d_status), _stream(stream)),
           "spa_select_pack_ordered")


def spa_train_workspace_bytes(p) -> int:
    return int(lib().spa_train_workspace_bytes(C.byref(p)))


def spa_score_pool(scores_prev, B, rows, cols, s_up, stream=None):
    _check(lib().spa_score_pool(_ptr(scores_prev), int(B), int(rows), int(cols), _ptr(s_up), _stream(stream)),
           "spa_score_pool")


def spa_select_loss(p, scores, labels, alpha, ds, loss, workspace, stream=None):
    _check(lib().spa_select_loss(C.byref(p), _ptr(scores), _ptr(labels), float(alpha), _ptr(ds), _ptr(loss),
                                 _ptr(workspace), _stream(stream)), "spa_select_loss")


def spa_select_pack_bwd_gated(p, dx_packed, x, scores, dY, idx, cu_seqlens, dX, ds, stream=None):
    _check(lib().spa_select_pack_bwd_gated(C.byref(p), _ptr(dx_packed), _ptr(x), _ptr(scores), _ptr(dY), _ptr(idx),
                                           _ptr(cu_seqlens), _ptr(dX), _ptr(ds), _stream(stream)),
           "spa_select_pack_bwd_gated")


def spa_gate_bwd(p, x, w_g, scores, s_up, ds, dX, dw_g, db_g, ds_up, workspace, stream=None):
    _check(lib().spa_gate_bwd(C.byref(p), _ptr(x), _ptr(w_g), _ptr(scores), _ptr(s_up), _ptr(ds), _ptr(dX), _ptr(dw_g),
                              _ptr(db_g), _ptr(ds_up), _ptr(workspace), _stream(stream)), "spa_gate_bwd")


def spa_packed_linear(p, a, W, b, n_in, n_out, cu_seqlens, out, accumulate=False, d_status=None, stream=None):
    _check(lib().spa_packed_linear(C.byref(p), _ptr(a), _ptr(W), _ptr(b), int(n_in), int(n_out), _ptr(cu_seqlens), _ptr(out),
                                   1 if accumulate else 0, _ptr(d_status), _stream(stream)), "spa_packed_linear")


def spa_layer_norm(p, x, gamma, beta, eps, y, mean, rstd, stream=None):
    _check(lib().spa_layer_norm(C.byref(p), _ptr(x), _ptr(gamma), _ptr(beta), float(eps), _ptr(y), _ptr(mean), _ptr(rstd),
                                _stream(stream)), "spa_layer_norm")


def spa_layer_norm_bwd(p, dy, x, gamma, mean, rstd, add, dx, dgamma, dbeta, workspace, stream=None):
    _check(lib().spa_layer_norm_bwd(C.byref(p), _ptr(dy), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(rstd), _ptr(add), _ptr(dx),
                                    _ptr(dgamma), _ptr(dbeta), _ptr(workspace), _stream(stream)), "spa_layer_norm_bwd")


def spa_gelu(p, u, n_cols, h, stream=None):
    _check(lib().spa_gelu(C.byref(p), _ptr(u), int(n_cols), _ptr(h), _stream(stream)), "spa_gelu")


def spa_gelu_bwd(p, dh, u, n_cols, du, stream=None):
    _check(lib().spa_gelu_bwd(C.byref(p), _ptr(dh), _ptr(u), int(n_cols), _ptr(du), _stream(stream)), "spa_gelu_bwd")


def spa_overlap_create() -> int:
    """Handle of a second stream plus fork / join events, for spa_block_buffers.overlap."""
    h = C.c_void_p()
    _check(lib().spa_overlap_create(C.byref(h)), "spa_overlap_create")
    return h.value


def spa_overlap_destroy(handle) -> None:
    if handle:
        _check(lib().spa_overlap_destroy(C.c_void_p(handle)), "spa_overlap_destroy")


def block_buffers(**fields) -> SpaBlockBuffers:
    """A spa_block_buffers filled from tensors (device pointers), scalars and None (NULL)."""
    b = SpaBlockBuffers()
    for name, v in fields.items():
        if isinstance(v, torch.Tensor):
            p = _ptr(v)
            v = p.value if p is not None else None
        setattr(b, name, v)
    return b


def spa_block_fwd(p, bufs: SpaBlockBuffers, stream=None):
    _check(lib().spa_block_fwd(C.byref(p), C.byref(bufs), _stream(stream)), "spa_block_fwd")


def spa_block_bwd(p, bufs: SpaBlockBuffers, stream=None):
    _check(lib().spa_block_bwd(C.byref(p), C.byref(bufs), _stream(stream)), "spa_block_bwd")


def spa_probe_exp2(n_ctas, iters, sink, stream=None) -> int:
    """Enqueue the exponential-throughput probe; returns the number of exponentials it evaluates."""
    n = C.c_ulonglong(0)
    _check(lib().spa_probe_exp2(int(n_ctas), int(iters), _ptr(sink), C.byref(n), _stream(stream)), "spa_probe_exp2")
    return int(n.value)


def spa_probe_wait_expiry(limit, d_status, polls_done=None, stream=None):
    _check(lib().spa_probe_wait_expiry(int(limit), _ptr(d_status), _ptr(polls_done), _stream(stream)),
           "spa_probe_wait_expiry")


def spa_probe_mma_issue(variant, elected, cycles, d_status, stream=None):
    """Enqueue the product-issue probe: cycles (device int32[2]) receives the SM clocks to issue 32 products and until
    they complete (variant 0-3: operands in shared memory N = 64, A in TMEM N = 64, shared memory N = 128, N = 256)."""
    _check(lib().spa_probe_mma_issue(int(variant), int(bool(elected)), _ptr(cycles), _ptr(d_status), _stream(stream)),
           "spa_probe_mma_issue")


def spa_read_status(d_status, stream=None) -> int:
    return int(lib().spa_read_status(_ptr(d_status), _stream(stream)))


def spa_launch_count() -> int:
    return int(lib().spa_launch_count())
