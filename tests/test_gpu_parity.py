"""GPU parity: the CUDA library, called through its C boundary, against the fp64 oracle on the same
seeded inputs.  Integer and index outputs must match bit for bit; floating point within the stated
tolerances (fp32: max-abs 1e-4; bf16: max-abs 3e-2 and relative RMS 1e-2)."""
import functools

import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from spa_workloads import get_config, make_inputs, scaled_config
from tests.gpu_util import TOL, assert_close, dev, host, round_to

pytestmark = pytest.mark.gpu


@functools.lru_cache(maxsize=None)
def problem(i, residual=False):
    cfg = get_config(i)
    inp = make_inputs(cfg)
    fwd = O.block_fwd(inp.x, inp.w_g, inp.b_g, inp.tau, inp.W_qkv, inp.b_qkv, inp.W_o, inp.b_o, cfg.H,
                      residual=residual)
    bwd = O.block_bwd(fwd, inp.dY, inp.x, inp.W_qkv, inp.W_o, cfg.H, residual=residual)
    return cfg, inp, fwd, bwd


def device_inputs(cfg, inp):
    names = ("x", "w_g", "W_qkv", "b_qkv", "W_o", "b_o", "dY")
    return {n: dev(getattr(inp, n), cfg.dtype) for n in names}


def make_block(cfg, flags=0, capacity=None, tau=None, fused=None):
    from paper_2410_23608_b200.block import SpaBlock
    return SpaBlock(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, tau=cfg.tau if tau is None else tau, flags=flags,
                    capacity=capacity, fused=fused)


def check_indices(blk, fwd):
    Np = int(fwd["cu_seqlens"][-1])
    assert np.array_equal(blk.mask.cpu().numpy().astype(bool), fwd["mask"].reshape(-1))
    assert np.array_equal(blk.cu.cpu().numpy(), fwd["cu_seqlens"])
    assert np.array_equal(blk.idx.cpu().numpy()[:Np], fwd["idx"])
    assert np.array_equal(blk.inv.cpu().numpy(), fwd["inv"])
    return Np


# (config, extra flags); 8 = fp32-FMA kernels, 16 = one-CTA GEMMs where CTA pairs would be used (configs 4, 5),
# 64 = one-pass attention backward for segments of at most 128 rows (all of config 5, most of 2, half of 4)
VARIANTS = [(1, 0), (2, 0), (2, 8), (2, 64), (3, 0), (3, 8), (4, 0), (4, 16), (4, 64), (5, 0), (5, 8), (5, 64)]
# the same with the unpack scatter either fused into the matrix products (tensor-core problems) or as kernels of its own
E2E_VARIANTS = [(ci, fl, False) for ci, fl in VARIANTS] + [(ci, 0, True) for ci in (2, 3, 4, 5)]


@pytest.mark.parametrize("ci,xflags,fused", E2E_VARIANTS)
def test_block_forward_backward_end_to_end(ci, xflags, fused):
    cfg, inp, fwd, bwd = problem(ci)
    d = device_inputs(cfg, inp)
    blk = make_block(cfg, flags=xflags, fused=fused)
    y = blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
    dX = blk.backward(d["dY"])
    torch.cuda.synchronize()
    assert blk.read_status() == 0
    dt = cfg.dtype
    Np = check_indices(blk, fwd)
    assert np.abs(host(blk.scores) - fwd["scores"].reshape(-1)).max() <= TOL[dt]["score"]
    assert np.array_equal(host(blk.xp)[:Np], fwd["xp"])            # a pure row gather: exact
    assert_close(host(blk.qkv)[:Np], fwd["qkv"], dt, "qkv")
    assert_close(host(blk.ao)[:Np], fwd["ao"], dt, "attn_out")
    assert np.abs(host(blk.lse)[:, :Np] - fwd["lse"]).max() <= TOL[dt]["lse_chain"]
    if not fused:
        assert_close(host(blk.z)[:Np], fwd["z"], dt, "z")
    yh = host(y)
    assert_close(yh, fwd["y"], dt, "y")
    unsel = ~fwd["mask"]
    assert np.array_equal(yh[unsel], inp.x[unsel])                 # pass-through rows: bitwise
    # backward
    assert np.array_equal(host(blk.dz)[:Np], bwd["dz"])
    assert_close(host(blk.dao)[:Np], bwd["dao"], dt, "d_attn_out", scale_max_abs=True)
    assert_close(host(blk.dqkv)[:Np], bwd["dqkv"], dt, "dqkv", scale_max_abs=True)
    if not fused:
        assert_close(host(blk.dxp)[:Np], bwd["dxp"], dt, "dx_packed", scale_max_abs=True)
    dXh = host(dX)
    assert_close(dXh, bwd["dX"], dt, "dX", scale_max_abs=True)
    assert np.array_equal(dXh[unsel], inp.dY[unsel])
    for name in ("dW_qkv", "db_qkv", "dW_o", "db_o"):
        assert_close(host(getattr(blk, name)), bwd[name], dt, name, scale_max_abs=True)


@pytest.mark.parametrize("ci,xflags", VARIANTS)
def test_each_call_on_oracle_upstream(ci, xflags):
    """Every call is fed the oracle's own upstream tensors (rounded to the storage dtype), so an error
    cannot hide behind, or be blamed on, an earlier step."""
    from paper_2410_23608_b200 import binding as L
    cfg, inp, fwd, bwd = problem(ci)
    dt = cfg.dtype
    d = device_inputs(cfg, inp)
    blk = make_block(cfg, flags=xflags)
    p = blk.p
    Np = int(fwd["cu_seqlens"][-1])
    cap = blk.cap
    cu = torch.from_numpy(fwd["cu_seqlens"]).cuda()
    H, C = cfg.H, cfg.C

    def padded(a, cols):
        buf = np.zeros((cap, cols))
        buf[:Np] = a
        return buf

    # QKV on the oracle's packed rows (exact copies of x rows)
    xp = dev(padded(fwd["xp"], C), dt)
    L.spa_packed_qkv(p, xp, d["W_qkv"], d["b_qkv"], cu, blk.qkv, blk.status)
    assert_close(host(blk.qkv)[:Np], fwd["qkv"], dt, "qkv")
    # attention on the oracle's qkv, rounded
    qkv_r = round_to(fwd["qkv"], dt)
    ao_ref, lse_ref = O.attention_fwd(qkv_r, fwd["cu_seqlens"], H)
    qkv = dev(padded(qkv_r, 3 * C), dt)
    L.spa_packed_attention_fwd(p, qkv, cu, cfg.B, blk.ao, blk.lse, blk.status)
    assert_close(host(blk.ao)[:Np], ao_ref, dt, "attn_out")
    assert np.abs(host(blk.lse)[:, :Np] - lse_ref).max() <= TOL[dt]["lse"]
    # projection
    ao_r = round_to(ao_ref, dt)
    L.spa_packed_proj(p, dev(padded(ao_r, C), dt), d["W_o"], d["b_o"], cu, blk.z, blk.status)
    assert_close(host(blk.z)[:Np], O.linear(ao_r, inp.W_o, inp.b_o), dt, "z")
    # attention backward on rounded oracle tensors
    dao_r = round_to(bwd["dao"], dt)
    lse_t = torch.zeros(H, cap, dtype=torch.float32, device="cuda")
    lse_t[:, :Np] = torch.from_numpy(lse_ref).float().cuda()
    dqkv_ref = O.attention_bwd(qkv_r, ao_r, lse_t[:, :Np].double().cpu().numpy(), dao_r, fwd["cu_seqlens"], H)
    L.spa_packed_attention_bwd(p, qkv, dev(padded(ao_r, C), dt), lse_t, dev(padded(dao_r, C), dt), cu, cfg.B,
                               blk.dqkv, blk.workspace, blk.status)
    assert_close(host(blk.dqkv)[:Np], dqkv_ref, dt, "dqkv", scale_max_abs=True)
    # linear backward (QKV layer) on rounded oracle tensors
    dqkv_r = round_to(bwd["dqkv"], dt)
    da_ref, dW_ref, db_ref = O.linear_bwd(fwd["xp"], inp.W_qkv, dqkv_r)
    L.spa_packed_linear_bwd(p, xp, d["W_qkv"], dev(padded(dqkv_r, 3 * C), dt), C, 3 * C, cu, blk.dxp, blk.dW_qkv,
                            blk.db_qkv, blk.workspace, blk.status)
    assert_close(host(blk.dxp)[:Np], da_ref, dt, "dx_packed", scale_max_abs=True)
    assert_close(host(blk.dW_qkv), dW_ref, dt, "dW_qkv", scale_max_abs=True)
    assert_close(host(blk.db_qkv), db_ref, dt, "db_qkv", scale_max_abs=True)
    torch.cuda.synchronize()
    assert blk.read_status() == 0


@pytest.mark.parametrize("ci,fused", [(1, False), (2, False), (2, True)])
@pytest.mark.parametrize("flags", [1, 2, 3])   # residual, in-place, both
def test_residual_and_inplace_flags(ci, fused, flags):
    residual = bool(flags & 1)
    cfg, inp, fwd, bwd = problem(ci, residual)
    d = device_inputs(cfg, inp)
    blk = make_block(cfg, flags=flags, fused=fused)
    x = d["x"].clone()
    y = blk.forward(x, d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
    if flags & 2:
        assert y.data_ptr() == x.data_ptr()
    assert_close(host(y), fwd["y"], cfg.dtype, "y")
    unsel = ~fwd["mask"]
    assert np.array_equal(host(y)[unsel], inp.x[unsel])
    dX = blk.backward(d["dY"])
    assert_close(host(dX), bwd["dX"], cfg.dtype, "dX", scale_max_abs=True)
    # dX aliasing dY: only the selected rows are rewritten
    dY2 = d["dY"].clone()
    dX2 = blk.backward(dY2, dX=dY2)
    assert torch.equal(dX2, dX)
    assert blk.read_status() == 0


def test_fused_calls_on_oracle_upstream():
    """spa_unpack_prefill + spa_packed_proj_scatter, and spa_packed_linear_bwd_scatter, each fed the oracle's
    own upstream tensors."""
    from paper_2410_23608_b200 import binding as L
    cfg, inp, fwd, bwd = problem(2)
    dt = cfg.dtype
    d = device_inputs(cfg, inp)
    blk = make_block(cfg)
    p, C, cap = blk.p, cfg.C, blk.cap
    assert L.spa_fused_scatter_supported(p)
    Np = int(fwd["cu_seqlens"][-1])
    cu = torch.from_numpy(fwd["cu_seqlens"]).cuda()
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    idx[:Np] = torch.from_numpy(fwd["idx"]).cuda()

    def padded(a, cols):
        buf = np.zeros((cap, cols))
        buf[:Np] = a
        return buf

    # forward: y = x, then the projection writes the selected rows
    y = torch.empty_like(d["x"])
    L.spa_unpack_prefill(p, d["x"], y)
    assert torch.equal(y, d["x"])
    ao_r = round_to(fwd["ao"], dt)
    L.spa_packed_proj_scatter(p, dev(padded(ao_r, C), dt), d["W_o"], d["b_o"], idx, cu, y, blk.status)
    y_ref = O.unpack_scatter(O.linear(ao_r, inp.W_o, inp.b_o), inp.x, fwd["idx"])
    assert_close(host(y), y_ref, dt, "y")
    unsel = ~fwd["mask"]
    assert np.array_equal(host(y)[unsel], inp.x[unsel])
    # backward: dX = dY, then the input gradient of the QKV layer writes the selected rows
    dX = torch.empty_like(d["dY"])
    L.spa_unpack_prefill(p, d["dY"], dX)
    dqkv_r = round_to(bwd["dqkv"], dt)
    da_ref, dW_ref, db_ref = O.linear_bwd(fwd["xp"], inp.W_qkv, dqkv_r)
    L.spa_packed_linear_bwd_scatter(p, dev(padded(fwd["xp"], C), dt), d["W_qkv"], dev(padded(dqkv_r, 3 * C), dt), C,
                                    3 * C, idx, cu, dX, blk.dW_qkv, blk.db_qkv, blk.workspace, blk.status)
    dX_ref = O.select_pack_bwd(da_ref, fwd["idx"], O.unpack_scatter_bwd(inp.dY, fwd["idx"])[1])
    assert_close(host(dX), dX_ref, dt, "dX", scale_max_abs=True)
    assert np.array_equal(host(dX)[unsel], inp.dY[unsel])
    assert_close(host(blk.dW_qkv), dW_ref, dt, "dW_qkv", scale_max_abs=True)
    assert_close(host(blk.db_qkv), db_ref, dt, "db_qkv", scale_max_abs=True)
    torch.cuda.synchronize()
    assert blk.read_status() == 0


def test_fused_scatter_matches_separate_kernels_bitwise():
    """The fused calls round exactly as the separate projection + scatter kernels do."""
    cfg, inp, fwd, bwd = problem(2, True)
    d = device_inputs(cfg, inp)
    outs = []
    for fused in (False, True):
        blk = make_block(cfg, flags=1, fused=fused)   # residual: the scatter accumulates
        y = blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
        dX = blk.backward(d["dY"])
        torch.cuda.synchronize()
        assert blk.read_status() == 0
        outs.append((y.clone(), dX.clone(), blk.dW_qkv.clone(), blk.dW_o.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_run_to_run_determinism():
    cfg, inp, fwd, bwd = problem(2)
    d = device_inputs(cfg, inp)
    outs = []
    for _ in range(2):
        blk = make_block(cfg)
        y = blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
        dX = blk.backward(d["dY"])
        Np = int(fwd["cu_seqlens"][-1])
        outs.append([t.clone() for t in (y, dX, blk.dW_qkv, blk.db_qkv, blk.dW_o, blk.db_o, blk.dqkv[:Np])])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("ci", [2, 4])
def test_graph_replay_is_stable_and_reproducible(ci):
    """The whole step as one CUDA graph (second stream, programmatic dependent launches), replayed many times:
    no device-side wait may expire and every replay must give the same bits as the first."""
    cfg, inp, fwd, bwd = problem(ci)
    d = device_inputs(cfg, inp)
    blk = make_block(cfg)

    def step():
        blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
        blk.backward(d["dY"])

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    g.replay()
    torch.cuda.synchronize()
    outs = (blk.y, blk.dX, blk.dW_qkv, blk.db_qkv, blk.dW_o, blk.db_o)
    first = [t.clone() for t in outs]
    for _ in range(300):
        g.replay()
    torch.cuda.synchronize()
    assert blk.read_status() == 0
    for a, b in zip(first, outs):
        assert torch.equal(a, b)
    assert_close(host(blk.y), fwd["y"], cfg.dtype, "y")


CANARY = 0x5A


def guarded(shape, dtype, guard_rows=2):
    """A device buffer with `guard_rows` extra rows before and after it, every byte set to a fixed pattern; returns
    (the inner view, a function that checks that the guard rows still hold the pattern)."""
    rows = shape[0] if len(shape) > 1 else 1
    row_elems = int(np.prod(shape[1:])) if len(shape) > 1 else int(shape[0])
    # a guard row is one row of the buffer, rounded up so that the inner view stays 256-byte aligned
    esz = torch.empty(0, dtype=dtype).element_size()
    g = ((guard_rows * row_elems * esz + 255) // 256) * 256
    inner_bytes = rows * row_elems * esz
    raw = torch.full((g + inner_bytes + g,), CANARY, dtype=torch.uint8, device="cuda")
    inner = raw[g:g + inner_bytes].view(dtype).view(*shape)

    def intact():
        return bool((raw[:g] == CANARY).all()) and bool((raw[g + inner_bytes:] == CANARY).all())

    return inner, intact


# flags 32: separate scatter kernels; 1: residual.  one_pass: gate, selection and packing as one kernel
@pytest.mark.parametrize("ci,flags,one_pass", [(1, 0, False), (2, 0, False), (2, 32, False), (2, 1, False),
                                               (1, 0, True), (2, 0, True), (4, 1, True)])
def test_block_calls_alone_with_guard_bands(ci, flags, one_pass):
    """One forward and one backward pass through nothing but spa_block_fwd / spa_block_bwd (no Python class in
    between), every buffer the library writes framed by guard rows that must come back untouched."""
    from paper_2410_23608_b200 import binding as L
    cfg, inp, fwd, bwd = problem(ci, residual=bool(flags & 1))
    d = device_inputs(cfg, inp)
    B, N, C, H, dt = cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype
    T = torch.float32 if dt == "f32" else torch.bfloat16
    cap = B * N
    p = L.make_params(B, N, C, H, dt, cap, flags, cfg.tau)
    f32, i32, u8 = torch.float32, torch.int32, torch.uint8
    spec = dict(scores=((cap,), f32), mask=((cap,), u8), cu_seqlens=((B + 1,), i32), idx=((cap,), i32),
                inv=((cap,), i32), x_packed=((cap, C), T), qkv=((cap, 3 * C), T), attn_out=((cap, C), T),
                lse=((H, cap), f32), z=((cap, C), T), y=((B * N, C), T), dz=((cap, C), T), d_attn_out=((cap, C), T),
                dqkv=((cap, 3 * C), T), dx_packed=((cap, C), T), dX=((B * N, C), T), dW_qkv=((3 * C, C), f32),
                db_qkv=((3 * C,), f32), dW_o=((C, C), f32), db_o=((C,), f32))
    buf, checks = {}, {}
    for name, (shape, dtype) in spec.items():
        buf[name], checks[name] = guarded(shape, dtype)
    ws_bytes = max(L.spa_workspace_bytes(p), 256)
    buf["workspace"], checks["workspace"] = guarded((ws_bytes,), u8)
    buf["workspace_side"], checks["workspace_side"] = guarded((ws_bytes,), u8)
    if one_pass:
        buf["pack_state"], checks["pack_state"] = guarded((max(L.spa_pack_state_bytes(p), 256),), u8)
        buf["pack_state"].zero_()
    status = torch.zeros(4, dtype=i32, device="cuda")
    ov = L.spa_overlap_create()
    try:
        bufs = L.block_buffers(x=d["x"], w_g=d["w_g"], b_g=float(inp.b_g), W_qkv=d["W_qkv"], b_qkv=d["b_qkv"],
                               W_o=d["W_o"], b_o=d["b_o"], dY=d["dY"], overlap=ov, d_status=status, **buf)
        L.spa_block_fwd(p, bufs)
        L.spa_block_bwd(p, bufs)
        torch.cuda.synchronize()
    finally:
        L.spa_overlap_destroy(ov)
    assert L.spa_read_status(status) == 0
    if one_pass:
        assert not buf["pack_state"].any()          # the kernel leaves its scratch zeroed
    touched = [name for name, ok in checks.items() if not ok()]
    assert not touched, f"writes outside the buffer: {touched}"
    Np = int(fwd["cu_seqlens"][-1])
    assert np.array_equal(buf["cu_seqlens"].cpu().numpy(), fwd["cu_seqlens"])
    assert np.array_equal(buf["idx"].cpu().numpy()[:Np], fwd["idx"])
    assert np.array_equal(buf["inv"].cpu().numpy(), fwd["inv"])
    assert np.array_equal(buf["mask"].cpu().numpy().astype(bool), fwd["mask"].reshape(-1))
    yh, dXh = host(buf["y"]).reshape(B, N, C), host(buf["dX"]).reshape(B, N, C)
    assert_close(yh, fwd["y"], dt, "y")
    assert_close(dXh, bwd["dX"], dt, "dX", scale_max_abs=True)
    unsel = ~fwd["mask"]
    assert np.array_equal(yh[unsel], inp.x[unsel])
    if not flags & 1:
        assert np.array_equal(dXh[unsel], inp.dY[unsel])
    for name in ("dW_qkv", "db_qkv", "dW_o", "db_o"):
        assert_close(host(buf[name]), bwd[name], dt, name, scale_max_abs=True)
