"""GPU test of the one-pass gate + selection + packing call against the oracle and against the two separate calls
(bit for bit), through the C boundary: all five workloads, the optional inputs, the degenerate selections, an
undersized capacity, and repeated calls that share one state array."""
import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from spa_workloads import get_config, make_inputs, scaled_config
from tests.gpu_util import dev, host

pytestmark = pytest.mark.gpu


def buffers(B, N, C, T, cap):
    mk = lambda shape, dt: torch.empty(*shape, dtype=dt, device="cuda")
    return dict(scores=mk((B * N,), torch.float32), mask=mk((B * N,), torch.uint8), y=mk((B, N, C), T),
                xp=mk((cap, C), T).fill_(0), idx=mk((cap,), torch.int32).fill_(-7), inv=mk((B * N,), torch.int32),
                cu=mk((B + 1,), torch.int32).fill_(-1))


def run_both(L, p, x, w_g, b_g, s_up, T, cap, with_y=True):
    B, N, C = p.B, p.N, p.C
    a, b = buffers(B, N, C, T, cap), buffers(B, N, C, T, cap)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    state = torch.zeros(max(L.spa_pack_state_bytes(p), 256), dtype=torch.uint8, device="cuda")
    L.spa_gate_select_pack(p, x, w_g, b_g, s_up, a["scores"], a["mask"], a["y"] if with_y else None, a["xp"], a["idx"],
                           a["inv"], a["cu"], state, status)
    if with_y:
        L.spa_gate_prefill(p, x, w_g, b_g, s_up, b["scores"], b["mask"], b["y"])
    else:
        L.spa_gate(p, x, w_g, b_g, s_up, b["scores"], b["mask"])
    L.spa_select_pack(p, x, b["mask"], b["scores"], b["xp"], b["idx"], b["inv"], b["cu"], status)
    torch.cuda.synchronize()
    assert not state.any(), "the state array must come back zeroed"
    return a, b, status, state


@pytest.mark.parametrize("ci,B", [(1, None), (2, None), (3, None), (4, None), (5, None), (2, 1), (3, 1)])
def test_one_pass_equals_two_calls_and_the_oracle(ci, B):
    from paper_2410_23608_b200 import binding as L
    cfg = get_config(ci) if B is None else scaled_config(get_config(ci), B=B)
    inp = make_inputs(cfg)
    T = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    cap = cfg.B * cfg.N
    p = L.make_params(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, cap, 0, cfg.tau)
    assert L.spa_gate_select_pack_supported(p)
    x, w_g = dev(inp.x, cfg.dtype), dev(inp.w_g, cfg.dtype)
    a, b, status, _ = run_both(L, p, x, w_g, inp.b_g, None, T, cap)
    assert L.spa_read_status(status) == 0
    s = O.gate(inp.x, inp.w_g, inp.b_g)
    mask = O.select(s, inp.tau)
    cu, idx, inv = O.pack_indices(mask)
    Np = int(cu[-1])
    assert np.array_equal(a["mask"].cpu().numpy().astype(bool), mask.reshape(-1))
    assert np.array_equal(a["cu"].cpu().numpy(), cu)
    assert np.array_equal(a["idx"].cpu().numpy()[:Np], idx)
    assert np.array_equal(a["inv"].cpu().numpy(), inv)
    assert np.array_equal(host(a["xp"])[:Np], O.pack_rows(inp.x, idx))
    assert np.abs(host(a["scores"]) - s.reshape(-1)).max() <= 1e-4
    assert torch.equal(a["y"], x)
    for name in ("scores", "mask", "cu", "inv", "y"):
        assert torch.equal(a[name], b[name]), name
    assert torch.equal(a["idx"][:Np], b["idx"][:Np]) and torch.equal(a["xp"][:Np], b["xp"][:Np])


@pytest.mark.parametrize("tau", [float("inf"), float("-inf")])
def test_one_pass_none_and_all_selected(tau):
    from paper_2410_23608_b200 import binding as L
    cfg = scaled_config(get_config(2), B=5)
    inp = make_inputs(cfg)
    cap = cfg.B * cfg.N
    p = L.make_params(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, cap, 0, tau)
    x, w_g = dev(inp.x, cfg.dtype), dev(inp.w_g, cfg.dtype)
    a, b, status, _ = run_both(L, p, x, w_g, inp.b_g, None, torch.bfloat16, cap, with_y=False)
    assert L.spa_read_status(status) == 0
    n = 0 if tau > 0 else cfg.N
    assert np.array_equal(a["cu"].cpu().numpy(), np.arange(cfg.B + 1) * n)
    if n:
        assert torch.equal(a["xp"], x.view(cap, cfg.C))
        assert np.array_equal(a["idx"].cpu().numpy(), np.arange(cap)) and np.array_equal(a["inv"].cpu().numpy(), np.arange(cap))
    else:
        assert bool((a["inv"] == -1).all())


def test_one_pass_with_upscale_scores_gate_scale_and_small_capacity():
    from paper_2410_23608_b200 import binding as L
    cfg = scaled_config(get_config(2), B=6)
    inp = make_inputs(cfg)
    rng = np.random.default_rng(3)
    s_up_np = (rng.normal(size=(cfg.B, cfg.N)) * 3).astype(np.float32)
    s = O.gate(inp.x, inp.w_g, inp.b_g, s_up_np)
    assert np.abs(s - inp.tau).min() > 1e-3
    mask = O.select(s, inp.tau)
    cu, idx, inv = O.pack_indices(mask)
    Np = int(cu[-1])
    x, w_g = dev(inp.x, cfg.dtype), dev(inp.w_g, cfg.dtype)
    s_up = torch.from_numpy(s_up_np.reshape(-1)).cuda()
    for cap, flags in ((cfg.B * cfg.N, L.SPA_FLAG_GATE_SCALE), (Np - 37, 0)):
        p = L.make_params(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, cap, flags, cfg.tau)
        a, b, status, _ = run_both(L, p, x, w_g, inp.b_g, s_up, torch.bfloat16, cap)
        assert L.spa_read_status(status) == (0 if cap >= Np else L.SPA_ERR_CAPACITY)
        assert np.array_equal(a["cu"].cpu().numpy(), cu)                 # the true counts, also when rows are dropped
        n_ok = min(Np, cap)
        assert np.array_equal(a["idx"].cpu().numpy()[:n_ok], idx[:n_ok])
        for name in ("scores", "mask", "cu", "inv", "y"):
            assert torch.equal(a[name], b[name]), name
        assert torch.equal(a["xp"][:n_ok], b["xp"][:n_ok])


def test_one_pass_repeated_calls_and_graph_replay_share_one_state():
    """The state array is cleared by the kernel itself: many calls in a row, eager and replayed from a CUDA graph,
    on different inputs, each give the oracle's indices."""
    from paper_2410_23608_b200 import binding as L
    cfg = scaled_config(get_config(3), B=3)
    cap = cfg.B * cfg.N
    p = L.make_params(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, cap, 0, cfg.tau)
    state = torch.zeros(max(L.spa_pack_state_bytes(p), 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    o = buffers(cfg.B, cfg.N, cfg.C, torch.bfloat16, cap)
    cases = []
    for seed in (0, 1):
        inp = make_inputs(scaled_config(cfg, seed=50 + seed))
        mask = O.select(O.gate(inp.x, inp.w_g, inp.b_g), inp.tau)
        cases.append((inp, dev(inp.x, cfg.dtype), dev(inp.w_g, cfg.dtype), O.pack_indices(mask)))
    xs = torch.empty_like(cases[0][1])
    ws = torch.empty_like(cases[0][2])

    def call(b_g):
        L.spa_gate_select_pack(p, xs, ws, b_g, None, o["scores"], o["mask"], None, o["xp"], o["idx"], o["inv"], o["cu"],
                               state, status)

    assert cases[0][0].b_g == pytest.approx(cases[1][0].b_g, rel=0.2)
    for rep in range(6):
        inp, x, w, (cu, idx, inv) = cases[rep % 2]
        xs.copy_(x); ws.copy_(w)
        call(inp.b_g)
        torch.cuda.synchronize()
        assert np.array_equal(o["cu"].cpu().numpy(), cu) and np.array_equal(o["inv"].cpu().numpy(), inv)
    inp, x, w, (cu, idx, inv) = cases[0]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call(inp.b_g)
        call(inp.b_g)
    for rep in range(20):
        xs.copy_(x); ws.copy_(w)
        g.replay()
    torch.cuda.synchronize()
    assert L.spa_read_status(status) == 0 and not state.any()
    assert np.array_equal(o["cu"].cpu().numpy(), cu) and np.array_equal(o["idx"].cpu().numpy()[:idx.size], idx)
