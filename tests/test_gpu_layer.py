"""GPU parity of the pre-norm transformer block around SPA (LayerNorm, SPA with residual, feed-forward with GELU)
against the fp64 oracle, call by call and as a whole, through the C boundary."""
import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from spa_workloads import get_config, make_inputs, scaled_config
from tests.gpu_util import TOL, assert_close, dev, host, round_to

pytestmark = pytest.mark.gpu


def layer_problem(ci, B):
    cfg = scaled_config(get_config(ci), B=B)
    inp = make_inputs(cfg)
    rng = np.random.default_rng(200 + ci)
    C, Hd, dt = cfg.C, 4 * cfg.C, cfg.dtype
    r = lambda a: round_to(a, dt)
    prm = dict(g1=r(1 + 0.1 * rng.normal(size=C)), be1=r(0.1 * rng.normal(size=C)), g2=r(1 + 0.1 * rng.normal(size=C)),
               be2=r(0.1 * rng.normal(size=C)), W1=r(rng.normal(size=(Hd, C)) / np.sqrt(C)), b1=r(0.02 * rng.normal(size=Hd)),
               W2=r(rng.normal(size=(C, Hd)) / np.sqrt(Hd)), b2=r(0.02 * rng.normal(size=C)),
               W_qkv=inp.W_qkv, b_qkv=inp.b_qkv, W_o=inp.W_o, b_o=inp.b_o)
    # a gate direction and bias that select about 40 % of the normalised tokens with a clear margin
    z, _, _ = O.layer_norm(inp.x, prm["g1"], prm["be1"])
    w_g = r(rng.normal(size=C) / np.sqrt(C))
    s = z.reshape(-1, C) @ w_g
    b_g = float(np.float32(-np.quantile(s, 0.6)))
    bad = np.abs(s + b_g) < 2e-2
    x = inp.x.copy()
    if bad.any():   # move tokens that sit near the threshold well below it
        flat = x.reshape(-1, C)
        flat[bad] = r(flat[bad] * 0.0 + rng.normal(size=(int(bad.sum()), C)) - 3.0 * np.sign(w_g))
    prm["w_g"], prm["b_g"] = w_g, b_g
    f = O.layer_fwd(x, prm, cfg.H)
    assert np.abs(f["spa"]["scores"]).min() > 5e-3
    return cfg, inp, x, prm, f


# C = 96, 384, 256 and 768: every row-width instantiation of the LayerNorm backward; (4, 8) has 4 608 tokens, so its
# 768 -> 3072 -> 768 feed-forward products and their input gradients run on CTA pairs
@pytest.mark.parametrize("ci,B", [(1, 3), (2, 4), (3, 1), (4, 8)])
def test_layer_forward_backward(ci, B):
    from paper_2410_23608_b200.layer import SpaLayer
    cfg, inp, x, prm, f = layer_problem(ci, B)
    bwd = O.layer_bwd(f, inp.dY, x, prm, cfg.H)
    dt = cfg.dtype
    dprm = {k: (dev(v, dt) if isinstance(v, np.ndarray) else v) for k, v in prm.items()}
    lay = SpaLayer(cfg.B, cfg.N, cfg.C, cfg.H, dt)
    out = lay.forward(dev(x, dt), dprm)
    dX = lay.backward(dev(inp.dY, dt))
    torch.cuda.synchronize()
    assert lay.read_status() == 0
    spa = f["spa"]
    assert np.array_equal(lay.blk.mask.cpu().numpy().astype(bool), spa["mask"].reshape(-1))
    assert np.array_equal(lay.blk.cu.cpu().numpy(), spa["cu_seqlens"])
    assert_close(host(lay.z), f["z"], dt, "LN1(x)")
    assert_close(host(lay.y1), f["y1"], dt, "y1", scale_max_abs=True)
    unsel = ~spa["mask"]
    assert np.array_equal(host(lay.y1)[unsel], x[unsel])            # no attention update off the selection
    assert_close(host(lay.t), f["t"], dt, "LN2(y1)", scale_max_abs=True)
    assert_close(host(lay.u), f["u"], dt, "u", scale_max_abs=True)
    assert_close(host(lay.h), f["h"], dt, "gelu(u)", scale_max_abs=True)
    assert_close(host(out), f["out"], dt, "out", scale_max_abs=True)
    assert_close(host(dX), bwd["dX"], dt, "dX", scale_max_abs=True)
    for name in ("dW1", "db1", "dW2", "db2", "dg1", "dbe1", "dg2", "dbe2"):
        assert_close(host(getattr(lay, name)), bwd[name], dt, name, scale_max_abs=True)
    for name in ("dW_qkv", "db_qkv", "dW_o", "db_o"):
        assert_close(host(getattr(lay.blk, name)), bwd[name], dt, name, scale_max_abs=True)


@pytest.mark.parametrize("ci", [2, 3, 4])   # C = 384, 256, 768
def test_layer_norm_and_gelu_calls_alone(ci):
    """Each new call on its own inputs: LayerNorm forward / backward (with and without the added branch), GELU."""
    from paper_2410_23608_b200 import binding as L
    from paper_2410_23608_b200.block import SpaBlock
    cfg = scaled_config(get_config(ci), B=2 if ci != 3 else 1)
    dt = cfg.dtype
    rng = np.random.default_rng(9)
    B, N, C = cfg.B, cfg.N, cfg.C
    blk = SpaBlock(B, N, C, cfg.H, dt)
    x = round_to(rng.normal(size=(B, N, C)) * 2 + 0.3, dt)
    g, b = round_to(1 + 0.2 * rng.normal(size=C), dt), round_to(0.2 * rng.normal(size=C), dt)
    dy = round_to(rng.normal(size=(B, N, C)), dt)
    add = round_to(rng.normal(size=(B, N, C)), dt)
    y_ref, mean, rstd = O.layer_norm(x, g, b)
    dx_ref, dg_ref, db_ref = O.layer_norm_bwd(dy, x, g, mean, rstd)
    y = torch.empty(B, N, C, dtype=torch.bfloat16, device="cuda")
    m = torch.empty(B * N, dtype=torch.float32, device="cuda")
    r = torch.empty_like(m)
    L.spa_layer_norm(blk.p, dev(x, dt), dev(g, dt), dev(b, dt), 1e-5, y, m, r)
    assert_close(host(y), y_ref, dt, "y")
    assert np.abs(m.cpu().numpy() - mean.reshape(-1)).max() <= 1e-5 and np.abs(r.cpu().numpy() / rstd.reshape(-1) - 1).max() <= 1e-5
    ws = torch.empty(L.spa_train_workspace_bytes(blk.p), dtype=torch.uint8, device="cuda")
    dg = torch.empty(C, dtype=torch.float32, device="cuda")
    dbt = torch.empty(C, dtype=torch.float32, device="cuda")
    for with_add in (False, True):
        dx = torch.empty_like(y)
        L.spa_layer_norm_bwd(blk.p, dev(dy, dt), dev(x, dt), dev(g, dt), m, r, dev(add, dt) if with_add else None, dx, dg, dbt, ws)
        assert_close(host(dx), dx_ref + (add if with_add else 0.0), dt, "dx", scale_max_abs=True)
        assert_close(dg.cpu().numpy().astype(np.float64), dg_ref, dt, "dgamma", scale_max_abs=True)
        assert_close(dbt.cpu().numpy().astype(np.float64), db_ref, dt, "dbeta", scale_max_abs=True)
    u = round_to(rng.normal(size=(B * N, 4 * C)) * 2, dt)
    dh = round_to(rng.normal(size=(B * N, 4 * C)), dt)
    h = torch.empty(B * N, 4 * C, dtype=torch.bfloat16, device="cuda")
    L.spa_gelu(blk.p, dev(u, dt), 4 * C, h)
    assert_close(host(h), O.gelu(u), dt, "gelu")
    du = dev(dh, dt)
    L.spa_gelu_bwd(blk.p, du, dev(u, dt), 4 * C, du)      # in place
    assert_close(host(du), dh * O.gelu_grad(u), dt, "gelu_bwd")


def test_two_blocks_in_one_graph():
    """A stage of two blocks with its own selection in each, captured as one CUDA graph and replayed: the second
    block's gate sees the first block's output, nothing returns to the host in between."""
    from paper_2410_23608_b200.layer import SpaLayer
    cfg, inp, x, prm, f1 = layer_problem(2, 3)
    dt = cfg.dtype
    dprm = {k_: (dev(v, dt) if isinstance(v, np.ndarray) else v) for k_, v in prm.items()}
    a, b = SpaLayer(cfg.B, cfg.N, cfg.C, cfg.H, dt), SpaLayer(cfg.B, cfg.N, cfg.C, cfg.H, dt)
    xd = dev(x, dt)
    a.forward(xd, dprm)
    torch.cuda.synchronize()
    assert_close(host(a.out), f1["out"], dt, "block 1", scale_max_abs=True)
    # the oracle's second block reads the very bits the device's first block wrote (runs are reproducible), with
    # the threshold of the second gate placed in the widest gap of its scores
    x2 = host(a.out)
    z2, _, _ = O.layer_norm(x2, prm["g1"], prm["be1"])
    srt = np.sort(z2.reshape(-1, cfg.C) @ prm["w_g"])
    lo, hi = len(srt) // 3, 2 * len(srt) // 3
    k = int(np.argmax(np.diff(srt)[lo:hi])) + lo
    assert srt[k + 1] - srt[k] > 2e-3
    prm2 = dict(prm)
    prm2["b_g"] = float(np.float32(-(srt[k] + srt[k + 1]) / 2))
    f2 = O.layer_fwd(x2, prm2, cfg.H)
    dprm2 = dict(dprm)
    dprm2["b_g"] = prm2["b_g"]

    def stage():
        return b.forward(a.forward(xd, dprm), dprm2)

    stage()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = stage()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    assert a.read_status() == 0 and b.read_status() == 0
    assert np.array_equal(host(a.out), x2)                      # block 1 reproduced bit for bit inside the graph
    assert np.array_equal(b.blk.mask.cpu().numpy().astype(bool), f2["spa"]["mask"].reshape(-1))
    assert 0 < int(b.blk.cu[-1].item()) < cfg.B * cfg.N
    assert_close(host(out), f2["out"], dt, "block 2", scale_max_abs=True)
