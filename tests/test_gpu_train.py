"""GPU parity of the trainable-selection calls (up-scale score pooling, selection loss, backward through the
sigmoid scaling and the gate) against the fp64 oracle, through the C boundary."""
import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from spa_workloads import get_config, make_inputs
from tests.gpu_util import TOL, assert_close, dev, host

pytestmark = pytest.mark.gpu


def test_score_pool_exact():
    from paper_2410_23608_b200 import binding as L
    rng = np.random.default_rng(7)
    B, rows, cols = 3, 14, 14
    prev = rng.normal(size=(B, 2 * rows, 2 * cols)).astype(np.float32)
    out = torch.empty(B, rows * cols, dtype=torch.float32, device="cuda")
    L.spa_score_pool(torch.from_numpy(prev).cuda(), B, rows, cols, out)
    assert np.array_equal(out.cpu().numpy(), O.score_pool(prev, B, rows, cols).astype(np.float32))


def _problem(ci, residual, B=None):
    from spa_workloads import scaled_config
    cfg = get_config(ci) if B is None else scaled_config(get_config(ci), B=B)
    inp = make_inputs(cfg)
    rng = np.random.default_rng(100 + ci)
    s_lin = O.gate(inp.x, inp.w_g, inp.b_g)
    # an up-scale score map that wins on about a third of the tokens, never within 1e-2 of the linear score
    # and never across the threshold (the selection stays the generator's)
    win = rng.uniform(size=s_lin.shape) < 0.33
    s_up = np.where(win & (s_lin > inp.tau + 0.1), s_lin + rng.uniform(0.05, 1.0, size=s_lin.shape),
                    np.where(s_lin > inp.tau, s_lin - rng.uniform(0.05, 1.0, size=s_lin.shape), s_lin - 1.0))
    s_up = s_up.astype(np.float32).astype(np.float64)
    labels = (rng.uniform(size=s_lin.shape) < 0.4)
    fwd = O.block_fwd(inp.x, inp.w_g, inp.b_g, inp.tau, inp.W_qkv, inp.b_qkv, inp.W_o, inp.b_o, cfg.H, s_up=s_up,
                      residual=residual, gate_scale=True)
    return cfg, inp, s_up, labels, fwd


# configs 3-5 (C = 256 and 768: the widest rows of the gate backward and of the gated pack transpose) on a slice
# of their batch
@pytest.mark.parametrize("ci,residual,B", [(1, False, None), (2, False, None), (2, True, None), (3, False, 2),
                                            (4, True, 4), (5, False, 12)])
def test_trainable_block_against_oracle(ci, residual, B):
    from paper_2410_23608_b200 import binding as L
    from paper_2410_23608_b200.block import SpaBlock
    cfg, inp, s_up, labels, fwd = _problem(ci, residual, B)
    alpha = 0.25
    bwd = O.block_bwd_trainable(fwd, inp.dY, inp.x, inp.w_g, inp.W_qkv, inp.W_o, cfg.H, labels=labels, alpha=alpha,
                                s_up=s_up, residual=residual, gate_scale=True)
    dt = cfg.dtype
    d = {n: dev(getattr(inp, n), dt) for n in ("x", "w_g", "W_qkv", "b_qkv", "W_o", "b_o", "dY")}
    flags = L.SPA_FLAG_GATE_SCALE | (L.SPA_FLAG_RESIDUAL if residual else 0)
    blk = SpaBlock(cfg.B, cfg.N, cfg.C, cfg.H, dt, tau=cfg.tau, flags=flags)
    s_up_d = torch.from_numpy(s_up.astype(np.float32)).cuda()
    lab_d = torch.from_numpy(labels.astype(np.uint8)).cuda()
    y = blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"], s_up=s_up_d)
    dX = blk.backward_trainable(d["dY"], d["x"], d["w_g"], labels=lab_d, alpha=alpha, s_up=s_up_d)
    torch.cuda.synchronize()
    assert blk.read_status() == 0
    Np = int(fwd["cu_seqlens"][-1])
    assert np.array_equal(blk.mask.cpu().numpy().astype(bool), fwd["mask"].reshape(-1))
    assert_close(host(y), fwd["y"], dt, "y")
    # loss: a sum of B*N terms of order one, fp32 accumulation
    loss_ref = bwd["loss"]
    assert abs(float(blk.loss.item()) - loss_ref) <= 1e-4 * max(1.0, abs(loss_ref))
    ds_tol = 1e-4 if dt == "f32" else 3e-2
    ds_ref = bwd["ds"]
    assert np.abs(blk.ds.cpu().numpy() - ds_ref).max() <= ds_tol * max(1.0, np.abs(ds_ref).max())
    lin = (fwd["scores"] > s_up).reshape(-1)
    got_up = blk.ds_up.cpu().numpy()
    assert np.all(got_up[lin] == 0.0)
    assert np.abs(got_up - bwd["ds_up"]).max() <= ds_tol * max(1.0, np.abs(ds_ref).max())
    assert_close(host(dX), bwd["dX"], dt, "dX", scale_max_abs=True)
    assert_close(blk.dw_g.cpu().numpy().astype(np.float64), bwd["dw_g"], dt, "dw_g", scale_max_abs=True)
    db_ref = bwd["db_g"]
    assert abs(float(blk.db_g.item()) - db_ref) <= TOL[dt]["max_abs"] * max(1.0, abs(db_ref), np.abs(ds_ref).sum() * 1e-2)
    for name in ("dW_qkv", "db_qkv", "dW_o", "db_o"):
        assert_close(host(getattr(blk, name)), bwd[name], dt, name, scale_max_abs=True)


def test_select_loss_without_labels_clears_ds():
    from paper_2410_23608_b200 import binding as L
    from paper_2410_23608_b200.block import SpaBlock
    cfg = get_config(1)
    blk = SpaBlock(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype)
    n = cfg.B * cfg.N
    ds = torch.full((n,), 7.0, dtype=torch.float32, device="cuda")
    loss = torch.full((1,), 7.0, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(L.spa_train_workspace_bytes(blk.p), 256), dtype=torch.uint8, device="cuda")
    scores = torch.randn(n, dtype=torch.float32, device="cuda")
    L.spa_select_loss(blk.p, scores, None, 1.0, ds, loss, ws)
    assert float(ds.abs().max()) == 0.0 and float(loss.item()) == 0.0


@pytest.mark.parametrize("tau", [float("inf"), float("-inf")])
def test_trainable_block_none_and_all_selected(tau):
    """Nothing selected: only the selection loss reaches the gate.  Everything selected: every token carries the
    sigmoid-scaling path."""
    from paper_2410_23608_b200 import binding as L
    from paper_2410_23608_b200.block import SpaBlock
    from spa_workloads import scaled_config
    cfg = scaled_config(get_config(2), B=3)
    inp = make_inputs(cfg)
    rng = np.random.default_rng(5)
    labels = rng.uniform(size=(cfg.B, cfg.N)) < 0.5
    fwd = O.block_fwd(inp.x, inp.w_g, inp.b_g, tau, inp.W_qkv, inp.b_qkv, inp.W_o, inp.b_o, cfg.H, gate_scale=True)
    bwd = O.block_bwd_trainable(fwd, inp.dY, inp.x, inp.w_g, inp.W_qkv, inp.W_o, cfg.H, labels=labels, alpha=1.0,
                                gate_scale=True)
    dt = cfg.dtype
    d = {n: dev(getattr(inp, n), dt) for n in ("x", "w_g", "W_qkv", "b_qkv", "W_o", "b_o", "dY")}
    blk = SpaBlock(cfg.B, cfg.N, cfg.C, cfg.H, dt, tau=tau, flags=L.SPA_FLAG_GATE_SCALE)
    y = blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"])
    dX = blk.backward_trainable(d["dY"], d["x"], d["w_g"], labels=torch.from_numpy(labels.astype(np.uint8)).cuda())
    torch.cuda.synchronize()
    assert blk.read_status() == 0
    assert int(blk.cu[-1].item()) == (0 if tau > 0 else cfg.B * cfg.N)
    assert_close(host(y), fwd["y"], dt, "y")
    assert_close(host(dX), bwd["dX"], dt, "dX", scale_max_abs=True)
    assert_close(blk.dw_g.cpu().numpy().astype(np.float64), bwd["dw_g"], dt, "dw_g", scale_max_abs=True)
    assert abs(float(blk.loss.item()) - bwd["loss"]) <= 1e-4 * max(1.0, abs(bwd["loss"]))
    assert not blk.ds_up.any()   # no up-scale scores were given: nothing goes to them
