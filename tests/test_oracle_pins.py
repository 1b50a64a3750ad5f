"""Pins for the fp64 oracle: closed forms, brute force, invariants, limits that reduce to a
library routine, finite differences.  Each test is chosen so that a plausible mistake in the
oracle (dropped term, wrong sign or index, transposed operand) makes it fail.  CPU only."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from oracle.brute_force import block_fwd_bruteforce
from spa_workloads import get_config, make_inputs, scaled_config

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_problem(seed=0, B=3, N=12, C=8, H=2, keep=0.5):
    rng = np.random.default_rng(seed)
    x = rng.normal(size=(B, N, C))
    w_g = rng.normal(size=C) / np.sqrt(C)
    b_g = float(np.quantile(x @ w_g, 1 - keep) * -1.0)
    W_qkv = rng.normal(size=(3 * C, C)) / np.sqrt(C)
    b_qkv = rng.normal(size=3 * C) * 0.1
    W_o = rng.normal(size=(C, C)) / np.sqrt(C)
    b_o = rng.normal(size=C) * 0.1
    return dict(x=x, w_g=w_g, b_g=b_g, tau=0.0, W_qkv=W_qkv, b_qkv=b_qkv, W_o=W_o, b_o=b_o, H=H)


# ------------------------------------------------------------------ gate + select
def test_gate_closed_form_along_w():
    rng = np.random.default_rng(1)
    C = 16
    w = rng.normal(size=C)
    u = w / np.linalg.norm(w)
    k = np.array([[-2.0, 0.0, 0.5, 3.0]])
    x = k[:, :, None] * u[None, None, :]
    s = O.gate(x, w, 0.25)
    np.testing.assert_allclose(s, k * np.linalg.norm(w) + 0.25, rtol=0, atol=1e-13)


def test_gate_exact_rational_on_integers():
    rng = np.random.default_rng(2)
    x = rng.integers(-5, 6, size=(4, 4, 8))
    w = rng.integers(-3, 4, size=8)
    s = O.gate(x.astype(float), w.astype(float), 2.0)
    for b in range(4):
        for n in range(4):
            exact = Fraction(2) + sum(Fraction(int(w[c])) * int(x[b, n, c]) for c in range(8))
            assert Fraction(float(s[b, n])) == exact


def test_gate_max_with_upscale_scores():
    x = np.zeros((1, 3, 2))
    s = O.gate(x, np.ones(2), 0.5, s_up=np.array([[-1.0, 0.5, 2.0]]))
    np.testing.assert_array_equal(s, [[0.5, 0.5, 2.0]])


def test_select_is_strict_threshold():
    m = O.select(np.array([[-1.0, 0.0, 1e-9, 2.0]]), 0.0)
    np.testing.assert_array_equal(m, [[False, False, True, True]])


def test_mask_matches_generator_blobs_where_noise_is_small():
    cfg = get_config(1)
    inp = make_inputs(cfg)
    s = O.gate(inp.x, inp.w_g, inp.b_g)
    m = O.select(s, inp.tau)
    u = inp.w_g / np.linalg.norm(inp.w_g)
    along = inp.x @ u - cfg.offset * inp.blob_mask       # noise coordinate along the gate direction
    calm = np.abs(along) < 0.45 * cfg.offset
    assert calm.mean() > 0.7
    np.testing.assert_array_equal(m[calm], inp.blob_mask[calm])


def test_margin_of_generated_inputs():
    for i in (1, 2):
        inp = make_inputs(get_config(i))
        s = O.gate(inp.x, inp.w_g, inp.b_g)
        assert np.abs(s - inp.tau).min() >= 1e-3


# ------------------------------------------------------------------ packing indices
def test_pack_indices_invariants_and_pushback():
    rng = np.random.default_rng(3)
    B, N = 5, 17
    mask = rng.random((B, N)) < 0.4
    mask[2] = False                       # an image with nothing selected
    cu, idx, inv = O.pack_indices(mask)
    assert cu.dtype == np.int32 and idx.dtype == np.int32 and inv.dtype == np.int32
    assert cu[0] == 0 and cu[-1] == mask.sum() == idx.size
    assert np.all(np.diff(idx) > 0)
    ref = []                              # brute force: push back in scan order
    for b in range(B):
        for n in range(N):
            if mask[b, n]:
                ref.append(b * N + n)
    np.testing.assert_array_equal(idx, ref)
    for i, t in enumerate(idx):
        b = t // N
        assert cu[b] <= i < cu[b + 1]
        assert inv[t] == i
    assert np.all(inv[~mask.reshape(-1)] == -1)
    assert cu[3] == cu[2]


def test_pack_unpack_identity_bitwise():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(3, 10, 4))
    mask = rng.random((3, 10)) < 0.5
    _, idx, _ = O.pack_indices(mask)
    xp = O.pack_rows(x, idx)
    assert np.array_equal(xp, x.reshape(-1, 4)[mask.reshape(-1)])
    y = O.unpack_scatter(xp, x, idx)
    assert np.array_equal(y, x)
    z = rng.normal(size=xp.shape)
    y = O.unpack_scatter(z, x, idx)
    assert np.array_equal(y.reshape(-1, 4)[~mask.reshape(-1)], x.reshape(-1, 4)[~mask.reshape(-1)])
    assert np.array_equal(y.reshape(-1, 4)[mask.reshape(-1)], z)
    yr = O.unpack_scatter(z, x, idx, residual=True)
    assert np.array_equal(yr.reshape(-1, 4)[mask.reshape(-1)], xp + z)


def test_gate_scale_is_sigmoid_times_row():
    x = np.ones((1, 2, 3))
    xp = O.pack_rows(x, np.array([0, 1]), s=np.array([[0.0, np.log(3.0)]]), gate_scale=True)
    np.testing.assert_allclose(xp, [[0.5] * 3, [0.75] * 3], atol=1e-15)


# ------------------------------------------------------------------ attention
def test_block_matches_bruteforce():
    for seed, keep in ((0, 0.5), (1, 0.25), (2, 0.9)):
        p = tiny_problem(seed=seed, keep=keep)
        fwd = O.block_fwd(**p)
        y_bf = block_fwd_bruteforce(**p)
        assert 0 < fwd["idx"].size < p["x"].shape[0] * p["x"].shape[1]
        np.testing.assert_allclose(fwd["y"], y_bf, rtol=0, atol=1e-12)
    p = tiny_problem(seed=5)
    np.testing.assert_allclose(O.block_fwd(**p, residual=True)["y"],
                               block_fwd_bruteforce(**p, residual=True), rtol=0, atol=1e-12)


def test_per_image_equals_masked_dense_and_rows_sum_to_one():
    p = tiny_problem(seed=7, B=4, N=9)
    fwd = O.block_fwd(**p)
    ao2 = O.attention_fwd_masked_dense(fwd["qkv"], fwd["cu_seqlens"], p["H"])
    np.testing.assert_allclose(fwd["ao"], ao2, rtol=0, atol=1e-12)
    _, _, probs = O.attention_fwd(fwd["qkv"], fwd["cu_seqlens"], p["H"], return_probs=True)
    assert probs
    for _, _, P in probs:
        np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-14)
        assert np.all(P >= 0)


def _dense_mha_torch(x, W_qkv, b_qkv, W_o, b_o, H):
    xt = torch.tensor(x, dtype=torch.float64)
    B, N, C = xt.shape
    qkv = torch.nn.functional.linear(xt, torch.tensor(W_qkv), torch.tensor(b_qkv))
    q, k, v = qkv.split(C, dim=-1)
    sh = lambda t: t.reshape(B, N, H, C // H).transpose(1, 2)
    o = torch.nn.functional.scaled_dot_product_attention(sh(q), sh(k), sh(v))
    o = o.transpose(1, 2).reshape(B, N, C)
    return torch.nn.functional.linear(o, torch.tensor(W_o), torch.tensor(b_o))


def test_all_selected_limit_is_dense_mha():
    p = tiny_problem(seed=8, B=2, N=11, C=12, H=3)
    p["tau"] = -np.inf
    fwd = O.block_fwd(**p)
    assert fwd["mask"].all()
    ref = _dense_mha_torch(p["x"], p["W_qkv"], p["b_qkv"], p["W_o"], p["b_o"], p["H"]).numpy()
    np.testing.assert_allclose(fwd["y"], ref, rtol=0, atol=1e-12)


def test_lse_against_library_logsumexp():
    from scipy.special import logsumexp
    p = tiny_problem(seed=9)
    fwd = O.block_fwd(**p)
    C, H = p["x"].shape[2], p["H"]
    d = C // H
    cu = fwd["cu_seqlens"]
    for b in range(len(cu) - 1):
        lo, hi = cu[b], cu[b + 1]
        for h in range(H):
            q = fwd["qkv"][lo:hi, h * d:(h + 1) * d]
            k = fwd["qkv"][lo:hi, C + h * d:C + (h + 1) * d]
            np.testing.assert_allclose(fwd["lse"][h, lo:hi], logsumexp(q @ k.T / np.sqrt(d), axis=1),
                                       atol=1e-13)


def test_zero_query_weights_give_segment_mean_of_v():
    p = tiny_problem(seed=10)
    C = p["x"].shape[2]
    p["W_qkv"][:C] = 0.0
    p["b_qkv"][:C] = 0.0
    fwd = O.block_fwd(**p)
    cu = fwd["cu_seqlens"]
    v = fwd["qkv"][:, 2 * C:]
    for b in range(len(cu) - 1):
        lo, hi = cu[b], cu[b + 1]
        if hi > lo:
            np.testing.assert_allclose(fwd["ao"][lo:hi], np.tile(v[lo:hi].mean(0), (hi - lo, 1)), atol=1e-13)


def test_equal_values_pass_through_attention():
    rng = np.random.default_rng(11)
    C, H = 8, 2
    qkv = rng.normal(size=(7, 3 * C))
    qkv[:, 2 * C:] = rng.normal(size=C)[None, :]
    ao, _ = O.attention_fwd(qkv, np.array([0, 3, 7]), H)
    np.testing.assert_allclose(ao, qkv[:, 2 * C:], atol=1e-14)


def test_single_token_segment():
    rng = np.random.default_rng(12)
    C, H = 8, 2
    d = C // H
    qkv = rng.normal(size=(3, 3 * C))
    ao, lse = O.attention_fwd(qkv, np.array([0, 1, 2, 3]), H)
    np.testing.assert_allclose(ao, qkv[:, 2 * C:], atol=1e-15)
    for h in range(H):
        s11 = (qkv[:, h * d:(h + 1) * d] * qkv[:, C + h * d:C + (h + 1) * d]).sum(1) / np.sqrt(d)
        np.testing.assert_allclose(lse[h], s11, atol=1e-14)


def test_permutation_equivariance_and_image_independence():
    p = tiny_problem(seed=13, B=3, N=10)
    y0 = O.block_fwd(**p)["y"]
    perm = np.random.default_rng(0).permutation(10)
    p2 = dict(p)
    p2["x"] = p["x"].copy()
    p2["x"][1] = p["x"][1][perm]
    y1 = O.block_fwd(**p2)["y"]
    np.testing.assert_allclose(y1[1], y0[1][perm], atol=1e-12)
    assert np.array_equal(y1[0], y0[0]) and np.array_equal(y1[2], y0[2])
    p3 = dict(p)
    p3["x"] = p["x"].copy()
    p3["x"][2] = np.random.default_rng(1).normal(size=p["x"][2].shape)
    y2 = O.block_fwd(**p3)["y"]
    assert np.array_equal(y2[0], y0[0]) and np.array_equal(y2[1], y0[1])


def test_none_selected_limit():
    p = tiny_problem(seed=14)
    p["tau"] = np.inf
    fwd = O.block_fwd(**p)
    assert fwd["idx"].size == 0 and fwd["cu_seqlens"][-1] == 0
    assert np.array_equal(fwd["y"], p["x"])
    dY = np.random.default_rng(2).normal(size=p["x"].shape)
    bwd = O.block_bwd(fwd, dY, p["x"], p["W_qkv"], p["W_o"], p["H"])
    assert np.array_equal(bwd["dX"], dY)
    assert not bwd["dW_qkv"].any() and not bwd["dW_o"].any()


def test_container_cuts():
    p = tiny_problem(seed=15, B=2, N=12, keep=0.8)
    fwd = O.block_fwd(**p)
    big = O.block_fwd(**p, container_len=10_000)
    np.testing.assert_allclose(big["y"], fwd["y"], atol=0)
    one = O.block_fwd(**p, container_len=1)
    np.testing.assert_allclose(one["ao"], one["qkv"][:, 2 * p["x"].shape[2]:], atol=1e-15)
    cuts = O.container_cuts(np.array([0, 5, 5, 12], np.int32), 4)
    np.testing.assert_array_equal(cuts, [0, 4, 5, 8, 12])


# ------------------------------------------------------------------ backward
def _loss(p, G, residual=False):
    return float((O.block_fwd(**p, residual=residual)["y"] * G).sum())


@pytest.mark.parametrize("residual", [False, True])
def test_backward_against_central_differences(residual):
    p = tiny_problem(seed=20, B=2, N=7, C=6, H=2, keep=0.6)
    rng = np.random.default_rng(21)
    G = rng.normal(size=p["x"].shape)
    fwd = O.block_fwd(**p, residual=residual)
    assert 2 < fwd["idx"].size < 14
    bwd = O.block_bwd(fwd, G, p["x"], p["W_qkv"], p["W_o"], p["H"], residual=residual)
    h = 1e-6
    for name, grad in (("x", bwd["dX"]), ("W_qkv", bwd["dW_qkv"]), ("b_qkv", bwd["db_qkv"]),
                       ("W_o", bwd["dW_o"]), ("b_o", bwd["db_o"])):
        base = p[name]
        num = np.zeros_like(base)
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            pp = dict(p); a = base.copy(); a[i] += h; pp[name] = a
            pm = dict(p); c = base.copy(); c[i] -= h; pm[name] = c
            num[i] = (_loss(pp, G, residual) - _loss(pm, G, residual)) / (2 * h)
        denom = max(np.abs(num).max(), 1e-12)
        assert np.abs(num - grad).max() / denom <= 1e-6, name


def test_backward_unselected_rows_and_key_shift_invariance():
    p = tiny_problem(seed=22, B=3, N=9)
    fwd = O.block_fwd(**p)
    dY = np.random.default_rng(23).normal(size=p["x"].shape)
    bwd = O.block_bwd(fwd, dY, p["x"], p["W_qkv"], p["W_o"], p["H"])
    unsel = ~fwd["mask"].reshape(-1)
    C = p["x"].shape[2]
    assert np.array_equal(bwd["dX"].reshape(-1, C)[unsel], dY.reshape(-1, C)[unsel])
    # softmax ignores a shift common to all keys of a segment, so dK sums to zero there
    cu = fwd["cu_seqlens"]
    dk = bwd["dqkv"][:, C:2 * C]
    for b in range(len(cu) - 1):
        if cu[b + 1] > cu[b]:
            np.testing.assert_allclose(dk[cu[b]:cu[b + 1]].sum(0), 0.0, atol=1e-12)


def test_all_selected_backward_is_dense_mha_backward():
    p = tiny_problem(seed=24, B=2, N=6, C=8, H=2)
    p["tau"] = -np.inf
    fwd = O.block_fwd(**p)
    G = np.random.default_rng(25).normal(size=p["x"].shape)
    bwd = O.block_bwd(fwd, G, p["x"], p["W_qkv"], p["W_o"], p["H"])
    t = {k: torch.tensor(p[k], dtype=torch.float64, requires_grad=True)
         for k in ("x", "W_qkv", "b_qkv", "W_o", "b_o")}
    B, N, C = p["x"].shape
    H = p["H"]
    qkv = t["x"] @ t["W_qkv"].T + t["b_qkv"]
    q, k, v = qkv.split(C, dim=-1)
    sh = lambda a: a.reshape(B, N, H, C // H).transpose(1, 2)
    att = torch.softmax(sh(q) @ sh(k).transpose(-1, -2) / (C // H) ** 0.5, dim=-1) @ sh(v)
    y = att.transpose(1, 2).reshape(B, N, C) @ t["W_o"].T + t["b_o"]
    (y * torch.tensor(G)).sum().backward()
    for name, key in (("x", "dX"), ("W_qkv", "dW_qkv"), ("b_qkv", "db_qkv"), ("W_o", "dW_o"), ("b_o", "db_o")):
        np.testing.assert_allclose(bwd[key], t[name].grad.numpy(), rtol=0, atol=1e-11)


# ------------------------------------------------------------------ complexity model
def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "eq7_eq9_macs.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                eq, *nums = line.split()
                rows.append((eq, *map(int, nums)))
    return rows


def test_mac_count_against_eq7_and_eq9():
    for eq, B, N, C, Bp, L, macs in _golden_rows():
        if eq == "eq7":    # everything selected, one segment per image: plain MSA
            m = O.mac_count(B, N, C, np.arange(B + 1) * N)
            assert m["qkv"] + m["attn"] + m["proj"] == macs
        else:              # containers of length L: the packed terms of Eq. 9 plus the gate term
            m = O.mac_count(B, N, C, np.arange(Bp + 1) * L)
            assert m["qkv"] + m["attn"] == Bp * (3 * L * C * C + 2 * L * L * C)
            assert m["gate"] + B * N * C * C + m["qkv"] + m["attn"] == macs


def test_full_config_shapes_run():
    cfg = scaled_config(get_config(2), B=4)
    inp = make_inputs(cfg)
    fwd = O.block_fwd(inp.x, inp.w_g, inp.b_g, inp.tau, inp.W_qkv, inp.b_qkv, inp.W_o, inp.b_o, cfg.H)
    frac = fwd["mask"].mean(axis=1)
    assert np.all(np.abs(frac - inp.keep_target) < 0.08)


# ------------------------------------------------------------------ trainable selection (Eq. 4-6 with scaling, Eq. 10)
def test_score_pool_against_loops():
    rng = np.random.default_rng(40)
    B, rows, cols = 2, 3, 4
    prev = rng.normal(size=(B, 2 * rows, 2 * cols))
    got = O.score_pool(prev, B, rows, cols)
    for b in range(B):
        for i in range(rows):
            for j in range(cols):
                want = max(prev[b, 2 * i + di, 2 * j + dj] for di in (0, 1) for dj in (0, 1))
                assert got[b, i * cols + j] == want


def test_select_loss_closed_forms():
    # all logits zero: every token contributes ln 2, whatever its label; gradient is 1/2 - y
    y = np.array([0.0, 1.0, 1.0, 0.0, 1.0])
    loss, g = O.select_loss(np.zeros(5), y)
    assert abs(loss - 5 * np.log(2.0)) < 1e-14
    np.testing.assert_allclose(g, 0.5 - y, atol=1e-15)
    # one token, logit = ln 3 => p = 3/4: loss -ln(3/4) for y = 1, -ln(1/4) for y = 0
    l1, g1 = O.select_loss(np.array([np.log(3.0)]), np.array([1.0]))
    l0, g0 = O.select_loss(np.array([np.log(3.0)]), np.array([0.0]))
    assert abs(l1 + np.log(0.75)) < 1e-14 and abs(l0 + np.log(0.25)) < 1e-14
    assert abs(g1[0] + 0.25) < 1e-14 and abs(g0[0] - 0.75) < 1e-14
    # against the library's binary cross entropy on logits, and no overflow far from zero
    rng = np.random.default_rng(41)
    s = rng.normal(size=50) * 30
    yy = (rng.uniform(size=50) > 0.5).astype(np.float64)
    ref = torch.nn.functional.binary_cross_entropy_with_logits(torch.from_numpy(s), torch.from_numpy(yy), reduction="sum")
    loss, _ = O.select_loss(s, yy)
    assert np.isfinite(loss) and abs(loss - float(ref)) <= 1e-10 * max(1.0, abs(float(ref)))


def _trainable_total(p, G, labels, alpha, s_up, residual):
    fwd = O.block_fwd(**p, s_up=s_up, residual=residual, gate_scale=True)
    loss, _ = O.select_loss(fwd["scores"].reshape(-1), labels.reshape(-1))
    return float((fwd["y"] * G).sum()) + alpha * loss, fwd


@pytest.mark.parametrize("residual", [False, True])
def test_trainable_backward_against_central_differences(residual):
    """Total = <y, G> + alpha * selection loss with the sigmoid scaling on and an up-scale score map:
    gradients to x, w_g, b_g and s_up (and the layer weights) against central differences.  The
    perturbations are far smaller than the distance of every logit from the threshold and from
    s_up, so neither the selection nor the winner of Max changes."""
    p = tiny_problem(seed=42, B=2, N=8, C=6, H=2, keep=0.6)
    p["b_g"] += 0.037   # tiny_problem puts one logit exactly on the threshold
    rng = np.random.default_rng(43)
    G = rng.normal(size=p["x"].shape)
    labels = (rng.uniform(size=(2, 8)) > 0.5).astype(np.float64)
    s_lin = O.gate(p["x"], p["w_g"], p["b_g"])
    s_up = s_lin + rng.choice([-0.7, 0.9], size=s_lin.shape)   # wins on some tokens, loses on others
    alpha = 0.3
    _, fwd = _trainable_total(p, G, labels, alpha, s_up, residual)
    assert 2 < fwd["idx"].size < 16
    assert np.abs(fwd["scores"] - p["tau"]).min() > 1e-3
    bwd = O.block_bwd_trainable(fwd, G, p["x"], p["w_g"], p["W_qkv"], p["W_o"], p["H"], labels=labels, alpha=alpha,
                                s_up=s_up, residual=residual, gate_scale=True)
    h = 1e-6
    grads = {"x": bwd["dX"], "w_g": bwd["dw_g"], "W_qkv": bwd["dW_qkv"], "W_o": bwd["dW_o"], "b_o": bwd["db_o"]}
    for name, grad in grads.items():
        base = p[name]
        num = np.zeros_like(base)
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            pp = dict(p); a = base.copy(); a[i] += h; pp[name] = a
            pm = dict(p); c = base.copy(); c[i] -= h; pm[name] = c
            num[i] = (_trainable_total(pp, G, labels, alpha, s_up, residual)[0] -
                      _trainable_total(pm, G, labels, alpha, s_up, residual)[0]) / (2 * h)
        assert np.abs(num - grad).max() / max(np.abs(num).max(), 1e-12) <= 1e-6, name
    # scalar bias of the gate
    pp = dict(p); pp["b_g"] = p["b_g"] + h
    pm = dict(p); pm["b_g"] = p["b_g"] - h
    num_b = (_trainable_total(pp, G, labels, alpha, s_up, residual)[0] -
             _trainable_total(pm, G, labels, alpha, s_up, residual)[0]) / (2 * h)
    assert abs(num_b - bwd["db_g"]) <= 1e-6 * max(abs(num_b), 1e-12)
    # the up-scale scores
    num_up = np.zeros_like(s_up)
    for i in np.ndindex(*s_up.shape):
        a = s_up.copy(); a[i] += h
        c = s_up.copy(); c[i] -= h
        num_up[i] = (_trainable_total(p, G, labels, alpha, a, residual)[0] -
                     _trainable_total(p, G, labels, alpha, c, residual)[0]) / (2 * h)
    assert np.abs(num_up.reshape(-1) - bwd["ds_up"]).max() <= 1e-6 * max(np.abs(num_up).max(), 1e-12)
    # where s_up wins the linear layer gets nothing, and the other way round
    lin = (fwd["scores"] > s_up).reshape(-1)
    assert np.all(bwd["ds_up"][lin] == 0.0) and np.all(bwd["ds_up"][~lin] == bwd["ds"][~lin])


def test_trainable_backward_reduces_to_plain_backward():
    """Scaling off, no labels, no s_up: nothing reaches the gate and dX equals block_bwd's."""
    p = tiny_problem(seed=44, B=2, N=9)
    rng = np.random.default_rng(45)
    G = rng.normal(size=p["x"].shape)
    fwd = O.block_fwd(**p)
    a = O.block_bwd(fwd, G, p["x"], p["W_qkv"], p["W_o"], p["H"])
    b = O.block_bwd_trainable(fwd, G, p["x"], p["w_g"], p["W_qkv"], p["W_o"], p["H"], gate_scale=False)
    assert np.array_equal(a["dX"], b["dX"]) and np.all(b["ds"] == 0) and np.all(b["dw_g"] == 0) and b["db_g"] == 0


# ------------------------------------------------------------------ shifted feature map before packing
def test_shift_order_is_a_cyclic_roll():
    rows, cols = 3, 5
    grid = np.arange(rows * cols).reshape(rows, cols)
    o = O.shift_order(rows, cols, 1, 2)
    np.testing.assert_array_equal(o.reshape(rows, cols), np.roll(grid, shift=(-1, -2), axis=(0, 1)))
    np.testing.assert_array_equal(O.shift_order(rows, cols, 0, 0), np.arange(rows * cols))
    assert sorted(o.tolist()) == list(range(rows * cols))


def test_ordered_packing_invariants_and_effect():
    """Packing in a shifted order permutes each image's packed rows and nothing else: without containers the
    block output is unchanged (attention inside an image does not depend on the order of its tokens); with
    containers of length L the output changes, because other token pairs share a container."""
    p = tiny_problem(seed=50, B=3, N=12, C=8, H=2, keep=0.7)
    order = O.shift_order(3, 4, 1, 1)
    a = O.block_fwd(**p)
    b = O.block_fwd(**p, order=order)
    # indices: same counts, idx a permutation inside each image, visited in the given order
    np.testing.assert_array_equal(a["cu_seqlens"], b["cu_seqlens"])
    mask = a["mask"]
    for img in range(3):
        lo, hi = a["cu_seqlens"][img], a["cu_seqlens"][img + 1]
        assert sorted(b["idx"][lo:hi].tolist()) == a["idx"][lo:hi].tolist()
        want = [img * 12 + t for t in order if mask[img, t]]        # push-back in visiting order
        assert b["idx"][lo:hi].tolist() == want
    assert np.array_equal(b["inv"][b["idx"]], np.arange(b["idx"].size))
    np.testing.assert_allclose(b["y"], a["y"], rtol=0, atol=1e-12)
    c = O.block_fwd(**p, container_len=4)
    d = O.block_fwd(**p, container_len=4, order=order)
    assert np.abs(c["y"] - d["y"]).max() > 1e-3
    # and the ordered, containerised block equals the plain one applied to the explicitly permuted input
    inv_o = np.argsort(order)
    pp = dict(p); pp["x"] = p["x"][:, order, :]
    e = O.block_fwd(**pp, container_len=4)
    np.testing.assert_allclose(d["y"], e["y"][:, inv_o, :], rtol=0, atol=1e-12)


# ------------------------------------------------------------------ LayerNorm, GELU, feed-forward, whole block
def test_layer_norm_and_gelu_against_library():
    rng = np.random.default_rng(60)
    x = rng.normal(size=(3, 5, 16)) * 2 + 0.5
    g, b = rng.normal(size=16), rng.normal(size=16)
    y, mean, rstd = O.layer_norm(x, g, b)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (16,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-12)
    xt = torch.from_numpy(x).requires_grad_(True)
    gt = torch.from_numpy(g).requires_grad_(True)
    bt = torch.from_numpy(b).requires_grad_(True)
    dy = rng.normal(size=x.shape)
    torch.nn.functional.layer_norm(xt, (16,), gt, bt, 1e-5).backward(torch.from_numpy(dy))
    dx, dg, db = O.layer_norm_bwd(dy, x, g, mean, rstd)
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dg, gt.grad.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(db, bt.grad.numpy(), rtol=0, atol=1e-12)
    u = rng.normal(size=200) * 3
    np.testing.assert_allclose(O.gelu(u), torch.nn.functional.gelu(torch.from_numpy(u)).numpy(), rtol=0, atol=1e-14)
    h = 1e-6
    np.testing.assert_allclose(O.gelu_grad(u), (O.gelu(u + h) - O.gelu(u - h)) / (2 * h), rtol=0, atol=1e-8)
    assert O.gelu(np.array([0.0]))[0] == 0.0 and abs(O.gelu_grad(np.array([0.0]))[0] - 0.5) < 1e-15


def _layer_params(rng, C, Hd):
    s = 1.0 / np.sqrt(C)
    return dict(g1=1 + 0.1 * rng.normal(size=C), be1=0.1 * rng.normal(size=C), w_g=rng.normal(size=C) * s, b_g=0.03,
                W_qkv=rng.normal(size=(3 * C, C)) * s, b_qkv=0.1 * rng.normal(size=3 * C), W_o=rng.normal(size=(C, C)) * s,
                b_o=0.1 * rng.normal(size=C), g2=1 + 0.1 * rng.normal(size=C), be2=0.1 * rng.normal(size=C),
                W1=rng.normal(size=(Hd, C)) * s, b1=0.1 * rng.normal(size=Hd), W2=rng.normal(size=(C, Hd)) / np.sqrt(Hd),
                b2=0.1 * rng.normal(size=C))


def test_layer_backward_against_central_differences():
    rng = np.random.default_rng(61)
    B, N, C, H = 2, 6, 8, 2
    prm = _layer_params(rng, C, 4 * C)
    x = rng.normal(size=(B, N, C))
    G = rng.normal(size=x.shape)
    f = O.layer_fwd(x, prm, H)
    assert 2 < f["spa"]["idx"].size < B * N and np.abs(f["spa"]["scores"]).min() > 1e-3
    bwd = O.layer_bwd(f, G, x, prm, H)
    # unselected tokens receive no attention update
    unsel = ~f["spa"]["mask"]
    assert np.array_equal(f["y1"][unsel], x[unsel])
    total = lambda xx, pp: float((O.layer_fwd(xx, pp, H)["out"] * G).sum())
    h = 1e-6
    num = np.zeros_like(x)
    for i in np.ndindex(*x.shape):
        a = x.copy(); a[i] += h
        c = x.copy(); c[i] -= h
        num[i] = (total(a, prm) - total(c, prm)) / (2 * h)
    assert np.abs(num - bwd["dX"]).max() / np.abs(num).max() <= 1e-6
    for name, gname in (("g1", "dg1"), ("be1", "dbe1"), ("g2", "dg2"), ("be2", "dbe2"), ("W1", "dW1"), ("b1", "db1"),
                        ("W2", "dW2"), ("b2", "db2"), ("W_qkv", "dW_qkv"), ("b_o", "db_o")):
        base = prm[name]
        numg = np.zeros_like(base)
        for i in np.ndindex(*base.shape):
            pa = dict(prm); a = base.copy(); a[i] += h; pa[name] = a
            pc = dict(prm); c = base.copy(); c[i] -= h; pc[name] = c
            numg[i] = (total(x, pa) - total(x, pc)) / (2 * h)
        assert np.abs(numg - bwd[gname]).max() / max(np.abs(numg).max(), 1e-12) <= 1e-6, name
