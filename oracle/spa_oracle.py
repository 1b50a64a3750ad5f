"""fp64 CPU oracle of one Select-and-Pack-Attention (SPA) block.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the block computes, written from the
paper (Sec. 3.2 "Select and Pack Attention", Eq. 4-6, the "Token Packing" paragraph,
the same-image attention mask, and the complexity model Eq. 7-9).  It exists to check
the CUDA library; it shares no code with it and must never be imported by the
product path.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may call it.

Everything is numpy in float64.  A matmul (`@`) is used as a step where the paper's
step is a dense linear map; nothing is blocked, fused or reordered.

Readings of the paper that this oracle fixes (each is stated where it is used):
  * selection is the deterministic inference form of Eq. 6: keep a token iff its
    logit exceeds a threshold tau, strictly;
  * the sigmoid scaling of Eq. 5 is optional (off by default) so that packing is a
    pure gather and "all tokens selected" reduces to ordinary multi-head attention;
  * tokens are packed image after image, each image in raster order, into one
    buffer described by cumulative lengths `cu_seqlens` (no fixed-length containers
    by default; a `container_len` argument gives the paper's container cut);
  * attention is softmax(q k^T / sqrt(d)) v per head with biases on the QKV and
    output projections and no positional bias;
  * unselected tokens are passed through unchanged.

Pinned by tests/test_oracle_pins.py: brute force per image, closed forms, the
all-selected limit against a library attention routine, invariants, and central
finite differences for every gradient.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- forward
def gate(x, w_g, b_g, s_up=None):
    """Gate logits, Eq. 4: s = Max(f_g(r), s_up) with f_g a linear layer C -> 1.

    x [B,N,C], w_g [C], b_g scalar, s_up [B,N] or None  ->  s [B,N].
    """
    x = np.asarray(x, F64)
    s = x @ np.asarray(w_g, F64) + F64(b_g)
    if s_up is not None:
        s = np.maximum(s, np.asarray(s_up, F64))
    return s


def select(s, tau):
    """Hard selection (deterministic form of Eq. 6): token kept iff s > tau (strict)."""
    return (np.asarray(s, F64) > F64(tau))


def shift_order(rows, cols, shift_r, shift_c):
    """Order in which the tokens of an image are visited when its feature map is shifted cyclically
    by (shift_r, shift_c) before packing (Sec. 1: the feature maps are shifted every two blocks so that
    the token pairs that share a container vary).  order[j] is the original raster index of the token
    that sits at raster position j of the shifted map."""
    i = (np.arange(rows)[:, None] + shift_r) % rows
    j = (np.arange(cols)[None, :] + shift_c) % cols
    return (i * cols + j).reshape(-1).astype(np.int32)


def pack_indices(mask, order=None):
    """Token packing, index part ("Token Packing" paragraph).

    mask [B,N] bool -> cu_seqlens int32 [B+1], idx int32 [N_p], inv int32 [B*N].
    Selected tokens keep batch order then raster order (or, with `order` [N], the order in which
    order[0], order[1], ... visits each image's tokens); idx[i] is the flat position
    b*N+n of packed row i; inv is its inverse with -1 at unselected positions.
    """
    mask = np.asarray(mask, bool)
    B, N = mask.shape
    cu = np.zeros(B + 1, dtype=np.int64)
    idx = []
    for b in range(B):
        if order is None:
            pos = np.nonzero(mask[b])[0]
        else:
            o = np.asarray(order, np.int64)
            pos = o[np.nonzero(mask[b][o])[0]]
        cu[b + 1] = cu[b] + pos.size
        idx.append(b * N + pos)
    idx = np.concatenate(idx) if idx else np.zeros(0, np.int64)
    inv = np.full(B * N, -1, dtype=np.int64)
    inv[idx] = np.arange(idx.size)
    return cu.astype(np.int32), idx.astype(np.int32), inv.astype(np.int32)


def pack_rows(x, idx, s=None, gate_scale=False):
    """Packed positive tokens r_p [N_p, C]: row i is token idx[i].

    With gate_scale the rows are first scaled by Sigmoid(s) as in Eq. 5.
    """
    x2 = np.asarray(x, F64).reshape(-1, np.shape(x)[-1])
    xp = x2[idx]
    if gate_scale:
        sig = 1.0 / (1.0 + np.exp(-np.asarray(s, F64).reshape(-1)[idx]))
        xp = xp * sig[:, None]
    return xp


def linear(a, W, b=None):
    """Dense layer on packed rows: out = a W^T + b, W stored [out, in]."""
    out = np.asarray(a, F64) @ np.asarray(W, F64).T
    if b is not None:
        out = out + np.asarray(b, F64)[None, :]
    return out


def container_cuts(cu_seqlens, L):
    """Boundaries when attention is limited to the same image AND the same length-L container.

    The packed buffer is cut at every multiple of L (containers, "Token Packing") and
    at every image boundary (the attention mask); returns the merged boundary list.
    """
    total = int(cu_seqlens[-1])
    cuts = set(int(c) for c in cu_seqlens)
    cuts.update(range(0, total + 1, L))
    cuts.add(total)
    return np.array(sorted(cuts), dtype=np.int32)


def attention_fwd(qkv, cu_seqlens, H, scale=None, return_probs=False):
    """Multi-head self-attention where packed tokens attend only within their own image.

    qkv [N_p, 3C] with column = which*C + h*d + e (which in q,k,v) -> ao [N_p, C]
    (column h*d+e) and lse [H, N_p] = log sum_j exp(S_ij).
    For each segment [cu[b], cu[b+1]) and head: S = scale * q k^T, P = softmax rows, o = P v.
    """
    qkv = np.asarray(qkv, F64)
    Np, C3 = qkv.shape
    C = C3 // 3
    d = C // H
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    ao = np.zeros((Np, C), F64)
    lse = np.zeros((H, Np), F64)
    probs = []
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if hi == lo:
            continue
        for h in range(H):
            q = qkv[lo:hi, 0 * C + h * d: 0 * C + (h + 1) * d]
            k = qkv[lo:hi, 1 * C + h * d: 1 * C + (h + 1) * d]
            v = qkv[lo:hi, 2 * C + h * d: 2 * C + (h + 1) * d]
            S = scale * (q @ k.T)
            m = S.max(axis=1, keepdims=True)
            E = np.exp(S - m)
            l = E.sum(axis=1, keepdims=True)
            P = E / l
            ao[lo:hi, h * d:(h + 1) * d] = P @ v
            lse[h, lo:hi] = (m + np.log(l))[:, 0]
            if return_probs:
                probs.append((b, h, P))
    if return_probs:
        return ao, lse, probs
    return ao, lse


def attention_fwd_masked_dense(qkv, cu_seqlens, H, scale=None):
    """The same attention written the way the paper words it: one attention over the
    whole packed buffer with a mask that hides tokens of other images (small inputs only)."""
    qkv = np.asarray(qkv, F64)
    Np, C3 = qkv.shape
    C = C3 // 3
    d = C // H
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    seg = np.zeros(Np, dtype=np.int64)
    for b in range(len(cu_seqlens) - 1):
        seg[int(cu_seqlens[b]):int(cu_seqlens[b + 1])] = b
    allowed = seg[:, None] == seg[None, :]
    ao = np.zeros((Np, C), F64)
    for h in range(H):
        q = qkv[:, h * d:(h + 1) * d]
        k = qkv[:, C + h * d: C + (h + 1) * d]
        v = qkv[:, 2 * C + h * d: 2 * C + (h + 1) * d]
        S = np.where(allowed, scale * (q @ k.T), -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        E = np.exp(S)
        ao[:, h * d:(h + 1) * d] = (E / E.sum(axis=1, keepdims=True)) @ v
    return ao


def unpack_scatter(z, x, idx, residual=False):
    """Write packed results back to their grid positions; other tokens pass through (Sec. 3.2:
    negative tokens go on unchanged).  residual=True gives y_sel = x + z instead of z."""
    x = np.asarray(x, F64)
    y = x.copy().reshape(-1, x.shape[-1])
    z = np.asarray(z, F64)
    if residual:
        y[idx] = y[idx] + z
    else:
        y[idx] = z
    return y.reshape(x.shape)


def block_fwd(x, w_g, b_g, tau, W_qkv, b_qkv, W_o, b_o, H, s_up=None, residual=False,
              gate_scale=False, scale=None, container_len=None, order=None):
    """One SPA block: gate -> select -> pack -> QKV -> same-image attention -> projection -> unpack.
    `order` packs each image's tokens in a given order (a shifted feature map) instead of raster order."""
    s = gate(x, w_g, b_g, s_up)
    mask = select(s, tau)
    cu, idx, inv = pack_indices(mask, order)
    xp = pack_rows(x, idx, s, gate_scale)
    qkv = linear(xp, W_qkv, b_qkv)
    seg = cu if container_len is None else container_cuts(cu, container_len)
    ao, lse = attention_fwd(qkv, seg, H, scale)
    z = linear(ao, W_o, b_o)
    y = unpack_scatter(z, x, idx, residual)
    return dict(scores=s, mask=mask, cu_seqlens=cu, idx=idx, inv=inv, xp=xp, qkv=qkv, ao=ao,
                lse=lse, z=z, y=y, seg=seg)


# --------------------------------------------------------------------------- backward
def unpack_scatter_bwd(dY, idx, residual=False):
    """Transpose of unpack_scatter: dz[i] = dY[idx[i]]; the pass-through part of dX is dY on
    unselected rows and (without residual) zero on selected rows, to which the packed path's
    gradient is added later by select_pack_bwd."""
    dY = np.asarray(dY, F64)
    flat = dY.reshape(-1, dY.shape[-1])
    dz = flat[idx].copy()
    dX = flat.copy()
    if not residual:
        dX[idx] = 0.0
    return dz, dX.reshape(dY.shape)


def linear_bwd(a, W, dout, need_bias=True):
    """Gradients of out = a W^T + b: da = dout W, dW = dout^T a, db = column sums of dout."""
    a = np.asarray(a, F64)
    W = np.asarray(W, F64)
    dout = np.asarray(dout, F64)
    da = dout @ W
    dW = dout.T @ a
    db = dout.sum(axis=0) if need_bias else None
    return da, dW, db


def attention_bwd(qkv, ao, lse, dao, cu_seqlens, H, scale=None):
    """Gradient of attention_fwd with respect to qkv.

    Per segment and head, with P_ij = exp(S_ij - lse_i) and D_i = sum_e dao_ie * ao_ie:
      dV = P^T dO;  dP = dO V^T;  dS = P * (dP - D);  dQ = scale * dS K;  dK = scale * dS^T Q.
    """
    qkv = np.asarray(qkv, F64)
    ao = np.asarray(ao, F64)
    dao = np.asarray(dao, F64)
    lse = np.asarray(lse, F64)
    Np, C3 = qkv.shape
    C = C3 // 3
    d = C // H
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    dqkv = np.zeros_like(qkv)
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if hi == lo:
            continue
        for h in range(H):
            cs = slice(h * d, (h + 1) * d)
            q = qkv[lo:hi, 0 * C + h * d: 0 * C + (h + 1) * d]
            k = qkv[lo:hi, 1 * C + h * d: 1 * C + (h + 1) * d]
            v = qkv[lo:hi, 2 * C + h * d: 2 * C + (h + 1) * d]
            dO = dao[lo:hi, cs]
            O = ao[lo:hi, cs]
            P = np.exp(scale * (q @ k.T) - lse[h, lo:hi][:, None])
            D = (dO * O).sum(axis=1, keepdims=True)
            dV = P.T @ dO
            dP = dO @ v.T
            dS = P * (dP - D)
            dqkv[lo:hi, 0 * C + h * d: 0 * C + (h + 1) * d] = scale * (dS @ k)
            dqkv[lo:hi, 1 * C + h * d: 1 * C + (h + 1) * d] = scale * (dS.T @ q)
            dqkv[lo:hi, 2 * C + h * d: 2 * C + (h + 1) * d] = dV
    return dqkv


def select_pack_bwd(dxp, idx, dX):
    """Transpose of the pack gather: dX[idx[i]] += dxp[i] (rows of idx are distinct)."""
    out = np.asarray(dX, F64).copy()
    flat = out.reshape(-1, out.shape[-1])
    flat[idx] = flat[idx] + np.asarray(dxp, F64)
    return out


def block_bwd(fwd, dY, x, W_qkv, W_o, H, residual=False, scale=None):
    """Backward of block_fwd (default flags) given its saved tensors `fwd` and upstream dY.

    No gradient reaches the gate: the hard threshold has zero derivative and the
    sigmoid scaling is off.  Returns dX and the four parameter gradients.
    """
    idx = fwd["idx"]
    dz, dX = unpack_scatter_bwd(dY, idx, residual)
    dao, dW_o, db_o = linear_bwd(fwd["ao"], W_o, dz)
    dqkv = attention_bwd(fwd["qkv"], fwd["ao"], fwd["lse"], dao, fwd["seg"], H, scale)
    dxp, dW_qkv, db_qkv = linear_bwd(fwd["xp"], W_qkv, dqkv)
    dX = select_pack_bwd(dxp, idx, dX)
    return dict(dz=dz, dao=dao, dqkv=dqkv, dxp=dxp, dX=dX, dW_o=dW_o, db_o=db_o,
                dW_qkv=dW_qkv, db_qkv=db_qkv)


# --------------------------------------------------------------------------- work model
def mac_count(B, N, C, cu_seqlens):
    """Multiply-accumulate count of the block in the notation of Eq. 7-9, with the packed terms
    written for variable segment lengths n_b: gate B*N*C; QKV 3*N_p*C^2; attention
    2*C*sum n_b^2; projection N_p*C^2."""
    n = np.diff(np.asarray(cu_seqlens, np.int64))
    Np = int(n.sum())
    S2 = int((n * n).sum())
    return dict(gate=B * N * C, qkv=3 * Np * C * C, attn=2 * C * S2, proj=Np * C * C,
                Np=Np, S2=S2)


# --------------------------------------------------------------------------- trainable selection
# Multi-scale supervised selection (Sec. 3.2) and the selection loss (Sec. 3.3, Eq. 10), with the
# gradients that make the gate trainable when the sigmoid scaling of Eq. 5 is on.  Readings fixed
# here: the up-scale scores reach the current scale by a 2x2 max-pool (each stage halves the grid);
# the loss is the sum over all B*N tokens of one block; "Max" in Eq. 4 passes its gradient to the
# larger argument (to s_up on a tie); the hard selection itself has no gradient.

def score_pool(scores_prev, B, rows, cols):
    """Scores of the previous (finer) stage, [B, 2*rows, 2*cols], max-pooled 2x2 to this stage's
    grid: s_up [B, rows*cols] (Sec. 3.2: scores from up-scaled features, adjusted via max-pooling)."""
    s = np.asarray(scores_prev, F64).reshape(B, rows, 2, cols, 2)
    return s.max(axis=(2, 4)).reshape(B, rows * cols)


def sigmoid(s):
    return 1.0 / (1.0 + np.exp(-np.asarray(s, F64)))


def select_loss(s, labels):
    """Selection loss of one block, Eq. 10: -sum(y log p + (1-y) log(1-p)), p = Sigmoid(s).

    Returns the loss and its gradient with respect to the logits s (p - y)."""
    s = np.asarray(s, F64)
    y = np.asarray(labels, F64)
    p = sigmoid(s)
    # log p and log(1-p) written through softplus so that large |s| does not overflow
    log_p = -np.logaddexp(0.0, -s)
    log_1mp = -np.logaddexp(0.0, s)
    loss = -(y * log_p + (1.0 - y) * log_1mp).sum()
    return loss, p - y


def pack_rows_bwd(dxp, x, s, idx, gate_scale=False):
    """Backward of pack_rows: gradient to the gathered rows of x and, with the sigmoid scaling of
    Eq. 5, to the logits of the selected tokens.

    xp_i = Sigmoid(s_t) x_t (t = idx[i])  =>  dx_t = Sigmoid(s_t) dxp_i,
    ds_t = Sigmoid'(s_t) (dxp_i . x_t) with Sigmoid' = p (1 - p)."""
    dxp = np.asarray(dxp, F64)
    x2 = np.asarray(x, F64).reshape(-1, np.shape(x)[-1])
    ds = np.zeros(x2.shape[0], F64)
    if not gate_scale:
        return dxp.copy(), ds
    p = sigmoid(np.asarray(s, F64).reshape(-1)[idx])
    ds[idx] = p * (1.0 - p) * (dxp * x2[idx]).sum(axis=1)
    return dxp * p[:, None], ds


def gate_bwd(ds, x, w_g, s, s_up=None):
    """Backward of gate(): ds [B*N] is the gradient with respect to the logits s = Max(f_g(r), s_up).

    Where the linear layer supplied the maximum (always, without s_up) the gradient goes to it:
    dx_t += ds_t w_g, dw_g = sum_t ds_t x_t, db_g = sum_t ds_t; elsewhere it goes to s_up."""
    x2 = np.asarray(x, F64).reshape(-1, np.shape(x)[-1])
    ds = np.asarray(ds, F64).reshape(-1)
    if s_up is None:
        lin = np.ones(ds.shape, bool)
    else:
        lin = np.asarray(s, F64).reshape(-1) > np.asarray(s_up, F64).reshape(-1)
    ds_lin = np.where(lin, ds, 0.0)
    dx = ds_lin[:, None] * np.asarray(w_g, F64)[None, :]
    dw_g = ds_lin @ x2
    db_g = ds_lin.sum()
    ds_up = np.where(lin, 0.0, ds)
    return dx.reshape(np.shape(x)), dw_g, db_g, ds_up


def block_bwd_trainable(fwd, dY, x, w_g, W_qkv, W_o, H, labels=None, alpha=1.0, s_up=None, residual=False,
                        gate_scale=True, scale=None):
    """Backward of block_fwd(..., gate_scale=...) for the total alpha * select_loss + <y, dY>:
    block_bwd plus the gradient through the sigmoid scaling (Eq. 5), the selection loss (Eq. 10)
    and the gate's linear layer (Eq. 4).  Returns block_bwd's dict extended by ds (gradient at the
    logits), dw_g, db_g, ds_up, loss."""
    idx = fwd["idx"]
    dz, dX = unpack_scatter_bwd(dY, idx, residual)
    dao, dW_o, db_o = linear_bwd(fwd["ao"], W_o, dz)
    dqkv = attention_bwd(fwd["qkv"], fwd["ao"], fwd["lse"], dao, fwd["seg"], H, scale)
    dxp, dW_qkv, db_qkv = linear_bwd(fwd["xp"], W_qkv, dqkv)
    dx_sel, ds = pack_rows_bwd(dxp, x, fwd["scores"], idx, gate_scale)
    dX = select_pack_bwd(dx_sel, idx, dX)
    loss = 0.0
    if labels is not None:
        loss, dl = select_loss(fwd["scores"].reshape(-1), np.asarray(labels, F64).reshape(-1))
        ds = ds + alpha * dl
    dx_gate, dw_g, db_g, ds_up = gate_bwd(ds, x, w_g, fwd["scores"], s_up)
    dX = dX + dx_gate
    return dict(dz=dz, dao=dao, dqkv=dqkv, dxp=dxp, dX=dX, dW_o=dW_o, db_o=db_o, dW_qkv=dW_qkv, db_qkv=db_qkv,
                ds=ds, dw_g=dw_g, db_g=db_g, ds_up=ds_up, loss=loss)


# --------------------------------------------------------------------------- the rest of the transformer block
# Pre-norm block around SPA (Sec. 3.2: selected tokens go through attention, the others are passed on to the
# feed-forward network): y1 = x + scatter(SPA(LN1(x))), out = y1 + FFN(LN2(y1)), FFN = W2 gelu(W1 t + b1) + b2.
# Readings fixed here (the paper's block figure is not in the text we have): LayerNorm with eps = 1e-5 over the
# channels, exact (erf) GELU, hidden width 4C, the gate reads the normalised tokens, the residual base of the
# selected tokens is x itself, and unselected tokens receive no attention update.

def layer_norm(x, gamma, beta, eps=1e-5):
    """y = (x - mean) / sqrt(var + eps) * gamma + beta over the last axis; also returns mean and rstd."""
    x = np.asarray(x, F64)
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    return (x - mean) * rstd * np.asarray(gamma, F64) + np.asarray(beta, F64), mean[..., 0], rstd[..., 0]


def layer_norm_bwd(dy, x, gamma, mean, rstd):
    """Gradients of layer_norm: dx, dgamma, dbeta."""
    dy = np.asarray(dy, F64)
    x = np.asarray(x, F64)
    xh = (x - mean[..., None]) * rstd[..., None]
    g = dy * np.asarray(gamma, F64)
    C = x.shape[-1]
    dx = (g - g.mean(axis=-1, keepdims=True) - xh * (g * xh).mean(axis=-1, keepdims=True)) * rstd[..., None]
    red = tuple(range(dy.ndim - 1))
    return dx, (dy * xh).sum(axis=red), dy.sum(axis=red)


def gelu(u):
    """Exact GELU: u Phi(u), Phi the standard normal distribution function."""
    from math import erf, sqrt
    u = np.asarray(u, F64)
    return 0.5 * u * (1.0 + np.vectorize(erf)(u / sqrt(2.0)))


def gelu_grad(u):
    """d gelu / du = Phi(u) + u phi(u)."""
    from math import erf, sqrt, pi
    u = np.asarray(u, F64)
    return 0.5 * (1.0 + np.vectorize(erf)(u / sqrt(2.0))) + u * np.exp(-0.5 * u * u) / sqrt(2.0 * pi)


def layer_fwd(x, prm, H, tau=0.0, eps=1e-5):
    """One pre-norm block.  prm: dict with g1, be1, w_g, b_g, W_qkv, b_qkv, W_o, b_o, g2, be2, W1, b1, W2, b2."""
    x = np.asarray(x, F64)
    z, m1, r1 = layer_norm(x, prm["g1"], prm["be1"], eps)
    spa = block_fwd(z, prm["w_g"], prm["b_g"], tau, prm["W_qkv"], prm["b_qkv"], prm["W_o"], prm["b_o"], H)
    y1 = x.reshape(-1, x.shape[-1]).copy()
    y1[spa["idx"]] += spa["z"]                      # residual on the selected tokens only
    y1 = y1.reshape(x.shape)
    t, m2, r2 = layer_norm(y1, prm["g2"], prm["be2"], eps)
    u = linear(t.reshape(-1, x.shape[-1]), prm["W1"], prm["b1"])
    h = gelu(u)
    out = y1 + linear(h, prm["W2"], prm["b2"]).reshape(x.shape)
    return dict(z=z, m1=m1, r1=r1, spa=spa, y1=y1, t=t, m2=m2, r2=r2, u=u, h=h, out=out)


def layer_bwd(f, d_out, x, prm, H):
    """Backward of layer_fwd: gradient to x and to every parameter except the gate (hard selection)."""
    x = np.asarray(x, F64)
    C = x.shape[-1]
    d_out = np.asarray(d_out, F64)
    dh, dW2, db2 = linear_bwd(f["h"], prm["W2"], d_out.reshape(-1, C))
    du = dh * gelu_grad(f["u"])
    dt, dW1, db1 = linear_bwd(f["t"].reshape(-1, C), prm["W1"], du)
    dy1_ln, dg2, dbe2 = layer_norm_bwd(dt.reshape(x.shape), f["y1"], prm["g2"], f["m2"], f["r2"])
    dy1 = d_out + dy1_ln
    spa = f["spa"]
    idx = spa["idx"]
    dz_packed = dy1.reshape(-1, C)[idx]
    dao, dW_o, db_o = linear_bwd(spa["ao"], prm["W_o"], dz_packed)
    dqkv = attention_bwd(spa["qkv"], spa["ao"], spa["lse"], dao, spa["seg"], H)
    dxp, dW_qkv, db_qkv = linear_bwd(spa["xp"], prm["W_qkv"], dqkv)
    dZ = np.zeros((x.size // C, C), F64)
    dZ[idx] = dxp
    dx_ln, dg1, dbe1 = layer_norm_bwd(dZ.reshape(x.shape), x, prm["g1"], f["m1"], f["r1"])
    return dict(dX=dy1 + dx_ln, dg1=dg1, dbe1=dbe1, dg2=dg2, dbe2=dbe2, dW1=dW1, db1=db1, dW2=dW2, db2=db2,
                dW_qkv=dW_qkv, db_qkv=db_qkv, dW_o=dW_o, db_o=db_o, dy1=dy1, du=du, dt=dt, dZ=dZ)
