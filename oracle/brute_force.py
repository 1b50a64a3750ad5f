"""Brute-force second opinion on the SPA block.  TEST INFRASTRUCTURE ONLY.

For every image on its own: copy the rows whose gate logit exceeds the threshold into a
small dense matrix, run textbook multi-head attention on it with scalar loops, and copy
the results back.  No packed buffer, no cu_seqlens, no gather index is ever built, so an
indexing mistake in the packed oracle cannot be repeated here.  Pure-Python loops: use
on tiny inputs only.  (Paper Sec. 3.2: selected tokens get multi-head self-attention
among tokens of the same image; the others pass through.)
"""
from __future__ import annotations

import math

import numpy as np


def block_fwd_bruteforce(x, w_g, b_g, tau, W_qkv, b_qkv, W_o, b_o, H, residual=False):
    x = np.asarray(x, np.float64)
    B, N, C = x.shape
    d = C // H
    y = x.copy()
    for b in range(B):
        rows = []
        for n in range(N):
            s = float(b_g)
            for c in range(C):
                s += float(w_g[c]) * x[b, n, c]
            if s > tau:
                rows.append(n)
        L = len(rows)
        if L == 0:
            continue
        t = np.stack([x[b, n] for n in rows])                     # [L, C]
        q = np.zeros((L, C)); k = np.zeros((L, C)); v = np.zeros((L, C))
        for i in range(L):
            for j in range(C):
                q[i, j] = b_qkv[j] + float(np.dot(W_qkv[j], t[i]))
                k[i, j] = b_qkv[C + j] + float(np.dot(W_qkv[C + j], t[i]))
                v[i, j] = b_qkv[2 * C + j] + float(np.dot(W_qkv[2 * C + j], t[i]))
        o = np.zeros((L, C))
        for h in range(H):
            for i in range(L):
                logits = [float(np.dot(q[i, h * d:(h + 1) * d], k[j, h * d:(h + 1) * d])) / math.sqrt(d)
                          for j in range(L)]
                mx = max(logits)
                w = [math.exp(a - mx) for a in logits]
                tot = sum(w)
                for j in range(L):
                    o[i, h * d:(h + 1) * d] += (w[j] / tot) * v[j, h * d:(h + 1) * d]
        for i, n in enumerate(rows):
            zi = np.array([b_o[j] + float(np.dot(W_o[j], o[i])) for j in range(C)])
            y[b, n] = x[b, n] + zi if residual else zi
    return y
