"""Brute-force and independently formulated checks for oracle/layer.py.

TEST INFRASTRUCTURE ONLY.  Two things live here, both used only to pin the oracle:

* ``naive_attention``: scalar triple loops straight from the definition
  P_ij = exp(S_ij) / sum_j exp(S_ij) with no max subtraction (float64 has the
  range for the tiny cases it is used on).
* ``einsum_layer``: the whole layer, all heads and batches at once through
  ``numpy.einsum`` on 4-D head-split arrays, with the softmax Jacobian applied in
  its textbook form dS = P*(dP - sum_j P dP) (so D is obtained a second way), and
  GQA done by physically repeating K and V and summing the repeated gradients.
"""
from __future__ import annotations

import math

import numpy as np


def naive_attention(q, k, v, scale, causal):
    T, hd = q.shape
    O = [[0.0] * hd for _ in range(T)]
    P = [[0.0] * T for _ in range(T)]
    for i in range(T):
        last = i if causal else T - 1
        w = []
        for j in range(last + 1):
            s = 0.0
            for d in range(hd):
                s += float(q[i, d]) * float(k[j, d])
            w.append(math.exp(scale * s))
        tot = sum(w)
        for j in range(last + 1):
            P[i][j] = w[j] / tot
            for d in range(hd):
                O[i][d] += P[i][j] * float(v[j, d])
    return np.array(O), np.array(P)


def einsum_layer(cfg, inp):
    X, dY = inp["X"], inp["dY"]
    B, T, D = X.shape
    Hq, Hkv, hd, G = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.group
    gamma = inp["gamma"]
    zero = lambda v: 0.0 if v is None else v
    if cfg.norm == "layernorm":
        xc = X - np.einsum("btd->bt", X)[..., None] / D
        rstd = (np.einsum("btd,btd->bt", xc, xc) / D + cfg.eps) ** -0.5
        xhat = xc * rstd[..., None]
        Xn = xhat * gamma + zero(inp["beta"])
    else:
        rstd = (np.einsum("btd,btd->bt", X, X) / D + cfg.eps) ** -0.5
        xhat = X * rstd[..., None]
        Xn = xhat * gamma
    Q = (np.einsum("btd,de->bte", Xn, inp["Wq"]) + zero(inp["bq"])).reshape(B, T, Hq, hd)
    K = (np.einsum("btd,de->bte", Xn, inp["Wk"]) + zero(inp["bk"])).reshape(B, T, Hkv, hd)
    V = (np.einsum("btd,de->bte", Xn, inp["Wv"]) + zero(inp["bv"])).reshape(B, T, Hkv, hd)
    Kr, Vr = np.repeat(K, G, axis=2), np.repeat(V, G, axis=2)        # explicit GQA expansion
    S = cfg.scale * np.einsum("bihd,bjhd->bhij", Q, Kr)
    if cfg.causal:
        S = S + np.triu(np.full((T, T), -np.inf), k=1)
    P = np.exp(S - S.max(axis=-1, keepdims=True))
    P = P / P.sum(axis=-1, keepdims=True)
    O = np.einsum("bhij,bjhd->bihd", P, Vr)
    A = O.reshape(B, T, Hq * hd)
    Y = np.einsum("bte,ed->btd", A, inp["Wo"]) + zero(inp["bo"]) + (X if cfg.residual else 0.0)

    dWo = np.einsum("bte,btd->ed", A, dY)
    dO = np.einsum("btd,ed->bte", dY, inp["Wo"]).reshape(B, T, Hq, hd)
    dVr = np.einsum("bhij,bihd->bjhd", P, dO)
    dP = np.einsum("bihd,bjhd->bhij", dO, Vr)
    dS = P * (dP - np.einsum("bhij,bhij->bhi", P, dP)[..., None])
    dQ = cfg.scale * np.einsum("bhij,bjhd->bihd", dS, Kr)
    dKr = cfg.scale * np.einsum("bhij,bihd->bjhd", dS, Q)
    dK = dKr.reshape(B, T, Hkv, G, hd).sum(axis=3)
    dV = dVr.reshape(B, T, Hkv, G, hd).sum(axis=3)
    dQf, dKf, dVf = dQ.reshape(B, T, -1), dK.reshape(B, T, -1), dV.reshape(B, T, -1)
    dXn = (np.einsum("bte,de->btd", dQf, inp["Wq"]) + np.einsum("bte,de->btd", dKf, inp["Wk"])
           + np.einsum("bte,de->btd", dVf, inp["Wv"]))
    g = dXn * gamma
    gx = np.einsum("btd,btd->bt", g, xhat)[..., None] / D
    dX = g - xhat * gx
    if cfg.norm == "layernorm":
        dX = dX - np.einsum("btd->bt", g)[..., None] / D
    dX = dX * rstd[..., None] + (dY if cfg.residual else 0.0)
    return dict(Y=Y, dX=dX, dWo=dWo,
                dWq=np.einsum("btd,bte->de", Xn, dQf), dWk=np.einsum("btd,bte->de", Xn, dKf),
                dWv=np.einsum("btd,bte->de", Xn, dVf),
                dbq=dQf.sum((0, 1)), dbk=dKf.sum((0, 1)), dbv=dVf.sum((0, 1)), dbo=dY.sum((0, 1)),
                dgamma=np.einsum("btd,btd->d", dXn, xhat), dbeta=dXn.sum((0, 1)))
