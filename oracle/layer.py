"""CPU float64 oracle for one pre-norm self-attention layer, forward and backward.

TEST INFRASTRUCTURE ONLY.  This file is the plain definition of what the CUDA path
must compute; it shares no code with that path and is imported only by tests, the
smoke check and the CPU-baseline leg of the benchmark.

What it follows.  The paper names the layer's operators (its motivating example:
projections, P = softmax(QK^T), O = PV, and their gradients) and fixes the matmul
convention through dW = X^T dY (its operator-classification section, FTD-D
matmul), i.e. Y = X W with W of shape [d_in, d_out].  The arithmetic itself is the
textbook definition, written out here step by step in float64:

forward, per batch element
  1. LayerNorm  mu = mean_d X, var = mean_d (X-mu)^2 (biased), rstd = (var+eps)^-1/2,
                xhat = (X-mu) rstd, Xn = xhat*gamma + beta
     RMSNorm    rstd = (mean_d X^2 + eps)^-1/2, xhat = X rstd, Xn = xhat*gamma
  2. Q = Xn Wq + bq, K = Xn Wk + bk, V = Xn Wv + bv
  2b. (optional, cfg.rope_base > 0) rotary position embedding on Q and K, see ``rope``
  3. query head h owns columns [h*hd, (h+1)*hd); its KV head is g = h // G
  4. S_ij = scale * sum_d Q[i,h,d] K[j,g,d]; causal keeps only j <= i
     m_i = max_j S_ij, l_i = sum_j exp(S_ij - m_i), P_ij = exp(S_ij - m_i)/l_i,
     LSE_i = m_i + ln l_i
  5. O[i,h,:] = sum_j P_ij V[j,g,:], A = heads concatenated, Y = A Wo + bo (+ X)

backward, given dY
  6. dWo = A^T dY, dbo = sum_tokens dY, dA = dY Wo^T
  7. dV_h = P^T dO_h, dP = dO_h V_g^T, D_i = sum_d dO[i,h,d] O[i,h,d],
     dS = P * (dP - D_i), dQ_h = scale dS K_g, dK_h = scale dS^T Q_h,
     dK_g = sum_{h in g} dK_h, dV_g = sum_{h in g} dV_h
  8. dW* = Xn^T d*, db* = sum_tokens d*, dXn = dQ Wq^T + dK Wk^T + dV Wv^T
  9. dgamma = sum_tokens dXn*xhat, dbeta = sum_tokens dXn, g = dXn*gamma,
     LayerNorm dX = rstd (g - mean_d g - xhat mean_d(g xhat))
     RMSNorm   dX = rstd (g - xhat mean_d(g xhat)),   (+ dY if residual)

S and P are materialised per (batch, head); numpy's matmul is the only library
step.  Nothing is blocked, fused or reordered.

Pins (tests/test_oracle_pins.py): central finite differences of every gradient,
softmax rows summing to one, rows of dS summing to zero, a triple-loop attention
(oracle/naive.py), closed forms (zero Wq gives uniform attention; T = 1), GQA
against the equivalent MHA layer, batch additivity, causality, linearity of the
backward, dbk == 0, and an independently written einsum formulation.
"""
from __future__ import annotations

import numpy as np


def norm_fwd(X, gamma, beta, eps, kind):
    """Step 1.  X: [..., D].  Returns Xn, xhat, rstd (and mu for LayerNorm, else None)."""
    if kind == "layernorm":
        mu = X.mean(axis=-1, keepdims=True)
        var = ((X - mu) ** 2).mean(axis=-1, keepdims=True)
        rstd = 1.0 / np.sqrt(var + eps)
        xhat = (X - mu) * rstd
        Xn = xhat * gamma + (beta if beta is not None else 0.0)
        return Xn, xhat, rstd, mu
    if kind == "rmsnorm":
        rstd = 1.0 / np.sqrt((X ** 2).mean(axis=-1, keepdims=True) + eps)
        xhat = X * rstd
        return xhat * gamma, xhat, rstd, None
    raise ValueError(kind)


def rope(x, heads, base, inverse=False, pos_offset=0):
    """Rotary position embedding on x: [B, T, heads * hd], half-split pairing: inside every head, element i < hd/2
    is paired with element i + hd/2 and the pair of token t is rotated by the angle (t + pos_offset) * base^(-2i/hd):
        y_i      = x_i cos - x_{i+hd/2} sin
        y_{i+hd/2} = x_{i+hd/2} cos + x_i sin
    ``inverse`` rotates by the opposite angle (the transpose of the rotation: what the backward applies)."""
    B, T, C = x.shape
    hd = C // heads
    half = hd // 2
    ang = (np.arange(T, dtype=np.float64)[:, None] + pos_offset) * base ** (-2.0 * np.arange(half, dtype=np.float64) / hd)[None, :]
    cos, sin = np.cos(ang)[None, :, None, :], np.sin(ang)[None, :, None, :]
    if inverse:
        sin = -sin
    xh = x.reshape(B, T, heads, hd)
    lo, hi = xh[..., :half], xh[..., half:]
    return np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1).reshape(B, T, C)


def attention_head_fwd(q, k, v, scale, causal):
    """Steps 4-5 for one (batch, head).  q: [T, hd], k, v: [T, hd].  Returns O, P, LSE."""
    T = q.shape[0]
    S = scale * (q @ k.T)
    if causal:
        S = np.where(np.tril(np.ones((T, T), dtype=bool)), S, -np.inf)
    m = S.max(axis=1, keepdims=True)
    e = np.exp(S - m)
    l = e.sum(axis=1, keepdims=True)
    P = e / l
    return P @ v, P, (m + np.log(l))[:, 0]


def layer_fwd(cfg, X, gamma, beta, Wq, Wk, Wv, Wo, bq=None, bk=None, bv=None, bo=None):
    """Forward of the whole layer.  X: [B, T, D].  Returns Y and everything the backward reuses."""
    B, T, D = X.shape
    Hq, Hkv, hd, G = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.group
    Xn, xhat, rstd, mu = norm_fwd(X, gamma, beta, cfg.eps, cfg.norm)
    Q = Xn @ Wq + (bq if bq is not None else 0.0)
    K = Xn @ Wk + (bk if bk is not None else 0.0)
    V = Xn @ Wv + (bv if bv is not None else 0.0)
    if getattr(cfg, "rope_base", 0.0) > 0.0:       # optional step 2b: Q and K rotated by position; `saved` holds the rotated ones
        Q, K = rope(Q, Hq, cfg.rope_base), rope(K, Hkv, cfg.rope_base)
    A = np.zeros((B, T, Hq * hd))
    LSE = np.zeros((B, Hq, T))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            o, _, lse = attention_head_fwd(Q[b, :, h * hd:(h + 1) * hd], K[b, :, g * hd:(g + 1) * hd],
                                           V[b, :, g * hd:(g + 1) * hd], cfg.scale, cfg.causal)
            A[b, :, h * hd:(h + 1) * hd] = o
            LSE[b, h] = lse
    Y = A @ Wo + (bo if bo is not None else 0.0)
    if cfg.residual:
        Y = Y + X
    saved = dict(Xn=Xn, xhat=xhat, rstd=rstd, mu=mu, Q=Q, K=K, V=V, A=A, LSE=LSE)
    return Y, saved


def layer_bwd(cfg, dY, X, gamma, Wq, Wk, Wv, Wo, saved):
    """Backward of the whole layer.  Returns a dict of every gradient (and the intermediates)."""
    B, T, D = X.shape
    Hq, Hkv, hd, G = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.group
    Xn, xhat, rstd = saved["Xn"], saved["xhat"], saved["rstd"]
    Q, K, V, A = saved["Q"], saved["K"], saved["V"], saved["A"]
    flat = lambda t: t.reshape(B * T, -1)

    # step 6
    dWo = flat(A).T @ flat(dY)
    dbo = flat(dY).sum(axis=0)
    dA = dY @ Wo.T

    # step 7
    dQ = np.zeros_like(Q)
    dK = np.zeros_like(K)
    dV = np.zeros_like(V)
    Dvec = np.zeros((B, Hq, T))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            qs, ks = slice(h * hd, (h + 1) * hd), slice(g * hd, (g + 1) * hd)
            q, k, v = Q[b, :, qs], K[b, :, ks], V[b, :, ks]
            _, P, _ = attention_head_fwd(q, k, v, cfg.scale, cfg.causal)
            dO = dA[b, :, qs]
            dV[b, :, ks] += P.T @ dO
            dP = dO @ v.T
            Di = (dO * A[b, :, qs]).sum(axis=1)
            dS = P * (dP - Di[:, None])
            dQ[b, :, qs] = cfg.scale * (dS @ k)
            dK[b, :, ks] += cfg.scale * (dS.T @ q)
            Dvec[b, h] = Di

    # optional step 7b: back through the rotation of Q and K (an orthogonal map: its transpose is the inverse rotation)
    dQ_rot, dK_rot = dQ, dK
    if getattr(cfg, "rope_base", 0.0) > 0.0:
        dQ, dK = rope(dQ, Hq, cfg.rope_base, inverse=True), rope(dK, Hkv, cfg.rope_base, inverse=True)

    # step 8
    dWq = flat(Xn).T @ flat(dQ)
    dWk = flat(Xn).T @ flat(dK)
    dWv = flat(Xn).T @ flat(dV)
    dbq, dbk, dbv = flat(dQ).sum(axis=0), flat(dK).sum(axis=0), flat(dV).sum(axis=0)
    dXn = dQ @ Wq.T + dK @ Wk.T + dV @ Wv.T

    # step 9
    dgamma = flat(dXn * xhat).sum(axis=0)
    dbeta = flat(dXn).sum(axis=0)
    gg = dXn * gamma
    c2 = (gg * xhat).mean(axis=-1, keepdims=True)
    if cfg.norm == "layernorm":
        dX = rstd * (gg - gg.mean(axis=-1, keepdims=True) - xhat * c2)
    else:
        dX = rstd * (gg - xhat * c2)
    if cfg.residual:
        dX = dX + dY
    out = dict(dX=dX, dWq=dWq, dWk=dWk, dWv=dWv, dWo=dWo, dgamma=dgamma,
               dA=dA, dQ=dQ, dK=dK, dV=dV, dXn=dXn, D=Dvec, dQ_rot=dQ_rot, dK_rot=dK_rot)
    if cfg.norm == "layernorm":
        out["dbeta"] = dbeta
    out.update(dbq=dbq, dbk=dbk, dbv=dbv, dbo=dbo)   # defined with or without biases in the layer
    return out


def layer_fwd_bwd(cfg, inp):
    """Convenience wrapper over a dict from ``fbl_inputs.make_inputs``."""
    Y, saved = layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                         inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    grads = layer_bwd(cfg, inp["dY"], inp["X"], inp["gamma"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"], saved)
    return Y, saved, grads
