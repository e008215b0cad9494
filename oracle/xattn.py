"""CPU float64 oracle for one pre-norm cross-attention layer, forward and backward.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the CPU-baseline leg of the benchmark, never by
the product path; it shares no code with the CUDA side.

What it follows.  The paper lists cross-attention beside MHA and GQA among the attention mechanisms whose tensor
partitioning the layout has to serve (its background section), and evaluates models that contain it (Whisper,
Stable Diffusion in its model table).  The arithmetic is the textbook definition: the layer of ``oracle.layer`` with
the keys and values projected from a second sequence, the memory M, instead of from the normalised hidden states.

forward, per batch element (X: [Tq, D], M: [Tk, Dm])
  1. Xn = norm(X)                                    (LayerNorm or RMSNorm, as in the self-attention layer)
  2. Q = Xn Wq + bq,  K = M Wk + bk,  V = M Wv + bv   (Wk, Wv: [Dm, Dkv]; the memory is used as it is)
  3. query head h reads KV head g = h // G
  4. S_ij = scale * <Q[i,h,:], K[j,g,:]> for every i < Tq, j < Tk (no mask), P = softmax_j S, LSE_i
  5. O[i,h,:] = sum_j P_ij V[j,g,:], A = heads concatenated, Y = A Wo + bo (+ X)

backward, given dY
  6. dWo = A^T dY, dbo = sum dY, dA = dY Wo^T
  7. per head: dV += P^T dO, dP = dO V^T, D_i = <dO_i, O_i>, dS = P (dP - D_i), dQ = scale dS K, dK += scale dS^T Q
  8. dWq = Xn^T dQ, dbq = sum dQ, dXn = dQ Wq^T
     dWk = M^T dK, dWv = M^T dV, dbk, dbv,  dM = dK Wk^T + dV Wv^T
  9. dX, dgamma, dbeta through the norm (+ dY if residual)

Pins (tests/test_oracle_xattn_pins.py): central finite differences of every gradient including dM, a scalar-loop
attention over two lengths, the closed form for one memory token (P = 1, O = V, no gradient through the scores),
dbk == 0 and dbv as a column sum, invariance under a permutation of the memory axis, batch additivity, and the
self-attention oracle on the case where the two layers coincide (M := the normalised input, no mask).
"""
from __future__ import annotations

import numpy as np

from .layer import attention_head_fwd, norm_fwd


def xattn_fwd(cfg, X, M, gamma, beta, Wq, Wk, Wv, Wo, bq=None, bk=None, bv=None, bo=None):
    """Forward.  X: [B, Tq, D], M: [B, Tk, Dm].  Returns Y and what the backward reuses."""
    B, Tq, _ = X.shape
    Hq, hd, G = cfg.n_q_heads, cfg.head_dim, cfg.group
    Xn, xhat, rstd, mu = norm_fwd(X, gamma, beta, cfg.eps, cfg.norm)
    Q = Xn @ Wq + (bq if bq is not None else 0.0)
    K = M @ Wk + (bk if bk is not None else 0.0)
    V = M @ Wv + (bv if bv is not None else 0.0)
    A = np.zeros((B, Tq, Hq * hd))
    LSE = np.zeros((B, Hq, Tq))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            o, _, lse = attention_head_fwd(Q[b, :, h * hd:(h + 1) * hd], K[b, :, g * hd:(g + 1) * hd],
                                           V[b, :, g * hd:(g + 1) * hd], cfg.scale, False)
            A[b, :, h * hd:(h + 1) * hd] = o
            LSE[b, h] = lse
    Y = A @ Wo + (bo if bo is not None else 0.0)
    if cfg.residual:
        Y = Y + X
    return Y, dict(Xn=Xn, xhat=xhat, rstd=rstd, mu=mu, Q=Q, K=K, V=V, A=A, LSE=LSE)


def xattn_bwd(cfg, dY, X, M, gamma, Wq, Wk, Wv, Wo, saved):
    """Backward.  Returns a dict of every gradient and the intermediates."""
    B, Tq, _ = X.shape
    Hq, hd, G = cfg.n_q_heads, cfg.head_dim, cfg.group
    Xn, xhat, rstd = saved["Xn"], saved["xhat"], saved["rstd"]
    Q, K, V, A = saved["Q"], saved["K"], saved["V"], saved["A"]
    flat = lambda t: t.reshape(-1, t.shape[-1])

    dWo = flat(A).T @ flat(dY)
    dbo = flat(dY).sum(axis=0)
    dA = dY @ Wo.T

    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    Dvec = np.zeros((B, Hq, Tq))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            qs, ks = slice(h * hd, (h + 1) * hd), slice(g * hd, (g + 1) * hd)
            q, k, v = Q[b, :, qs], K[b, :, ks], V[b, :, ks]
            _, P, _ = attention_head_fwd(q, k, v, cfg.scale, False)
            dO = dA[b, :, qs]
            dV[b, :, ks] += P.T @ dO
            dP = dO @ v.T
            Di = (dO * A[b, :, qs]).sum(axis=1)
            dS = P * (dP - Di[:, None])
            dQ[b, :, qs] = cfg.scale * (dS @ k)
            dK[b, :, ks] += cfg.scale * (dS.T @ q)
            Dvec[b, h] = Di

    dWq = flat(Xn).T @ flat(dQ)
    dbq = flat(dQ).sum(axis=0)
    dXn = dQ @ Wq.T
    dWk = flat(M).T @ flat(dK)
    dWv = flat(M).T @ flat(dV)
    dbk, dbv = flat(dK).sum(axis=0), flat(dV).sum(axis=0)
    dM = dK @ Wk.T + dV @ Wv.T

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
    out = dict(dX=dX, dM=dM, dWq=dWq, dWk=dWk, dWv=dWv, dWo=dWo, dgamma=dgamma,
               dA=dA, dQ=dQ, dK=dK, dV=dV, dXn=dXn, D=Dvec, dbq=dbq, dbk=dbk, dbv=dbv, dbo=dbo)
    if cfg.norm == "layernorm":
        out["dbeta"] = dbeta
    return out


def xattn_fwd_bwd(cfg, inp):
    """Convenience wrapper over a dict from ``fbl_inputs.make_xattn_inputs``."""
    Y, saved = xattn_fwd(cfg, inp["X"], inp["M"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                         inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    grads = xattn_bwd(cfg, inp["dY"], inp["X"], inp["M"], inp["gamma"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"], saved)
    return Y, saved, grads
