"""Rounding floor of a bf16-storage implementation of the layer, computed on the CPU from the oracle alone.

The float64 oracle's steps are repeated with every tensor that a bf16 implementation must round -- whatever
crosses HBM or feeds a bf16 tensor-core operand: Xn, Q, K, V, the un-normalised probabilities, A, Y, dA, the
normalised probabilities and dS of the backward, dQ, dK, dV, dXn, dX and the weight gradients -- rounded to
bf16 (round to nearest even) and every sum kept exact (float64).  What comes out differs from the oracle only by
those roundings, so its error against the oracle bounds from below the error of any kernel with bf16 operands and
bf16 outputs, whatever its accumulation order.  The tolerance constants of the GPU parity tests are set from the
figures this produces (util.py).

Test infrastructure: imports numpy, ``oracle`` and the shared input generator only; nothing of the CUDA package.
"""
from __future__ import annotations

import numpy as np

from fbl_inputs import round_to_storage
from oracle import layer as orc

BF16_RTOL, BF16_ATOL = 2e-2, 1e-2


def r16(x):
    return round_to_storage(np.asarray(x, dtype=np.float64), "bf16")


def emulate(cfg, inp):
    """Forward and backward with bf16-rounded intermediates and exact sums.  Returns a dict of outputs."""
    X, dY = inp["X"], inp["dY"]
    Wq, Wk, Wv, Wo = inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"]
    z = lambda b: b if b is not None else 0.0
    B, T, D = X.shape
    Hq, hd, G = cfg.n_q_heads, cfg.head_dim, cfg.group
    flat = lambda t: t.reshape(-1, t.shape[-1])
    mem = inp.get("M")                 # cross-attention: K and V come from the memory, which is an input (no rounding)

    Xn_exact, xhat, rstd, mu = orc.norm_fwd(X, inp["gamma"], inp["beta"], cfg.eps, cfg.norm)
    Xn = r16(Xn_exact)
    src_kv = Xn if mem is None else mem
    Q, K, V = r16(Xn @ Wq + z(inp["bq"])), r16(src_kv @ Wk + z(inp["bk"])), r16(src_kv @ Wv + z(inp["bv"]))
    rope_base = getattr(cfg, "rope_base", 0.0)
    if rope_base > 0.0:               # rotated in place: read as bf16, written as bf16
        Q, K = r16(orc.rope(Q, Hq, rope_base)), r16(orc.rope(K, cfg.n_kv_heads, rope_base))
    A = np.zeros((B, T, Hq * hd))
    LSE = np.zeros((B, Hq, T))
    mask = np.tril(np.ones((T, T), dtype=bool)) if cfg.causal else None
    for b in range(B):
        for h in range(Hq):
            g = h // G
            qs, ks = slice(h * hd, (h + 1) * hd), slice(g * hd, (g + 1) * hd)
            S = cfg.scale * (Q[b, :, qs] @ K[b, :, ks].T)
            if mask is not None:
                S = np.where(mask, S, -np.inf)
            m = S.max(axis=1, keepdims=True)
            e = np.exp(S - m)
            l = e.sum(axis=1, keepdims=True)               # the row sum is kept in fp32: unrounded probabilities
            A[b, :, qs] = r16((r16(e) @ V[b, :, ks]) / l)   # the P V operand is bf16
            LSE[b, h] = (m + np.log(l))[:, 0]
    Y = A @ Wo + z(inp["bo"])
    if cfg.residual:
        Y = Y + X
    out = {"Y": r16(Y)}

    dA = r16(dY @ Wo.T)
    out["dWo"] = r16(flat(A).T @ flat(dY))
    out["dbo"] = flat(dY).sum(axis=0)
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            qs, ks = slice(h * hd, (h + 1) * hd), slice(g * hd, (g + 1) * hd)
            q, k, v, dO = Q[b, :, qs], K[b, :, ks], V[b, :, ks], dA[b, :, qs]
            S = cfg.scale * (q @ k.T)
            P = np.exp(S - LSE[b, h][:, None])
            if mask is not None:
                P = np.where(mask, P, 0.0)
            Di = (dO * A[b, :, qs]).sum(axis=1)
            dS = r16(P * (dO @ v.T - Di[:, None]))
            dV[b, :, ks] += r16(P).T @ dO
            dQ[b, :, qs] = cfg.scale * (dS @ k)
            dK[b, :, ks] += cfg.scale * (dS.T @ q)
    dQ, dK, dV = r16(dQ), r16(dK), r16(dV)
    if rope_base > 0.0:
        dQ, dK = r16(orc.rope(dQ, Hq, rope_base, inverse=True)), r16(orc.rope(dK, cfg.n_kv_heads, rope_base, inverse=True))
    out["dWq"], out["dWk"], out["dWv"] = r16(flat(Xn).T @ flat(dQ)), r16(flat(src_kv).T @ flat(dK)), r16(flat(src_kv).T @ flat(dV))
    out["dbq"], out["dbk"], out["dbv"] = flat(dQ).sum(axis=0), flat(dK).sum(axis=0), flat(dV).sum(axis=0)
    if mem is None:
        dXn = r16(dQ @ Wq.T + dK @ Wk.T + dV @ Wv.T)
    else:
        dXn = r16(dQ @ Wq.T)
        out["dM"] = r16(dK @ Wk.T + dV @ Wv.T)
    out["dgamma"] = flat(dXn * xhat).sum(axis=0)
    if cfg.norm == "layernorm":
        out["dbeta"] = flat(dXn).sum(axis=0)
    gg = dXn * inp["gamma"]
    c2 = (gg * xhat).mean(axis=-1, keepdims=True)
    dX = rstd * (gg - (gg.mean(axis=-1, keepdims=True) if cfg.norm == "layernorm" else 0.0) - xhat * c2)
    if cfg.residual:
        dX = dX + dY
    out["dX"] = r16(dX)
    return out


def floor_figures(cfg, inp, ref=None):
    """Per output tensor: max|e|, max|e| / (1e-2 + 2e-2 max|ref|), relative Frobenius error and the fraction of
    elements outside the element-wise bound |e| <= 1e-2 + 2e-2 |ref|, of the emulation against the oracle
    (``ref``: the oracle's outputs by name, computed here when not given)."""
    if ref is None:
        if "M" in inp:
            from oracle import xattn
            Y, _, g = xattn.xattn_fwd_bwd(cfg, inp)
        else:
            Y, _, g = orc.layer_fwd_bwd(cfg, inp)
        ref = dict(g)
        ref["Y"] = Y
    emu = emulate(cfg, inp)
    fig = {}
    for name, got in emu.items():
        if not cfg.has_bias and name in ("dbq", "dbk", "dbv", "dbo"):
            continue
        r = ref[name]
        e = np.abs(got - r)
        fig[name] = dict(max_abs=float(e.max()),
                         worst_over_bound=float(e.max() / (BF16_ATOL + BF16_RTOL * np.abs(r).max())),
                         fro=float(np.linalg.norm(got - r) / (np.linalg.norm(r) + 1e-300)),
                         viol=float((e > BF16_ATOL + BF16_RTOL * np.abs(r)).mean()),
                         numel=int(r.size))
    return fig


def emulate_mlp(cfg, inp):
    """The feed-forward block (oracle/mlp.py) with bf16-rounded intermediates (Xn, U, G, H, Y, dH-derived dU and
    dG, dXn, dX, weight gradients) and exact sums."""
    from oracle import mlp as om
    X, dY = inp["X"], inp["dY"]
    z = lambda b: b if b is not None else 0.0
    B, T, D = X.shape
    flat = lambda t: t.reshape(B * T, -1)
    Xn_exact, xhat, rstd, mu = orc.norm_fwd(X, inp["gamma"], inp["beta"], cfg.eps, cfg.norm)
    Xn = r16(Xn_exact)
    U = r16(Xn @ inp["W1"] + z(inp["b1"]))
    if cfg.gated:
        G = r16(Xn @ inp["Wg"] + z(inp["bg"]))
        H = r16(om.silu(G) * U)
    else:
        G = None
        H = r16(om.gelu(U))
    Y = H @ inp["W2"] + z(inp["b2"])
    if cfg.residual:
        Y = Y + X
    out = {"Y": r16(Y), "dW2": r16(flat(H).T @ flat(dY)), "db2": flat(dY).sum(axis=0)}
    dH = r16(dY @ inp["W2"].T)
    if cfg.gated:
        dU, dG = r16(dH * om.silu(G)), r16(dH * U * om.silu_grad(G))
        out["dWg"], out["dbg"] = r16(flat(Xn).T @ flat(dG)), flat(dG).sum(axis=0)
        dXn = r16(dU @ inp["W1"].T + dG @ inp["Wg"].T)
    else:
        dU = r16(dH * om.gelu_grad(U))
        dXn = r16(dU @ inp["W1"].T)
    out["dW1"], out["db1"] = r16(flat(Xn).T @ flat(dU)), flat(dU).sum(axis=0)
    out["dgamma"] = flat(dXn * xhat).sum(axis=0)
    if cfg.norm == "layernorm":
        out["dbeta"] = flat(dXn).sum(axis=0)
    gg = dXn * inp["gamma"]
    c2 = (gg * xhat).mean(axis=-1, keepdims=True)
    dX = rstd * (gg - (gg.mean(axis=-1, keepdims=True) if cfg.norm == "layernorm" else 0.0) - xhat * c2)
    if cfg.residual:
        dX = dX + dY
    out["dX"] = r16(dX)
    return out


def floor_figures_mlp(cfg, inp, ref):
    """As floor_figures, for the feed-forward block; ``ref``: the oracle's outputs by name."""
    fig = {}
    for name, got in emulate_mlp(cfg, inp).items():
        if not cfg.has_bias and name in ("db1", "dbg", "db2"):
            continue
        r = ref[name]
        e = np.abs(got - r)
        fig[name] = dict(max_abs=float(e.max()),
                         worst_over_bound=float(e.max() / (BF16_ATOL + BF16_RTOL * np.abs(r).max())),
                         fro=float(np.linalg.norm(got - r) / (np.linalg.norm(r) + 1e-300)),
                         viol=float((e > BF16_ATOL + BF16_RTOL * np.abs(r)).mean()),
                         numel=int(r.size))
    return fig
