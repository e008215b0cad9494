"""CPU float64 oracle for the feed-forward half of a transformer block, forward and backward.

TEST INFRASTRUCTURE ONLY: the plain definition of what the CUDA path's fbl_mlp_fwd / fbl_mlp_bwd must compute;
it shares no code with that path and is imported only by tests and the benchmark's CPU-baseline leg.

What it follows.  The paper treats MatMul as the reduce-axis-conflict operator (its operator classification: the
forward reduces over d_in, dW = X^T dY reduces over the tokens, dX = dY W^T over d_out) and benchmarks exactly the
two products of an up projection (its R-Tile ablation: forward (512, 2048, 8192), backward (512, 8192, 2048)).
The block around them is the textbook pre-norm feed-forward block, written out step by step:

forward
  1. Xn = norm(X)                      (LayerNorm or RMSNorm, as in oracle/layer.py)
  2. U = Xn W1 + b1                    W1: [d_model, d_ff]
     gated ("swiglu"): G = Xn Wg + bg  Wg: [d_model, d_ff]
  3. H = gelu(U)                       gelu(u) = u/2 (1 + tanh(sqrt(2/pi) (u + 0.044715 u^3)))     ("gelu")
     H = silu(G) * U                   silu(g) = g / (1 + exp(-g))                                  ("swiglu")
  4. Y = H W2 + b2 (+ X)               W2: [d_ff, d_model]

backward, given dY
  5. dW2 = H^T dY, db2 = sum_tokens dY, dH = dY W2^T
  6. gelu:   dU = dH * gelu'(U)
     swiglu: dU = dH * silu(G), dG = dH * U * silu'(G),  silu'(g) = s (1 + g (1 - s)), s = 1 / (1 + exp(-g))
  7. dW1 = Xn^T dU, db1 = sum_tokens dU (same for Wg, bg with dG); dXn = dU W1^T (+ dG Wg^T)
  8. dgamma, dbeta, dX from the norm's backward (+ dY if residual)

numpy's matmul is the only library step; nothing is blocked, fused or reordered.
Pins: tests/test_oracle_mlp_pins.py.
"""
from __future__ import annotations

import numpy as np

from .layer import norm_fwd

K0 = np.sqrt(2.0 / np.pi)
K1 = 0.044715


def gelu(u):
    return 0.5 * u * (1.0 + np.tanh(K0 * (u + K1 * u ** 3)))


def gelu_grad(u):
    t = np.tanh(K0 * (u + K1 * u ** 3))
    return 0.5 * (1.0 + t) + 0.5 * u * (1.0 - t * t) * K0 * (1.0 + 3.0 * K1 * u * u)


def sigmoid(g):
    return 1.0 / (1.0 + np.exp(-g))


def silu(g):
    return g * sigmoid(g)


def silu_grad(g):
    s = sigmoid(g)
    return s * (1.0 + g * (1.0 - s))


def mlp_fwd(cfg, X, gamma, beta, W1, Wg, W2, b1=None, bg=None, b2=None):
    z = lambda b: b if b is not None else 0.0
    Xn, xhat, rstd, mu = norm_fwd(X, gamma, beta, cfg.eps, cfg.norm)
    U = Xn @ W1 + z(b1)
    if cfg.act == "swiglu":
        G = Xn @ Wg + z(bg)
        H = silu(G) * U
    elif cfg.act == "gelu":
        G = None
        H = gelu(U)
    else:
        raise ValueError(cfg.act)
    Y = H @ W2 + z(b2)
    if cfg.residual:
        Y = Y + X
    return Y, dict(Xn=Xn, xhat=xhat, rstd=rstd, mu=mu, U=U, G=G, H=H)


def mlp_bwd(cfg, dY, X, gamma, W1, Wg, W2, saved):
    B, T, D = X.shape
    flat = lambda t: t.reshape(B * T, -1)
    Xn, xhat, rstd, U, G, H = (saved[k] for k in ("Xn", "xhat", "rstd", "U", "G", "H"))
    dW2 = flat(H).T @ flat(dY)
    db2 = flat(dY).sum(axis=0)
    dH = dY @ W2.T
    out = {}
    if cfg.act == "swiglu":
        dU = dH * silu(G)
        dG = dH * U * silu_grad(G)
        out.update(dWg=flat(Xn).T @ flat(dG), dbg=flat(dG).sum(axis=0), dG=dG)
        dXn = dU @ W1.T + dG @ Wg.T
    else:
        dU = dH * gelu_grad(U)
        dXn = dU @ W1.T
    out.update(dW1=flat(Xn).T @ flat(dU), db1=flat(dU).sum(axis=0), dW2=dW2, db2=db2, dH=dH, dU=dU, dXn=dXn)
    out["dgamma"] = flat(dXn * xhat).sum(axis=0)
    if cfg.norm == "layernorm":
        out["dbeta"] = flat(dXn).sum(axis=0)
    gg = dXn * gamma
    c2 = (gg * xhat).mean(axis=-1, keepdims=True)
    if cfg.norm == "layernorm":
        dX = rstd * (gg - gg.mean(axis=-1, keepdims=True) - xhat * c2)
    else:
        dX = rstd * (gg - xhat * c2)
    if cfg.residual:
        dX = dX + dY
    out["dX"] = dX
    return out


def mlp_fwd_bwd(cfg, inp):
    Y, saved = mlp_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["W1"], inp["Wg"], inp["W2"],
                       inp["b1"], inp["bg"], inp["b2"])
    grads = mlp_bwd(cfg, inp["dY"], inp["X"], inp["gamma"], inp["W1"], inp["Wg"], inp["W2"], saved)
    return Y, saved, grads
