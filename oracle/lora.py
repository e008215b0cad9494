"""CPU float64 oracle for the attention layer with low-rank adapters on the Q, K and V projections.

TEST INFRASTRUCTURE ONLY.  The paper's fine-tuning setting (its motivating example) is a frozen layer whose
projections carry trainable rank-r adapters: Q = Xn Wq + (Xn Aq) Bq, and likewise for K and V, with Aq: [d_model, r],
Bq: [r, d_q].  (A scale alpha / r, if any, is folded into B by the caller.)  Only the adapters and the layer input
receive gradients:

  forward    T* = Xn A*;  Q = Xn Wq + bq + Tq Bq;  K, V likewise;  then the layer of oracle/layer.py unchanged
  backward   dQ, dK, dV as in oracle/layer.py;
             dB* = T*^T d*            (token-axis reduction, rank rows)
             dT* = d* B*^T;  dA* = Xn^T dT*      (token-axis reduction, rank columns)
             dXn = dQ Wq^T + dK Wk^T + dV Wv^T + dTq Aq^T + dTk Ak^T + dTv Av^T;  dX from the norm's backward

Because Xn (W + A B) = Xn W + (Xn A) B exactly, the forward is the base layer evaluated with W + A B, and by the
chain rule through W_eff = W + A B the adapter gradients are dA = dW_eff B^T and dB = A^T dW_eff, which equal the
expressions above term by term (Xn^T d* B^T and A^T Xn^T d*).  This module uses that form on top of
oracle/layer.py and is pinned by finite differences taken directly in A and B (tests/test_oracle_lora_pins.py),
and by the explicit expressions above.
"""
from __future__ import annotations

from . import layer as base


def effective(inp):
    return {k: inp["W" + k] + inp["A" + k] @ inp["B" + k] for k in ("q", "k", "v")}


def lora_fwd_bwd(cfg, inp):
    """inp: the layer's inputs plus Aq, Ak, Av [d_model, r] and Bq [r, d_q], Bk, Bv [r, d_kv].
    Returns Y, saved and the gradients dX, dAq, dAk, dAv, dBq, dBk, dBv (plus the base layer's intermediates)."""
    w = effective(inp)
    Y, saved = base.layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], w["q"], w["k"], w["v"], inp["Wo"],
                              inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    g = base.layer_bwd(cfg, inp["dY"], inp["X"], inp["gamma"], w["q"], w["k"], w["v"], inp["Wo"], saved)
    out = dict(dX=g["dX"], dQ=g["dQ"], dK=g["dK"], dV=g["dV"], dXn=g["dXn"], dA=g["dA"], D=g["D"])
    for k in ("q", "k", "v"):
        out["dA" + k] = g["dW" + k] @ inp["B" + k].T
        out["dB" + k] = inp["A" + k].T @ g["dW" + k]
    return Y, saved, out
