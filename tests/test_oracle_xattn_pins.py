"""Pins for the cross-attention oracle (oracle/xattn.py): finite differences of every gradient (the memory's
included), a scalar-loop attention over two lengths, closed forms, symmetries, and the self-attention oracle on the
case where the two layers coincide."""
import math

import numpy as np
import pytest

from fbl_inputs import LayerConfig, XattnConfig, make_xattn_inputs
from oracle import layer as base
from oracle import xattn as orc


def tiny(norm="layernorm", hq=4, hkv=2, bias=True, residual=False, tq=5, tk=7, b=2, d=12, dm=10):
    return XattnConfig("tiny", b, tq, tk, d, dm, hq, hkv, 3, "fp32", norm, bias, residual, 1e-5, 31, 0.3)


def unrounded(cfg):
    inp = make_xattn_inputs(cfg, affine_noise=True)
    return {k: (None if v is None else v.copy()) for k, v in inp.items()}


def loss(cfg, inp):
    Y, _ = orc.xattn_fwd(cfg, inp["X"], inp["M"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                         inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    return float((Y * inp["dY"]).sum())


@pytest.mark.parametrize("kw", [dict(), dict(norm="rmsnorm", hq=2, hkv=2, bias=False, residual=True, tq=6, tk=3)])
def test_finite_differences_of_every_gradient(kw):
    cfg = tiny(**kw)
    inp = unrounded(cfg)
    _, _, g = orc.xattn_fwd_bwd(cfg, inp)
    names = [("X", "dX"), ("M", "dM"), ("Wq", "dWq"), ("Wk", "dWk"), ("Wv", "dWv"), ("Wo", "dWo"), ("gamma", "dgamma")]
    if cfg.norm == "layernorm":
        names.append(("beta", "dbeta"))
    if cfg.has_bias:
        names += [("bq", "dbq"), ("bk", "dbk"), ("bv", "dbv"), ("bo", "dbo")]
    h = 1e-6
    for pname, gname in names:
        flat, got = inp[pname].reshape(-1), g[gname].reshape(-1)
        assert flat.size == got.size, pname
        scale = np.abs(got).max() + 1e-3
        for i in range(0, flat.size, max(1, flat.size // 60)):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(cfg, inp)
            flat[i] = keep - h
            lm = loss(cfg, inp)
            flat[i] = keep
            assert abs((lp - lm) / (2 * h) - got[i]) <= 5e-6 * scale, (pname, i)


def test_bk_gradient_is_zero_and_bv_gradient_is_the_column_sum_of_dA_heads():
    # a constant added to every key shifts all scores of a row alike: softmax does not see it.  Each row of P sums to
    # one, so dbv[g] = sum over tokens and over the group's heads of dO
    cfg = tiny()
    inp = unrounded(cfg)
    _, _, g = orc.xattn_fwd_bwd(cfg, inp)
    assert np.abs(g["dbk"]).max() < 1e-12
    hd, G = cfg.head_dim, cfg.group
    want = np.zeros(cfg.d_kv)
    for h in range(cfg.n_q_heads):
        want[(h // G) * hd:(h // G + 1) * hd] += g["dA"][:, :, h * hd:(h + 1) * hd].sum(axis=(0, 1))
    assert np.abs(g["dbv"] - want).max() < 1e-12


def test_scalar_loop_attention_over_two_lengths():
    cfg = tiny(tq=4, tk=9, b=1)
    inp = unrounded(cfg)
    _, saved = orc.xattn_fwd(cfg, inp["X"], inp["M"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                             inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    Q, K, V, A, LSE = saved["Q"][0], saved["K"][0], saved["V"][0], saved["A"][0], saved["LSE"][0]
    hd = cfg.head_dim
    for h in range(cfg.n_q_heads):
        g = h // cfg.group
        for i in range(cfg.seq):
            w = []
            for j in range(cfg.seq_kv):
                s = 0.0
                for d in range(hd):
                    s += Q[i, h * hd + d] * K[j, g * hd + d]
                w.append(math.exp(cfg.scale * s))
            tot = sum(w)
            assert abs(math.log(tot) - LSE[h, i]) < 1e-12
            for d in range(hd):
                o = sum(w[j] / tot * V[j, g * hd + d] for j in range(cfg.seq_kv))
                assert abs(o - A[i, h * hd + d]) < 1e-12


def test_one_memory_token_closed_form():
    # Tk = 1: P = 1, every query row of head h outputs V[0, g]; the scores carry no gradient
    cfg = tiny(tk=1, residual=True)
    inp = unrounded(cfg)
    Y, saved, g = orc.xattn_fwd_bwd(cfg, inp)
    hd = cfg.head_dim
    for h in range(cfg.n_q_heads):
        gk = h // cfg.group
        want = np.broadcast_to(saved["V"][:, 0:1, gk * hd:(gk + 1) * hd], (cfg.batch, cfg.seq, hd))
        assert np.abs(saved["A"][:, :, h * hd:(h + 1) * hd] - want).max() < 1e-13
    assert np.abs(g["dQ"]).max() < 1e-13 and np.abs(g["dK"]).max() < 1e-13
    assert np.abs(g["dWq"]).max() < 1e-13 and np.abs(g["dWk"]).max() < 1e-13
    assert np.abs(g["dX"] - inp["dY"]).max() < 1e-13            # only the residual path reaches X
    assert np.abs(g["dM"] - g["dV"] @ inp["Wv"].T).max() < 1e-13


def test_memory_order_does_not_matter():
    cfg = tiny()
    inp = unrounded(cfg)
    Y, _, g = orc.xattn_fwd_bwd(cfg, inp)
    perm = np.array([3, 0, 6, 1, 5, 2, 4])
    inp2 = dict(inp)
    inp2["M"] = inp["M"][:, perm]
    Y2, _, g2 = orc.xattn_fwd_bwd(cfg, inp2)
    assert np.abs(Y - Y2).max() < 1e-12
    for k in ("dX", "dWq", "dWk", "dWv", "dWo", "dgamma", "dbeta", "dbq", "dbv", "dbo"):
        assert np.abs(g[k] - g2[k]).max() < 1e-11, k
    assert np.abs(g["dM"][:, perm] - g2["dM"]).max() < 1e-12


def test_coincides_with_self_attention_when_the_memory_is_the_normalised_input():
    # non-causal self-attention computes K, V from Xn; cross-attention given M = Xn computes the same Y and the same
    # weight gradients, and the self-attention layer's dXn is the cross layer's dXn + dM
    cfg = tiny(tq=6, tk=6, dm=12)
    inp = unrounded(cfg)
    scfg = LayerConfig("self", cfg.batch, cfg.seq, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, "fp32", cfg.norm,
                       False, True, cfg.residual, cfg.eps, 0, 0.3)
    Ys, saved_s = base.layer_fwd(scfg, inp["X"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                                 inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    gs = base.layer_bwd(scfg, inp["dY"], inp["X"], inp["gamma"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"], saved_s)
    inp2 = dict(inp)
    inp2["M"] = saved_s["Xn"]
    Yc, _, gc = orc.xattn_fwd_bwd(cfg, inp2)
    assert np.abs(Ys - Yc).max() < 1e-12
    for k in ("dWq", "dWk", "dWv", "dWo", "dbq", "dbv", "dbo", "dQ", "dK", "dV"):
        assert np.abs(gs[k] - gc[k]).max() < 1e-11, k
    assert np.abs(gs["dXn"] - (gc["dXn"] + gc["dM"])).max() < 1e-11


def test_batch_additivity_of_the_weight_gradients():
    cfg = tiny(b=3)
    inp = unrounded(cfg)
    _, _, g = orc.xattn_fwd_bwd(cfg, inp)
    acc = {k: 0.0 for k in ("dWq", "dWk", "dWv", "dWo", "dgamma")}
    one = tiny(b=1)
    for b in range(3):
        sub = dict(inp)
        for k in ("X", "M", "dY"):
            sub[k] = inp[k][b:b + 1]
        _, _, gb = orc.xattn_fwd_bwd(one, sub)
        for k in acc:
            acc[k] = acc[k] + gb[k]
        assert np.abs(gb["dX"][0] - g["dX"][b]).max() < 1e-12 and np.abs(gb["dM"][0] - g["dM"][b]).max() < 1e-12
    for k in acc:
        assert np.abs(acc[k] - g[k]).max() < 1e-11, k
