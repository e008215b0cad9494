"""Pins for the feed-forward oracle (oracle/mlp.py): numerical derivatives, known values of the activations,
closed-form special cases, a scalar-loop forward, and structural properties.  Nothing compares it with itself."""
import math

import numpy as np
import pytest

from fbl_inputs import MlpConfig, make_mlp_inputs
from oracle import mlp as orc


def tiny(act="gelu", norm="layernorm", bias=True, residual=False, B=2, T=5, D=6, F=8, seed=5):
    return MlpConfig("tiny", B, T, D, F, "fp32", norm, act, bias, residual, 1e-5, seed, 0.5)


def loss(cfg, inp):
    Y, _ = orc.mlp_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["W1"], inp["Wg"], inp["W2"], inp["b1"], inp["bg"], inp["b2"])
    return float((Y * inp["dY"]).sum())


@pytest.mark.parametrize("kw", [dict(act="gelu", norm="layernorm", residual=True), dict(act="gelu", norm="rmsnorm", bias=False),
                                dict(act="swiglu", norm="rmsnorm", residual=True), dict(act="swiglu", norm="layernorm", bias=True)])
def test_finite_differences_every_gradient(kw):
    cfg = tiny(**kw)
    inp = make_mlp_inputs(cfg, affine_noise=True)
    _, _, g = orc.mlp_fwd_bwd(cfg, inp)
    names = {"X": "dX", "W1": "dW1", "Wg": "dWg", "W2": "dW2", "gamma": "dgamma", "beta": "dbeta", "b1": "db1",
             "bg": "dbg", "b2": "db2"}
    h = 1e-6
    for pname, gname in names.items():
        if inp[pname] is None:
            continue
        flat, got = inp[pname].reshape(-1), g[gname].reshape(-1)
        scale = np.abs(got).max() + 1e-3
        for i in range(flat.size):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(cfg, inp)
            flat[i] = keep - h
            lm = loss(cfg, inp)
            flat[i] = keep
            assert abs((lp - lm) / (2 * h) - got[i]) <= 2e-6 * scale, (pname, i)


def test_activation_values_and_limits():
    # published values of the tanh form of GELU and of SiLU, and their limits
    assert abs(orc.gelu(np.array(1.0)) - 0.8411919906) < 1e-9
    assert abs(orc.gelu(np.array(-1.0)) + 0.1588080094) < 1e-9
    assert orc.gelu(np.array(0.0)) == 0.0 and abs(orc.gelu(np.array(10.0)) - 10.0) < 1e-12
    assert abs(orc.silu(np.array(1.0)) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(orc.silu(np.array(1.0)) - 0.7310585786) < 1e-9
    # gelu(u) - gelu(-u) = u and silu(g) - silu(-g) = g: exact identities of both forms
    u = np.linspace(-6, 6, 97)
    assert np.abs(orc.gelu(u) - orc.gelu(-u) - u).max() < 1e-14
    assert np.abs(orc.silu(u) - orc.silu(-u) - u).max() < 1e-14
    # the tanh form stays within 5e-4 of the erf definition x Phi(x)
    erf_form = np.array([0.5 * x * (1.0 + math.erf(x / math.sqrt(2.0))) for x in u])
    assert np.abs(orc.gelu(u) - erf_form).max() < 5e-4
    # derivatives against central differences
    h = 1e-6
    assert np.abs((orc.gelu(u + h) - orc.gelu(u - h)) / (2 * h) - orc.gelu_grad(u)).max() < 1e-8
    assert np.abs((orc.silu(u + h) - orc.silu(u - h)) / (2 * h) - orc.silu_grad(u)).max() < 1e-8


def test_scalar_loop_forward():
    # the whole forward in plain Python loops, straight from the definition
    for act in ("gelu", "swiglu"):
        cfg = tiny(act=act, norm="rmsnorm", residual=True, B=1, T=3, D=4, F=5)
        inp = make_mlp_inputs(cfg, affine_noise=True)
        Y, _ = orc.mlp_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["W1"], inp["Wg"], inp["W2"], inp["b1"], inp["bg"], inp["b2"])
        for t in range(cfg.seq):
            x = [float(v) for v in inp["X"][0, t]]
            rstd = 1.0 / math.sqrt(sum(v * v for v in x) / len(x) + cfg.eps)
            xn = [x[d] * rstd * float(inp["gamma"][d]) for d in range(cfg.d_model)]
            h = []
            for f in range(cfg.d_ff):
                u = sum(xn[d] * float(inp["W1"][d, f]) for d in range(cfg.d_model)) + float(inp["b1"][f])
                if act == "swiglu":
                    g = sum(xn[d] * float(inp["Wg"][d, f]) for d in range(cfg.d_model)) + float(inp["bg"][f])
                    h.append(g / (1.0 + math.exp(-g)) * u)
                else:
                    h.append(0.5 * u * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (u + 0.044715 * u ** 3))))
            for d in range(cfg.d_model):
                y = sum(h[f] * float(inp["W2"][f, d]) for f in range(cfg.d_ff)) + float(inp["b2"][d]) + x[d]
                assert abs(y - Y[0, t, d]) < 1e-12


def test_constant_gate_makes_the_block_linear():
    # Wg = 0, bg = c: silu(c) is one constant, so Y = silu(c) (Xn W1 + b1) W2 + b2 and dWg = 0-gate algebra holds:
    # dG = dH * U * silu'(c)
    cfg = tiny(act="swiglu", norm="layernorm")
    inp = make_mlp_inputs(cfg, affine_noise=True)
    inp["Wg"] = np.zeros_like(inp["Wg"])
    inp["bg"] = np.full_like(inp["bg"], 0.7)
    Y, saved, g = orc.mlp_fwd_bwd(cfg, inp)
    mu = inp["X"].mean(-1, keepdims=True)
    xn = (inp["X"] - mu) / np.sqrt(((inp["X"] - mu) ** 2).mean(-1, keepdims=True) + cfg.eps) * inp["gamma"] + inp["beta"]
    sc = 0.7 / (1.0 + math.exp(-0.7))
    assert np.abs(Y - (sc * (xn @ inp["W1"] + inp["b1"]) @ inp["W2"] + inp["b2"])).max() < 1e-12
    # the value path is linear in W1: its gradient is Xn^T (dY W2^T) silu(c)
    flat = lambda t: t.reshape(-1, t.shape[-1])
    assert np.abs(g["dW1"] - sc * flat(xn).T @ (flat(inp["dY"]) @ inp["W2"].T)).max() < 1e-11


def test_batch_additivity_and_linearity():
    cfg = tiny(act="swiglu", norm="rmsnorm", residual=True, B=3)
    inp = make_mlp_inputs(cfg, affine_noise=True)
    _, _, g = orc.mlp_fwd_bwd(cfg, inp)
    acc = None
    for b in range(cfg.batch):
        one = dict(inp)
        one["X"], one["dY"] = inp["X"][b:b + 1], inp["dY"][b:b + 1]
        from fbl_inputs import scaled_config
        _, _, gb = orc.mlp_fwd_bwd(scaled_config(cfg, batch=1), one)
        assert np.abs(gb["dX"][0] - g["dX"][b]).max() < 1e-12
        acc = gb if acc is None else {k: acc[k] + gb[k] for k in ("dW1", "dWg", "dW2", "dgamma")}
    for k in ("dW1", "dWg", "dW2", "dgamma"):
        assert np.abs(acc[k] - g[k]).max() < 1e-11
    two = dict(inp)
    two["dY"] = 2.5 * inp["dY"]
    _, _, g2 = orc.mlp_fwd_bwd(cfg, two)
    for k in ("dX", "dW1", "dWg", "dW2", "dgamma"):
        assert np.abs(g2[k] - 2.5 * g[k]).max() < 1e-10 * (1 + np.abs(g[k]).max())


def test_identity_weights_and_large_inputs():
    # d_ff = d_model, W1 = W2 = I, no biases, gamma = 1: gelu is the identity on large positive values and zero on
    # large negative ones, so Y = relu(Xn) there
    cfg = MlpConfig("id", 1, 4, 6, 6, "fp32", "rmsnorm", "gelu", False, False, 0.0, 3, 1.0)
    inp = make_mlp_inputs(cfg)
    inp["W1"], inp["W2"] = np.eye(6), np.eye(6)
    inp["X"] = 40.0 * np.sign(inp["X"]) * (1.0 + np.abs(inp["X"]))
    Y, saved = orc.mlp_fwd(cfg, inp["X"], 40.0 * np.ones(6), None, inp["W1"], None, inp["W2"])
    assert np.abs(Y - np.maximum(saved["Xn"], 0.0)).max() < 1e-9
