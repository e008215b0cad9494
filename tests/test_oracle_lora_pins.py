"""Pins for the adapter oracle (oracle/lora.py): finite differences taken directly in A and B and in X, the explicit
low-rank expressions, and the special cases B = 0 and A B = a known matrix."""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, make_lora_inputs
from oracle import layer as base
from oracle import lora as orc


def tiny(norm="layernorm", causal=True, hq=4, hkv=2, bias=True, residual=False):
    return LayerConfig("tiny", 2, 6, 12, hq, hkv, 3, "fp32", norm, causal, bias, residual, 1e-5, 17, 0.3)


def loss(cfg, inp):
    w = orc.effective(inp)
    Y, _ = base.layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], w["q"], w["k"], w["v"], inp["Wo"], inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    return float((Y * inp["dY"]).sum())


@pytest.mark.parametrize("kw", [dict(), dict(norm="rmsnorm", causal=False, hq=2, hkv=2, bias=False, residual=True)])
def test_finite_differences_in_the_adapters_and_the_input(kw):
    cfg = tiny(**kw)
    inp = make_lora_inputs(cfg, 3, affine_noise=True, a_std=0.4, b_std=0.4)
    _, _, g = orc.lora_fwd_bwd(cfg, inp)
    h = 1e-6
    for pname, gname in [("X", "dX")] + [(f"{m}{k}", f"d{m}{k}") for m in "AB" for k in "qkv"]:
        flat, got = inp[pname].reshape(-1), g[gname].reshape(-1)
        scale = np.abs(got).max() + 1e-3
        for i in range(flat.size):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(cfg, inp)
            flat[i] = keep - h
            lm = loss(cfg, inp)
            flat[i] = keep
            assert abs((lp - lm) / (2 * h) - got[i]) <= 3e-6 * scale, (pname, i)


def test_explicit_low_rank_expressions():
    # Q = Xn Wq + (Xn Aq) Bq;  dB = (Xn A)^T d*;  dA = Xn^T (d* B^T);  dXn carries the adapters' terms
    cfg = tiny()
    inp = make_lora_inputs(cfg, 3, affine_noise=True, a_std=0.4, b_std=0.4)
    _, saved, g = orc.lora_fwd_bwd(cfg, inp)
    flat = lambda t: t.reshape(-1, t.shape[-1])
    Xn = saved["Xn"]
    assert np.abs(saved["Q"] - (Xn @ inp["Wq"] + inp["bq"] + (Xn @ inp["Aq"]) @ inp["Bq"])).max() < 1e-12
    for k, d in (("q", "dQ"), ("k", "dK"), ("v", "dV")):
        T = flat(Xn) @ inp["A" + k]
        assert np.abs(g["dB" + k] - T.T @ flat(g[d])).max() < 1e-11
        assert np.abs(g["dA" + k] - flat(Xn).T @ (flat(g[d]) @ inp["B" + k].T)).max() < 1e-11
    dxn = sum(g[d] @ inp["W" + k].T + (g[d] @ inp["B" + k].T) @ inp["A" + k].T for k, d in (("q", "dQ"), ("k", "dK"), ("v", "dV")))
    assert np.abs(g["dXn"] - dxn).max() < 1e-11


def test_zero_b_is_the_base_layer_and_gives_zero_gradient_in_a():
    cfg = tiny(norm="rmsnorm", bias=False)
    inp = make_lora_inputs(cfg, 2, affine_noise=True)
    for k in "qkv":
        inp["B" + k] = np.zeros_like(inp["B" + k])
    Y, _, g = orc.lora_fwd_bwd(cfg, inp)
    Y0, _, g0 = base.layer_fwd_bwd(cfg, inp)
    assert np.array_equal(Y, Y0) and np.array_equal(g["dX"], g0["dX"])
    for k in "qkv":
        assert np.abs(g["dA" + k]).max() == 0.0
        assert np.abs(g["dB" + k] - inp["A" + k].T @ g0["dW" + k]).max() < 1e-12
