"""The rounding floor of a bf16 implementation (tests/bf16_floor.py), on the CPU: the figures the GPU parity
tolerances are derived from.  Uses only the oracle, numpy and the shared input generator."""
import numpy as np

from fbl_inputs import get_config, make_inputs, scaled_config

from bf16_floor import emulate, floor_figures, r16


def _show(tag, fig):
    for k, v in fig.items():
        print(f"{tag} {k:7s} max|e|={v['max_abs']:.3e} worst/bound={v['worst_over_bound']:.3f} fro={v['fro']:.3e} viol={v['viol']:.2e}")


def test_rounding_is_round_to_nearest_even_on_8_bit_mantissas():
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: ties go to the even mantissa; 1 + 3 * 2^-9 rounds up
    assert r16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert r16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert r16(np.array([1.0 + 3 * 2.0 ** -9]))[0] == 1.0 + 2.0 ** -7
    x = np.random.default_rng(0).normal(size=1000)
    assert np.abs(r16(x) - x).max() <= 2.0 ** -9 * np.abs(x).max() * 1.0001


def test_floor_of_workload_2():
    # GPT-2-small shape at full size: Y and dX meet the element-wise tolerance everywhere even after rounding every
    # intermediate, the reductions do not (their small elements carry noise on the tensor's scale), nothing comes
    # near the tensor-scale bound, and the identically-zero dbk comes out at 0.85e-2: inside 1e-2, with little room
    cfg = get_config(2)
    fig = floor_figures(cfg, make_inputs(cfg))
    _show("cfg2", fig)
    assert fig["Y"]["viol"] == 0.0 and fig["dX"]["viol"] == 0.0
    for name, v in fig.items():
        if name == "dbk":
            continue
        assert v["worst_over_bound"] < 0.3, name
        assert v["fro"] < 6e-3, name
    assert 1e-2 < fig["dWv"]["viol"] < 4e-2 and 1e-2 < fig["dbeta"]["viol"] < 4e-2
    assert 5e-3 < fig["dbk"]["max_abs"] < 1e-2


def test_floor_of_reduced_workloads_3_and_4():
    c3 = scaled_config(get_config(3), batch=8)
    f3 = floor_figures(c3, make_inputs(c3))
    _show("cfg3/B=8", f3)
    assert f3["Y"]["viol"] == 0.0 and f3["dX"]["viol"] == 0.0
    assert max(v["fro"] for v in f3.values()) < 6e-3
    c4 = scaled_config(get_config(4), batch=1, seq=512)
    f4 = floor_figures(c4, make_inputs(c4))
    _show("cfg4/B=1,T=512", f4)
    assert max(v["fro"] for v in f4.values()) < 6.5e-3
    assert max(v["worst_over_bound"] for v in f4.values()) < 0.5
    # wide layers (D = 2048): a few per cent of the weight gradients' elements miss the element-wise form already
    assert f4["dWk"]["viol"] > 1e-2


def test_zero_bias_gradient_noise_grows_with_tokens_and_group():
    # dbk is zero in exact arithmetic; the floor's dbk is pure rounding noise of bf16 dS and grows roughly like the
    # square root of (tokens x query heads per key head): the reason a fixed 1e-2 cannot hold for every layer
    from fbl_inputs import LayerConfig
    small = LayerConfig("n1", 2, 256, 256, 4, 4, 64, "bf16", "layernorm", False, True, False, 1e-5, 70, 0.02)
    large = LayerConfig("n2", 8, 512, 256, 8, 2, 64, "bf16", "layernorm", False, True, False, 1e-5, 70, 0.02)
    a = np.abs(emulate(small, make_inputs(small, affine_noise=True))["dbk"]).max()
    b = np.abs(emulate(large, make_inputs(large, affine_noise=True))["dbk"]).max()
    print(f"max|dbk| floor: {a:.3e} (512 tokens, G=1) -> {b:.3e} (4096 tokens, G=4)")
    assert b > 2.0 * a


def test_floor_of_a_cross_attention_layer():
    # the memory is an input, so K, V and dM see one rounding fewer than their self-attention counterparts; the
    # floor's figures stay in the same band, and dM (a token tensor) meets the element-wise form everywhere
    from fbl_inputs import XattnConfig, make_xattn_inputs
    cfg = XattnConfig("xf", 2, 200, 333, 256, 192, 4, 2, 64, "bf16", "layernorm", True, True, 1e-5, 101, 0.02)
    fig = floor_figures(cfg, make_xattn_inputs(cfg, affine_noise=True))
    _show("xattn", fig)
    assert "dM" in fig and fig["dM"]["viol"] == 0.0 and fig["Y"]["viol"] == 0.0 and fig["dX"]["viol"] == 0.0
    for name, v in fig.items():
        if name != "dbk":
            assert v["fro"] < 6e-3 and v["worst_over_bound"] < 0.3, name
