"""Parity of the cross-attention layer (keys and values from a memory sequence of its own length and width) with its
float64 oracle: every output, every gradient including dM, and the intermediates."""
import numpy as np
import pytest

from fbl_inputs import XATTN_CONFIGS, XattnConfig, make_xattn_inputs
from oracle import xattn as orc
from paper_2607_21624_b200 import XattnRunner
from paper_2607_21624_b200.binding import FblError, LayerRunner

from bf16_floor import floor_figures
from util import FP32_REL, bf16_ok, fp32_err, record, report

pytestmark = pytest.mark.gpu


def run_and_compare(cfg, path=0, guard_bytes=0, affine_noise=True):
    inp = make_xattn_inputs(cfg, affine_noise=affine_noise)
    Y, saved, g = orc.xattn_fwd_bwd(cfg, inp)
    ref = dict(g)
    ref["Y"] = Y
    run = XattnRunner(cfg, guard_bytes=guard_bytes)
    run.plan.set_kernel_path(path)
    run.load_inputs(inp)
    run.step()
    assert run.status() == 0
    names = ["Y", "dX", "dM", "dWq", "dWk", "dWv", "dWo", "dgamma"]
    if cfg.norm == "layernorm":
        names.append("dbeta")
    if cfg.has_bias:
        names += ["dbq", "dbk", "dbv", "dbo"]
    inter = dict(Xn=saved["Xn"], Q=saved["Q"], K=saved["K"], V=saved["V"], A=saved["A"], LSE=saved["LSE"], D=g["D"],
                 dA=g["dA"], dQ=g["dQ"], dK=g["dK"], dV=g["dV"], dXn=g["dXn"])
    floors = floor_figures(cfg, inp, ref) if cfg.dtype == "bf16" else {}
    bad, figures = [], {}
    for n in names + list(inter):
        got = run.fetch(n) if n in names else run.saved_view(n)
        want = ref[n] if n in names else inter[n]
        assert got.shape == want.shape, (n, got.shape, want.shape)
        assert np.isfinite(got).all(), n
        if cfg.dtype == "fp32":
            if n == "dbk":
                ok = np.abs(got).max() <= 1e-4 * (np.abs(ref["dbq"]).max() + 1e-6)
                print(f"{n:7s} max|.| {np.abs(got).max():.3e} (exact value 0)")
            else:
                err = fp32_err(got, want)
                ok = err <= FP32_REL
                print(f"{n:7s} fp32 scale-floored rel err {err:.3e}")
        else:
            ok, f, failed = bf16_ok(n, got, want, floors.get(n))
            figures[n] = f
            print(report(n, f, floors.get(n)), "" if ok else f"FAILED {failed}")
        if not ok:
            bad.append(n)
    if guard_bytes:
        assert run.guards_intact() == [], run.guards_intact()
    record(cfg.name, figures, floors)
    assert not bad, bad
    return run


def X(name, b, tq, tk, d, dm, hq, hkv, hd, dtype, norm, bias, res, seed, w=0.02):
    return XattnConfig(name, b, tq, tk, d, dm, hq, hkv, hd, dtype, norm, bias, res, 1e-5, seed, w)


CASES = [
    X("x1", 2, 200, 333, 256, 192, 4, 2, 64, "bf16", "layernorm", True, True, 101),       # ragged both sides, GQA
    X("x2", 3, 130, 77, 256, 256, 4, 4, 64, "bf16", "rmsnorm", False, False, 102),        # memory shorter than one tile
    X("x3", 1, 300, 520, 512, 128, 4, 1, 128, "bf16", "rmsnorm", False, True, 103),       # head_dim 128, MQA, narrow memory
    X("x4", 2, 64, 1, 128, 64, 2, 2, 64, "bf16", "layernorm", True, False, 104),          # one memory token (FFMA attention)
    X("x5", 2, 1, 140, 128, 128, 2, 1, 64, "bf16", "layernorm", True, True, 105),         # one query token
    X("x6", 1, 257, 129, 768, 1024, 12, 12, 64, "bf16", "layernorm", True, True, 106),    # one row past a tile on both sides
    XATTN_CONFIGS["tiny"],
    X("x8", 2, 70, 45, 64, 32, 2, 2, 32, "fp32", "rmsnorm", False, False, 108, 0.1),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("path", [0, 1], ids=["default", "ffma"])
def test_xattn_small(cfg, path):
    run_and_compare(cfg, path=path, guard_bytes=4096)


def test_xattn_whisper_large_shape():
    run = run_and_compare(XATTN_CONFIGS["whisper-large"], affine_noise=False)
    # the tensor-core kernels ran: one grouped projection launch, not three
    run.plan.profile_enable(True)
    run.forward()
    run.torch.cuda.synchronize()
    assert "proj_qkv" in [n for n, _ in run.plan.profile_read()]


def test_plan_kinds_do_not_mix():
    cfg = CASES[0]
    run = XattnRunner(cfg)
    run.load_inputs(make_xattn_inputs(cfg))
    with pytest.raises(FblError):
        LayerRunner.forward(run)                  # fbl_layer_fwd on a cross-attention plan
    with pytest.raises(FblError):
        XattnRunner(X("bad", 1, 64, 64, 128, 100, 2, 2, 64, "bf16", "layernorm", False, False, 1))   # d_mem not whole tiles


def test_back_to_back_steps_are_bit_identical():
    cfg = CASES[0]
    run = XattnRunner(cfg)
    run.load_inputs(make_xattn_inputs(cfg, affine_noise=True))
    run.step()
    first = {n: run.fetch(n) for n in ("Y", "dX", "dM", "dbv", "dWk")}
    run.step()
    assert run.status() == 0
    for n, v in first.items():
        got = run.fetch(n)
        # dQ is summed across key tiles with floating-point atomics, and so are the slices of a sliced weight-gradient
        # product: what depends on them may differ in the last bits.  Y, dK, dV and what follows from them alone
        # (dM, dbv) have a fixed summation order.
        if n in ("dX", "dWk"):
            assert np.abs(got - v).max() <= 2e-2 * np.abs(v).max()
        else:
            assert np.array_equal(got, v), n
