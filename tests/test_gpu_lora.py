"""Parity of the adapter path (frozen base weights, rank-r adapters on Q, K, V) with its float64 oracle."""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, get_config, make_lora_inputs
from oracle import lora as orc
from paper_2607_21624_b200 import LoraRunner

from util import FP32_REL, bf16_ok, fp32_err, record, report

pytestmark = pytest.mark.gpu


def run_and_compare(cfg, rank, path=0, guard_bytes=0, affine_noise=True):
    inp = make_lora_inputs(cfg, rank, affine_noise=affine_noise)
    Y, saved, g = orc.lora_fwd_bwd(cfg, inp)
    ref = dict(g)
    ref["Y"] = Y
    run = LoraRunner(cfg, rank, guard_bytes=guard_bytes)
    run.plan.set_kernel_path(path)
    run.load_inputs(inp)
    run.step()
    assert run.status() == 0
    names = ["Y", "dX"] + [f"d{m}{k}" for m in "AB" for k in "qkv"]
    inter = dict(Q=saved["Q"], K=saved["K"], V=saved["V"], A=saved["A"], LSE=saved["LSE"], dQ=g["dQ"], dK=g["dK"], dV=g["dV"], dXn=g["dXn"])
    bad, figures = [], {}
    for n in names + list(inter):
        got = run.fetch(n) if n in names else run.saved_view(n)
        want = ref[n] if n in names else inter[n]
        assert np.isfinite(got).all(), n
        if cfg.dtype == "fp32":
            err = fp32_err(got, want)
            ok = err <= FP32_REL
            print(f"{n:7s} fp32 scale-floored rel err {err:.3e}")
        else:
            ok, f, failed = bf16_ok(n, got, want)
            figures[n] = f
            print(report(n, f), "" if ok else f"FAILED {failed}")
        if not ok:
            bad.append(n)
    if guard_bytes:
        assert run.guards_intact() == [], run.guards_intact()
    record(cfg.name + f"-lora{rank}", figures, {})
    assert not bad, bad
    return run


CASES = [
    (LayerConfig("l1", 2, 200, 256, 4, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 91, 0.02), 8),
    (LayerConfig("l2", 3, 197, 256, 4, 4, 64, "bf16", "rmsnorm", False, False, False, 1e-5, 92, 0.02), 16),
    (LayerConfig("l3", 1, 333, 512, 4, 1, 128, "bf16", "rmsnorm", True, False, True, 1e-5, 93, 0.02), 64),
    (LayerConfig("l4", 2, 8, 128, 2, 2, 64, "bf16", "layernorm", True, True, False, 1e-5, 94, 0.02), 4),      # FFMA path
    (LayerConfig("l5", 1, 64, 64, 2, 2, 32, "fp32", "layernorm", True, False, False, 1e-5, 95, 0.1), 8),
    (LayerConfig("l6", 2, 77, 128, 2, 1, 64, "fp32", "rmsnorm", False, True, True, 1e-5, 96, 0.1), 5),
    # with the rotary embedding between the adapted projections and the scores (the Llama fine-tuning arrangement)
    (LayerConfig("l8", 2, 300, 256, 4, 2, 64, "bf16", "rmsnorm", True, False, True, 1e-5, 98, 0.02, 0.0, 10000.0), 16),
]


@pytest.mark.parametrize("cfg,rank", CASES, ids=lambda c: getattr(c, "name", str(c)))
@pytest.mark.parametrize("path", [0, 1], ids=["default", "ffma"])
def test_lora_small(cfg, rank, path):
    run_and_compare(cfg, rank, path=path, guard_bytes=4096)


@pytest.mark.parametrize("i,rank", [(2, 16), (4, 16)])
def test_lora_full_workloads(i, rank):
    # the GPT-2-small-shaped and the Llama-3.2-1B-shaped layer with rank-16 adapters (the paper fine-tunes with LoRA)
    run_and_compare(get_config(i), rank, affine_noise=False)


def test_zero_b_reproduces_the_base_layer_bit_for_bit():
    # with B = 0 the adapters add exact zeros to Q, K, V: Y equals the base layer's Y bit for bit
    from paper_2607_21624_b200 import LayerRunner
    cfg = LayerConfig("l7", 2, 300, 256, 4, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 97, 0.02)
    inp = make_lora_inputs(cfg, 8, affine_noise=True)
    for k in "qkv":
        inp["B" + k] = np.zeros_like(inp["B" + k])
    a = LoraRunner(cfg, 8)
    a.load_inputs(inp)
    a.step()
    b = LayerRunner(cfg)
    b.load_inputs(inp)
    b.step()
    assert a.status() == 0 and b.status() == 0
    assert np.array_equal(a.fetch("Y"), b.fetch("Y"))
    assert np.abs(a.fetch("dX") - b.fetch("dX")).max() <= 2e-2 * np.abs(b.fetch("dX")).max()
    assert np.abs(a.fetch("dAq")).max() == 0.0
