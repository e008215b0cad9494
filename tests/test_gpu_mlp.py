"""Parity of the feed-forward block's CUDA path (through the C ABI) with its float64 oracle on the same seeded inputs."""
import numpy as np
import pytest

from fbl_inputs import MLP_CONFIGS, MlpConfig, make_mlp_inputs
from oracle import mlp as orc
from paper_2607_21624_b200 import MlpRunner

from bf16_floor import floor_figures_mlp
from util import FP32_REL, bf16_ok, fp32_err, record, report

pytestmark = pytest.mark.gpu


def run_and_compare(cfg, affine_noise=True, path=0, guard_bytes=0):
    inp = make_mlp_inputs(cfg, affine_noise=affine_noise)
    Y, saved, g = orc.mlp_fwd_bwd(cfg, inp)
    ref = dict(g)
    ref["Y"] = Y
    floors = floor_figures_mlp(cfg, inp, ref) if cfg.dtype == "bf16" else {}
    run = MlpRunner(cfg, guard_bytes=guard_bytes)
    run.plan.set_kernel_path(path)
    run.load_inputs(inp)
    run.step()
    assert run.status() == 0
    names = ["Y", "dX", "dW1", "dW2", "dgamma"] + (["dWg"] if cfg.gated else [])
    if cfg.norm == "layernorm":
        names.append("dbeta")
    if cfg.has_bias:
        names += ["db1", "db2"] + (["dbg"] if cfg.gated else [])
    inter = {"Xn": saved["Xn"], "U": saved["U"], "H": saved["H"], "dU": g["dU"], "dXn": g["dXn"]}
    if cfg.gated:
        inter.update(G=saved["G"], dG=g["dG"])
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


SMALL = [
    MlpConfig("m1", 2, 200, 256, 512, "bf16", "layernorm", "gelu", True, True, 1e-5, 81, 0.05),
    MlpConfig("m2", 3, 197, 256, 768, "bf16", "rmsnorm", "swiglu", False, False, 1e-5, 82, 0.05),
    MlpConfig("m3", 1, 333, 512, 1024, "bf16", "rmsnorm", "swiglu", True, True, 1e-5, 83, 0.05),
    MlpConfig("m4", 2, 8, 128, 256, "bf16", "layernorm", "gelu", False, True, 1e-5, 84, 0.05),     # FFMA path: too few rows for a tile
    MlpConfig("m5", 1, 64, 64, 128, "fp32", "layernorm", "gelu", True, True, 1e-5, 85, 0.1),
    MlpConfig("m6", 2, 77, 64, 96, "fp32", "rmsnorm", "swiglu", True, False, 1e-5, 86, 0.1),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
@pytest.mark.parametrize("path", [0, 1], ids=["default", "ffma"])
def test_mlp_small(cfg, path):
    run_and_compare(cfg, path=path, guard_bytes=4096)


def test_mlp_sliced_weight_gradient_reductions(monkeypatch):
    monkeypatch.setenv("FBL_KSPLIT_MLP", "3")
    run_and_compare(MlpConfig("m7", 6, 197, 256, 512, "bf16", "layernorm", "swiglu", True, True, 1e-5, 87, 0.05))
    run_and_compare(MlpConfig("m8", 6, 197, 256, 512, "bf16", "rmsnorm", "gelu", False, True, 1e-5, 88, 0.05))


@pytest.mark.parametrize("key", ["matmul-512x2048x8192", "gpt2", "llama1b"])
def test_mlp_full_shapes(key):
    # the paper's MatMul benchmark shapes (forward 512 x 2048 x 8192, backward 512 x 8192 x 2048), a GPT-2-small-shaped
    # and a Llama-3.2-1B-shaped block at full size, with the workloads' own identity affine
    run_and_compare(MLP_CONFIGS[key], affine_noise=False)


def test_mlp_back_to_back_steps_are_identical():
    import torch
    cfg = MlpConfig("m9", 2, 300, 256, 768, "bf16", "layernorm", "swiglu", True, True, 1e-5, 89, 0.05)
    run = MlpRunner(cfg)
    run.load_inputs(make_mlp_inputs(cfg, affine_noise=True))
    run.step()
    torch.cuda.synchronize()
    names = ("Y", "dX", "dW1", "dWg", "dW2", "db1", "dgamma")
    first = {n: run.fetch(n) for n in names}
    for fill in (0xFF, 0x7F):
        run.saved.fill_(fill)
        run.scratch.fill_(fill)
        for _ in range(10):
            run.step()
        torch.cuda.synchronize()
        assert run.status() == 0
        for n in names:
            assert np.array_equal(first[n], run.fetch(n)), (n, hex(fill))
