"""Parity of the CUDA path (through the C ABI) with the float64 oracle on the same seeded inputs."""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, get_config, make_inputs, scaled_config
from oracle import layer as orc
from paper_2607_21624_b200 import LayerRunner

from bf16_floor import floor_figures
from util import FP32_REL, bf16_ok, fp32_err, record, report

pytestmark = pytest.mark.gpu

MATS = ("Y", "dX", "dWq", "dWk", "dWv", "dWo")
# forward tensors the backward reuses, and the backward's own intermediates, read back through fbl_workspace_offset
INTERMEDIATES = ("Xn", "Q", "K", "V", "A", "LSE", "dA", "D", "dQ", "dK", "dV", "dXn")


def run_and_compare(cfg, affine_noise=False, path=0, guard_bytes=0, intermediates=True):
    inp = make_inputs(cfg, affine_noise=affine_noise)
    Y, saved, g = orc.layer_fwd_bwd(cfg, inp)
    ref = dict(g)
    ref["Y"] = Y
    # rounding floor of any bf16 implementation on this very layer: the yardstick of the element-wise criterion
    floors = floor_figures(cfg, inp, ref) if cfg.dtype == "bf16" else {}
    run = LayerRunner(cfg, guard_bytes=guard_bytes)
    run.plan.set_kernel_path(path)
    run.load_inputs(inp)
    run.step()
    assert run.status() == 0
    names = list(MATS) + ["dgamma"]
    if cfg.norm == "layernorm":
        names.append("dbeta")
    if cfg.has_bias:
        names += ["dbq", "dbk", "dbv", "dbo"]
    bad = []
    figures = {}
    for n in names:
        got = run.fetch(n)
        assert np.isfinite(got).all(), n
        if cfg.dtype == "fp32":
            # dbk is identically zero in exact arithmetic (and with one token per sequence so are dWq, dWk): such a
            # tensor has no scale of its own and is judged against the scale of its value-path sibling
            sibling = {"dbk": "dbv", "dWq": "dWv", "dWk": "dWv", "dbq": "dbv"}.get(n)
            zero_ref = sibling is not None and ((n == "dbk" and not cfg.rope_base > 0) or np.abs(ref[n]).max() < 1e-12 * np.abs(ref[sibling]).max())
            err = float(np.abs(got).max() / np.abs(ref[sibling]).max()) if zero_ref else fp32_err(got, ref[n])
            ok = err <= FP32_REL
            print(f"{n:7s} fp32 scale-floored rel err {err:.3e}")
        else:
            ok, f, failed = bf16_ok(n, got, ref[n], floors.get(n), zero_ref_names=() if cfg.rope_base > 0 else ("dbk",))
            figures[n] = f
            print(report(n, f, floors.get(n)), "" if ok else f"FAILED {failed}")
        if not ok:
            bad.append(n)
    if intermediates:
        # the tensors the boundary exposes between the two passes: a wrong LSE or D that happened to cancel in the
        # gradients would show here
        iref = dict(Xn=saved["Xn"], Q=saved["Q"], K=saved["K"], V=saved["V"], A=saved["A"], LSE=saved["LSE"],
                    dA=g["dA"], D=g["D"], dQ=g["dQ"], dK=g["dK"], dV=g["dV"], dXn=g["dXn"])
        for n in INTERMEDIATES:
            got = run.saved_view(n)
            assert np.isfinite(got).all(), n
            if cfg.dtype == "fp32":
                # with one token per sequence dQ and dK (and D's partner dS) vanish identically: judge those against dV
                zero_ref = np.abs(iref[n]).max() < 1e-12 * max(np.abs(iref["dV"]).max(), 1e-300)
                err = float(np.abs(got).max() / np.abs(iref["dV"]).max()) if zero_ref else fp32_err(got, iref[n])
                ok = err <= FP32_REL
                print(f"{n:7s} fp32 scale-floored rel err {err:.3e}")
            else:
                zero_ref = np.abs(iref[n]).max() < 1e-12
                if zero_ref:
                    ok, f = bool(np.abs(got).max() <= 1e-2), dict(max_abs=float(np.abs(got).max()))
                    print(f"{n:7s} zero reference, max|got|={f['max_abs']:.3e}")
                else:
                    ok, f, failed = bf16_ok(n, got, iref[n])
                    print(report(n, f), "" if ok else f"FAILED {failed}")
                figures[n] = f
            if not ok:
                bad.append(n)
        stats = run.saved_view("stats")
        rstd_err = np.abs(stats[..., 1:2] - saved["rstd"]).max() / np.abs(saved["rstd"]).max()
        mean_ref = saved["mu"] if saved["mu"] is not None else np.zeros_like(saved["rstd"])
        mean_err = np.abs(stats[..., 0:1] - mean_ref).max()
        print(f"stats   rstd rel err {rstd_err:.3e} mean abs err {mean_err:.3e}")
        if rstd_err > 1e-5 or mean_err > 1e-5:
            bad.append("stats")
    if guard_bytes:
        assert run.guards_intact() == [], run.guards_intact()
    record(cfg.name, figures, floors)
    assert not bad, bad
    return run


def test_config1_fp32():
    run_and_compare(get_config(1))


@pytest.mark.parametrize("kw", [
    dict(norm="layernorm", causal=True, residual=True, has_bias=True),
    dict(norm="rmsnorm", causal=False, n_kv_heads=1),
    dict(norm="layernorm", causal=False, seq=77, batch=3),
    dict(norm="rmsnorm", causal=True, seq=150, head_dim=64, n_q_heads=2, n_kv_heads=1, d_model=128),
])
def test_fp32_variants(kw):
    run_and_compare(scaled_config(get_config(1), **kw), affine_noise=True)


SMALL_BF16 = [
    # several 128-row tiles with ragged tails, biases, GQA, both norms, hd 64 and 128
    LayerConfig("b1", 2, 200, 256, 4, 4, 64, "bf16", "layernorm", True, True, False, 1e-5, 21, 0.02),
    LayerConfig("b2", 3, 197, 256, 4, 2, 64, "bf16", "layernorm", False, False, True, 1e-6, 22, 0.02),
    LayerConfig("b3", 1, 333, 256, 4, 1, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 23, 0.02),
    LayerConfig("b4", 2, 130, 256, 2, 2, 128, "bf16", "rmsnorm", True, False, False, 1e-5, 24, 0.01),
    LayerConfig("b5", 1, 8, 128, 2, 2, 64, "bf16", "layernorm", True, True, False, 1e-5, 25, 0.02),
    LayerConfig("b6", 2, 1, 128, 2, 1, 64, "bf16", "rmsnorm", False, False, False, 1e-5, 26, 0.02),
    # enough blocks for the forward kernel to pair query tiles, with an odd tile count and a ragged last tile
    LayerConfig("b7", 10, 330, 512, 8, 2, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 27, 0.02),
    LayerConfig("b8", 20, 300, 512, 4, 4, 128, "bf16", "layernorm", False, True, True, 1e-5, 28, 0.02),
    # sequence an exact multiple of the 128-row tiles, group of 8 query heads per KV head
    LayerConfig("b9", 2, 256, 512, 8, 1, 64, "bf16", "layernorm", True, False, False, 1e-5, 29, 0.02),
]


@pytest.mark.parametrize("cfg", SMALL_BF16, ids=lambda c: c.name)
@pytest.mark.parametrize("path", [0, 1], ids=["default", "ffma"])
def test_bf16_small(cfg, path):
    run_and_compare(cfg, affine_noise=True, path=path)


@pytest.mark.parametrize("slices", [(3, 4), (19, 2)], ids=["o3-qkv4", "o19-qkv2"])
def test_sliced_weight_gradient_reductions(slices, monkeypatch):
    # The plan slices the token-axis reduction of dWo / dWq, dWk, dWv only when the replayed work dealing gains
    # from it (workload 3 does); the tuning knobs force it here on a shape with 19 k-blocks of tokens (ragged
    # last slice; one k-block per slice) and with biases, so that the sliced path is compared at a small size too.
    monkeypatch.setenv("FBL_KSPLIT_O", str(slices[0]))
    monkeypatch.setenv("FBL_KSPLIT_QKV", str(slices[1]))
    run_and_compare(LayerConfig("s1", 6, 197, 256, 4, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 31, 0.02),
                    affine_noise=True)


@pytest.mark.parametrize("cfg", [c for c in SMALL_BF16 if c.name in ("b1", "b4", "b8")] + [
    LayerConfig("p1", 3, 333, 512, 8, 4, 64, "bf16", "layernorm", True, True, True, 1e-5, 33, 0.02)], ids=lambda c: c.name)
def test_cta_pair_gemm_forced(cfg, monkeypatch):
    # Large layers run their GEMMs on CTA pairs (256 x 256 tiles, tcgen05 cta_group::2); workload 5 covers that at
    # full size.  The knob forces the pair kernel wherever its tile shape is legal, so that bias, residual, padding
    # rows, the fused row reduction, odd tile counts and tiles whose second half lies beyond the matrix are
    # compared at small sizes too.
    monkeypatch.setenv("FBL_GEMM_PAIR", "1")
    run_and_compare(cfg, affine_noise=True)


@pytest.mark.parametrize("sets", ["1", "2"])
def test_gemm_epilogue_sets_forced(sets, monkeypatch):
    # The single-CTA GEMM kernel drains a tile with one set of four warps, or, in launches where every block has one
    # tile, with two sets that share the tile's panels.  Small shapes get the second by default, large ones the
    # first; the knob forces each on shapes with bias, residual, padding rows, sliced reductions and the fused row
    # reduction at head_dim 64 and 128 (where a head spans both sets' panels and the first set takes the tile).
    monkeypatch.setenv("FBL_GEMM_ESETS", sets)
    for cfg in (LayerConfig("g1", 3, 333, 512, 8, 4, 64, "bf16", "layernorm", True, True, True, 1e-5, 51, 0.02),
                LayerConfig("g2", 2, 200, 256, 2, 1, 128, "bf16", "rmsnorm", False, False, True, 1e-5, 52, 0.02),
                LayerConfig("g3", 6, 197, 256, 4, 2, 64, "bf16", "layernorm", True, True, False, 1e-5, 53, 0.02)):
        run_and_compare(cfg, affine_noise=True)


@pytest.mark.parametrize("cfg", [
    LayerConfig("r1", 8, 600, 512, 8, 8, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 59, 0.02),
    # biases on: over 4800 tokens and four query heads per key head the rounding noise of the identically-zero dbk
    # passes 1e-2 even with exact sums of bf16-rounded operands, so it is judged against twice that floor (util.py)
    LayerConfig("r2", 8, 600, 512, 8, 2, 64, "bf16", "layernorm", False, True, True, 1e-5, 60, 0.02),
], ids=lambda c: c.name)
def test_forward_paired_tiles_with_odd_tile_count(cfg):
    # head_dim 64 forward with two query tiles per block and rotating score buffers, on a grid large enough for the
    # pairing to be chosen (192 blocks) and five query tiles per head: the last block of a head owns a single tile,
    # the other blocks two tiles whose key ranges differ by one tile (causal) or not at all (full attention)
    run_and_compare(cfg, affine_noise=True)


def test_forward_tile_variants_forced(monkeypatch):
    # head_dim 64 forward: one-tile blocks (two per SM) are the default for short sequences, two-tile blocks for long
    # ones; force each on a shape the other would get
    for mode, cfg in (("2", LayerConfig("f1", 2, 300, 256, 4, 2, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 34, 0.02)),
                      ("1", LayerConfig("f2", 1, 700, 256, 4, 4, 64, "bf16", "layernorm", True, True, False, 1e-5, 35, 0.02))):
        monkeypatch.setenv("FBL_FWD_TILES", mode)
        run_and_compare(cfg, affine_noise=True)


@pytest.mark.parametrize("i", [2, 3])
def test_full_configs_2_and_3(i):
    run_and_compare(get_config(i), guard_bytes=4096 if i == 3 else 0)


@pytest.mark.parametrize("cfg", [c for c in SMALL_BF16 if c.name in ("b1", "b2", "b4", "b8")] + [
    scaled_config(get_config(1), name="cfg1-guarded")], ids=lambda c: c.name)
def test_guard_bands_stay_intact(cfg):
    # Every device buffer of the step (matrices, vectors, `saved`, both scratch areas) sits between two 4 KiB bands
    # of a known byte pattern; a store past either end of a buffer (a bulk tensor store that is not clipped, the
    # 128-float copy window behind the last LSE row, a partial-sum area sized too small) would change one.
    run_and_compare(cfg, affine_noise=True, guard_bytes=4096)


@pytest.mark.parametrize("cfg", [
    LayerConfig("rp1", 2, 200, 256, 4, 2, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 71, 0.02, 0.0, 10000.0),
    LayerConfig("rp2", 3, 197, 256, 2, 2, 128, "bf16", "layernorm", False, True, True, 1e-5, 72, 0.02, 0.0, 10000.0),
    LayerConfig("rp3", 1, 64, 64, 2, 2, 32, "fp32", "layernorm", True, True, False, 1e-5, 73, 0.1, 0.0, 100.0),
    LayerConfig("rp4", 2, 2048, 512, 8, 2, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 74, 0.02, 0.0, 10000.0),
], ids=lambda c: c.name)
@pytest.mark.parametrize("path", [0, 1], ids=["default", "ffma"])
def test_rotary_embedding(cfg, path):
    # Q and K rotated by position between the projections and the scores, in place on the tiled buffers; the key bias
    # gradient is a real gradient here (the rotation breaks the shift invariance that makes it vanish)
    if path == 1 and cfg.seq > 1024:
        pytest.skip("the FFMA cross-check of the long case adds nothing")
    run_and_compare(cfg, affine_noise=True, path=path)


def test_padding_slots_are_zero_and_padded_equals_unpadded():
    import torch
    cfg = scaled_config(get_config(3), batch=2)
    run = run_and_compare(cfg)
    t_pad = 200
    y = run.buf["Y"].view(torch.bfloat16).float().view(cfg.d_model // 64, cfg.batch, t_pad, 64)
    dx = run.buf["dX"].view(torch.bfloat16).float().view(cfg.d_model // 64, cfg.batch, t_pad, 64)
    assert float(y[:, :, cfg.seq:].abs().max()) == 0.0 and float(dx[:, :, cfg.seq:].abs().max()) == 0.0


def test_config4_reduced_batch():
    run_and_compare(scaled_config(get_config(4), batch=1, seq=1024))


@pytest.mark.parametrize("i", [4, 5])
def test_full_configs_4_and_5(i):
    # the float64 oracle needs about half a minute (workload 4) and a few minutes (workload 5) on the host cores
    run_and_compare(get_config(i))
