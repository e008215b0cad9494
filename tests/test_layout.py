"""Integer index maps: the library's host code against the independent layout oracle (bit-exact)."""
import ctypes
import os
import re

import numpy as np
import pytest

from fbl_inputs import LayerConfig, get_config
from oracle import layout as lo
from paper_2607_21624_b200 import MAP, TENSOR, FblError, Plan, desc_from_config, lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def small(dtype="bf16", B=2, T=13, D=128, hq=2, hkv=1, hd=64):
    return LayerConfig("s", B, T, D, hq, hkv, hd, dtype, "layernorm", True, False, False, 1e-5, 0, 0.02)


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "fblayout.h")).read()
    names = set(re.findall(r"\b(fbl_[a-z_0-9]+)\s*\(", text))
    assert {"fbl_layer_fwd", "fbl_layer_bwd", "fbl_plan_create", "fbl_tile_map", "fbl_pack"} <= names
    L = lib()
    for n in sorted(names):
        assert hasattr(L, n), n


def test_paper_example_8x16_with_4x4_tiles():
    # the worked example of section 4.2: a [Dim2=8, Dim1=16] tensor cut into 4x4 tiles gives a 2x4 tile grid;
    # every tile is one contiguous run of 16 elements and the map is a bijection
    ids = np.arange(8 * 16).reshape(8, 16)
    buf = lo.pack_matrix(ids, 4, 4, fill=-1)
    assert sorted(buf.tolist()) == list(range(128))
    tiles = buf.reshape(8, 16)
    for t in tiles:
        r, c = np.divmod(t, 16)
        assert r.max() - r.min() == 3 and c.max() - c.min() == 3          # each run is one 4x4 block
        assert (np.diff(c.reshape(4, 4), axis=1) == 1).all()              # stride-1 innermost
    # reducing along either axis touches whole tiles only: tile sets of a row band / column band
    assert {int(x) // 16 for x in lo.rtile_offset(np.arange(4)[:, None], np.arange(16)[None], 8, 4, 4).ravel()} == {0, 2, 4, 6}
    assert {int(x) // 16 for x in lo.rtile_offset(np.arange(8)[:, None], np.arange(4)[None], 8, 4, 4).ravel()} == {0, 1}


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_element_map_matches_oracle_and_is_a_bijection(dtype):
    cfg = small(dtype, hd=64)
    plan = Plan(desc_from_config(cfg))
    tw = 64 if dtype == "bf16" else 32
    t_pad = lo.ceil_to(cfg.seq, 8)
    n_pad = cfg.batch * t_pad
    seen = set()
    for b in range(cfg.batch):
        for t in range(cfg.seq):
            for c in range(cfg.d_model):
                got = plan.tile_offset(TENSOR["X"], [b, t, c])
                assert got == lo.rtile_offset(b * t_pad + t, c, n_pad, 8, tw)
                seen.add(got)
    assert len(seen) == cfg.batch * cfg.seq * cfg.d_model
    assert max(seen) < plan.tensor_bytes(TENSOR["X"]) // (2 if dtype == "bf16" else 4)
    assert plan.tile_offset(TENSOR["X"], [0, cfg.seq, 0]) < 0 and plan.tile_offset(TENSOR["X"], [cfg.batch, 0, 0]) < 0
    # weights and their transposed views address the same element
    for r in range(0, cfg.d_model, 7):
        for c in range(0, cfg.d_q, 5):
            o = plan.tile_offset(TENSOR["WQ"], [r, c])
            assert o == lo.rtile_offset(r, c, cfg.d_model, 8, tw)
            assert o == plan.tile_offset(TENSOR["WQ_T"], [c, r])
    # head views address the same element as the flat view
    for b in range(cfg.batch):
        for h in range(cfg.n_q_heads):
            for t in range(0, cfg.seq, 3):
                for d in range(0, cfg.head_dim, 9):
                    assert plan.tile_offset(TENSOR["Q_HEADS"], [b, h, t, d]) == \
                        plan.tile_offset(TENSOR["Q"], [b, t, h * cfg.head_dim + d])


@pytest.mark.parametrize("dtype,hd,hq,hkv", [("bf16", 64, 3, 1), ("bf16", 128, 2, 2), ("fp32", 32, 4, 2), ("fp32", 64, 2, 1)])
def test_split_merge_maps_against_materialised_reshape_transpose(dtype, hd, hq, hkv):
    cfg = small(dtype, B=2, T=21, D=128, hq=hq, hkv=hkv, hd=hd)
    plan = Plan(desc_from_config(cfg))
    tw = 64 if dtype == "bf16" else 32
    t_pad = lo.ceil_to(cfg.seq, 8)
    for heads, split, merge in ((hq, "SPLIT_Q", "MERGE_Q"), (hkv, "SPLIT_KV", "MERGE_KV")):
        want = lo.brute_force_split_map(cfg.batch, t_pad, heads, hd, 8, tw)
        got = np.array([plan.tile_map(MAP[split], j) for j in range(len(want))])
        assert np.array_equal(got, want)
        back = np.array([plan.tile_map(MAP[merge], int(i)) for i in got])
        assert np.array_equal(back, np.arange(len(want)))
        with pytest.raises(FblError):
            plan.tile_map(MAP[split], len(want))


def test_transpose_and_physical_maps():
    cfg = small("bf16", D=128, hq=3, hd=64)
    plan = Plan(desc_from_config(cfg))
    R, Cc, tw = cfg.d_model, cfg.d_q, 64
    ids = np.arange(R * Cc).reshape(R, Cc)
    buf = lo.pack_matrix(ids, 8, tw)
    src_tiles = lo.tile_ids_of_view(ids, 8, tw)
    # transposed view: tiles become tw x 8 blocks of ids.T, numbered row-major in that view
    dst_tiles = lo.tile_ids_of_view(ids.T, tw, 8)
    key = {tuple(sorted(t)): i for i, t in enumerate(dst_tiles)}
    for j, t in enumerate(src_tiles):
        assert plan.tile_map(MAP["TRANSPOSE_WQ"], j) == key[tuple(sorted(t))]
        phys = plan.tile_map(MAP["PHYS_WQ"], j)
        assert np.array_equal(buf[phys * 8 * tw:(phys + 1) * 8 * tw], t)     # the tile sits, whole, at that slot
    # tile invariance: reading W for a K-axis reduction and W^T for an N-axis reduction touches the same slots
    fwd = {plan.tile_map(MAP["PHYS_WQ"], j) for j in range(len(src_tiles))}
    bwd = {plan.tile_map(MAP["TRANSPOSE_WQ"], j) for j in range(len(src_tiles))}
    assert fwd == bwd == set(range(len(src_tiles)))


def test_physical_map_of_token_matrix():
    cfg = small("bf16", B=2, T=13, hq=2, hd=64)
    plan = Plan(desc_from_config(cfg))
    t_pad = 16
    ids = np.arange(cfg.batch * cfg.seq * cfg.d_q).reshape(cfg.batch, cfg.seq, cfg.d_q)
    buf = lo.pack_tokens(ids, 8, 64, fill=-1)
    padded = np.full((cfg.batch, t_pad, cfg.d_q), -1)
    padded[:, :cfg.seq] = ids
    tiles = lo.tile_ids_of_view(padded.reshape(cfg.batch * t_pad, cfg.d_q), 8, 64)
    for j, t in enumerate(tiles):
        phys = plan.tile_map(MAP["PHYS_Q"], j)
        assert np.array_equal(buf[phys * 512:(phys + 1) * 512], t)


def test_strength_reduction_identity():
    # i mod Ca mod Cb == i mod Cb whenever Cb divides Ca (section 4.3), and not in general otherwise
    for ca in range(1, 40):
        for cb in range(1, 40):
            same = all((i % ca) % cb == i % cb for i in range(0, 400))
            if ca % cb == 0:
                assert same
    assert any((i % 6) % 4 != i % 4 for i in range(50))


def test_legality_checks():
    ok = small("bf16", D=768, hq=12, hkv=12, hd=64)
    Plan(desc_from_config(ok))
    for bad in (small("bf16", D=768, hq=16, hkv=16, hd=48),      # head boundary cuts a tile: 48 not a multiple of 64
                small("bf16", D=96, hq=1, hkv=1, hd=64),         # d_model not whole tiles
                small("bf16", D=128, hq=3, hkv=2, hd=64)):       # query heads not whole GQA groups
        with pytest.raises(FblError) as e:
            Plan(desc_from_config(bad))
        assert e.value.code == -2
    # fp32 tiles are 32 wide, so head_dim 32 keeps tiles whole there
    Plan(desc_from_config(small("fp32", D=64, hq=2, hkv=2, hd=32)))


def test_padding_rule_and_sizes():
    # 197 tokens pad to 200 (1.5 %, within the 10 % rule of constraint C3), not to a 128 multiple
    plan = Plan(desc_from_config(get_config(3)))
    assert plan.tensor_bytes(TENSOR["X"]) == 32 * 200 * 768 * 2
    saved, sf, sb = plan.workspace_bytes()
    assert saved > 0 and sf > 0 and sb > 0


def test_partial_sum_area_covers_what_the_backward_kernels_write():
    # The last area of the backward scratch takes the slab partials of the four bias column sums (one row of
    # D + Dq + 2 Dkv floats per slab of 256 token rows), then, from the next 256-float boundary, the norm backward's
    # per-block partial rows (dgamma and dbeta, at most two blocks per SM).  Recompute that requirement for large
    # layers and compare with what the plan reserves; the area must also end inside the scratch size the plan reports.
    from fbl_inputs import LayerConfig
    from paper_2607_21624_b200 import WS
    sms = 148
    for (b, t, d, hq, hkv, hd, bias) in [(16, 8192, 4096, 32, 32, 128, True), (1, 8192, 4096, 32, 32, 128, False),
                                         (64, 2048, 2048, 32, 8, 64, True), (32, 197, 768, 12, 12, 64, True),
                                         (4, 512, 768, 12, 12, 64, True), (128, 1024, 1024, 16, 16, 64, True)]:
        cfg = LayerConfig("big", b, t, d, hq, hkv, hd, "bf16", "layernorm", True, bias, False, 1e-5, 0, 0.02)
        plan = Plan(desc_from_config(cfg))
        n_pad = b * ((t + 7) // 8 * 8)
        slabs = (n_pad + 255) // 256
        cs_floats = slabs * (d + hq * hd + 2 * hkv * hd) if bias else 0
        wpr = {1: 1, 2: 1, 3: 1, 4: 2, 6: 2, 8: 4, 12: 4, 16: 8}[d // 256]
        blocks = min(2 * sms, n_pad // (8 // wpr))
        need = ((cs_floats + 255) // 256 * 256 + blocks * 2 * d) * 4
        off, nbytes = plan.workspace_offset(WS["PARTIALS"])
        _, _, sb = plan.workspace_bytes()
        assert nbytes >= need, (cfg, nbytes, need)
        assert off + nbytes <= sb


def test_cross_attention_plan_host_maps_follow_the_memory_side():
    # K, V, Wk, Wv (and the memory itself) of a cross-attention plan take the memory's sequence length and width;
    # everything else keeps the query side's.  Element map against the layout oracle, sizes, and the rejections.
    from fbl_inputs import XattnConfig
    from paper_2607_21624_b200 import WS
    cfg = XattnConfig("xl", 2, 13, 21, 128, 192, 2, 1, 64, "bf16", "layernorm", True, True, 1e-5, 0, 0.02)
    plan = Plan(desc_from_config(cfg), cross=(cfg.seq_kv, cfg.d_mem))
    tw, tq_pad, tk_pad = 64, 16, 24
    assert plan.tensor_bytes(TENSOR["X"]) == 2 * tq_pad * 128 * 2
    assert plan.tensor_bytes(TENSOR["MEM"]) == plan.tensor_bytes(TENSOR["DMEM"]) == 2 * tk_pad * 192 * 2
    assert plan.tensor_bytes(TENSOR["K"]) == 2 * tk_pad * 64 * 2 and plan.tensor_bytes(TENSOR["Q"]) == 2 * tq_pad * 128 * 2
    assert plan.tensor_bytes(TENSOR["WK"]) == 192 * 64 * 2 and plan.tensor_bytes(TENSOR["WQ"]) == 128 * 128 * 2
    seen = set()
    for b in range(cfg.batch):
        for t in range(cfg.seq_kv):
            for c in range(0, cfg.d_mem, 5):
                got = plan.tile_offset(TENSOR["MEM"], [b, t, c])
                assert got == lo.rtile_offset(b * tk_pad + t, c, 2 * tk_pad, 8, tw)
                seen.add(got)
            for d in range(0, 64, 7):
                assert plan.tile_offset(TENSOR["K_HEADS"], [b, 0, t, d]) == plan.tile_offset(TENSOR["K"], [b, t, d]) == \
                    lo.rtile_offset(b * tk_pad + t, d, 2 * tk_pad, 8, tw)
    assert len(seen) == cfg.batch * cfg.seq_kv * len(range(0, cfg.d_mem, 5))
    assert plan.tile_offset(TENSOR["K_HEADS"], [0, 0, cfg.seq_kv, 0]) < 0          # past the memory's length
    assert plan.tile_offset(TENSOR["Q_HEADS"], [0, 0, cfg.seq, 0]) < 0              # past the query side's
    assert plan.tile_offset(TENSOR["Q_HEADS"], [1, 1, cfg.seq - 1, 63]) == lo.rtile_offset(tq_pad + cfg.seq - 1, 127, 2 * tq_pad, 8, tw)
    for r in range(0, cfg.d_mem, 11):
        assert plan.tile_offset(TENSOR["WK"], [r, 3]) == lo.rtile_offset(r, 3, cfg.d_mem, 8, tw) == plan.tile_offset(TENSOR["WK_T"], [3, r])
    # the workspace areas of K, V, dK, dV are sized by the memory's rows and do not overlap their neighbours
    areas = sorted(plan.workspace_offset(WS[k]) for k in ("STATS", "XN", "Q", "K", "V", "A", "LSE"))
    for (o0, n0), (o1, _) in zip(areas, areas[1:]):
        assert o0 + n0 <= o1
    assert plan.workspace_offset(WS["K"])[1] == plan.workspace_offset(WS["DK"])[1] == 2 * tk_pad * 64 * 2
    # a self-attention plan has no memory; a cross plan takes no mask, and its memory width must be whole tiles
    with pytest.raises(FblError):
        Plan(desc_from_config(small())).tensor_bytes(TENSOR["MEM"])
    import dataclasses
    with pytest.raises(FblError):
        Plan(desc_from_config(dataclasses.replace(cfg, causal=True)), cross=(cfg.seq_kv, cfg.d_mem))
    with pytest.raises(FblError):
        Plan(desc_from_config(cfg), cross=(cfg.seq_kv, 100))
    with pytest.raises(FblError):
        Plan(desc_from_config(cfg), cross=(0, cfg.d_mem))
