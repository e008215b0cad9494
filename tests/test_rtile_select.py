"""Offline tile selection: the candidate filter (host code of the library) and the scoring of Eq. 2."""
import pytest

from fbl_inputs import get_config
from paper_2607_21624_b200 import rtile


def test_candidate_filter_keeps_the_descriptor_compatible_tiles():
    cfg = get_config(3)                                   # 32 x 197 tokens: the ragged one
    cands, rej = rtile.candidates(rtile.layer_matrix_shapes(cfg), 2, 0.10)
    # pool = 8 heights x 5 widths; C1 keeps only 128-byte rows with whole swizzle atoms that divide 128 rows
    # 8, 16, 32, 64, 128 rows pass C1; 64- and 128-row tiles exceed the 4 KiB of C2; 32-row tiles pad 197 rows by 13.7 %
    assert rej == {"C1": 35, "C2": 2, "C3": 1}
    assert [c["tile_h"] for c in cands] == [8, 16]
    assert cands[0]["tile_h"] == 8 and cands[0]["tile_w"] == 64 and cands[0]["n_cache"] == 8
    assert all(c["tile_w"] == 64 for c in cands)
    assert [c["tile_h"] for c in cands] == sorted(c["tile_h"] for c in cands)


def test_padding_constraint():
    # a 197-row matrix: 8-row tiles pad to 200 (1.5 %), 16-row tiles to 208 (5.6 %), 32-row tiles to 224 (13.7 %)
    cands, rej = rtile.candidates([(197, 768)], 2, 0.10)
    assert [c["tile_h"] for c in cands] == [8, 16]
    assert abs(cands[0]["pad_ratio"] - (200 / 197 - 1)) < 1e-6
    assert rej["C3"] == 1
    loose, _ = rtile.candidates([(197, 768)], 2, 0.20)
    assert [c["tile_h"] for c in loose] == [8, 16, 32]
    # fp32: 32 elements per 128-byte row
    c32, _ = rtile.candidates([(64, 64)], 4, 0.10)
    assert c32[0]["tile_w"] == 32
    with pytest.raises(Exception):
        rtile.candidates([(0, 64)], 2, 0.10)


def test_mem_efficiency_and_argmax_of_eq2():
    cfg = get_config(2)
    ops = rtile.launch_ops(cfg)["proj_o"]
    # wider and taller tiles fetch fewer bytes per flop
    e128 = rtile.mem_efficiency(ops, 128, 128, l2_bytes=0)
    e256 = rtile.mem_efficiency(ops, 128, 256, l2_bytes=0)
    epair = rtile.mem_efficiency(ops, 256, 256, l2_bytes=0)
    assert 0 < e128 < e256 < epair <= 1.0
    # this launch's operands (a few MB) stay in L2: every tile shape moves the once-only bytes across HBM
    assert rtile.mem_efficiency(ops, 128, 128) == 1.0
    # one tile covering the whole problem reads every operand once
    assert abs(rtile.mem_efficiency([(128, 128, 512)], 128, 128) - 1.0) < 1e-12
    times = {"proj_o": {(128, 0, 1): 0.010, (256, 0, 1): 0.0101, (256, 1, 1): 0.02}}
    picked, detail = rtile.choose(cfg, times)
    assert picked["proj_o"] == [128, 0, 1]            # L2-resident: the fastest wins
    big = get_config(5)                               # operands of 370 MB: the tile shape decides the HBM traffic
    picked, detail = rtile.choose(big, {"proj_qkv": {(128, 0, 1): 0.500, (256, 0, 1): 0.505, (256, 1, 1): 1.0}})
    # 1 % slower but a third fewer bytes: Eq. 2 prefers the wider tile; the pair tile is too slow here to win
    assert picked["proj_qkv"] == [256, 0, 1]
    assert detail["proj_qkv|128,0,1"]["gflops"] > detail["proj_qkv|256,0,1"]["gflops"]


def test_table_keys_are_shape_specific():
    assert rtile.shape_key(get_config(2)) != rtile.shape_key(get_config(3))
    assert set(rtile.launch_ops(get_config(4))) == set(rtile.LAUNCHES)
