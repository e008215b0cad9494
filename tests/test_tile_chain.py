"""Tile propagation through reshape / permute chains: the composed tile map against a brute-force materialisation
(numpy moves every element id through the chain), the three legality checks, and the strength reduction."""
import numpy as np
import pytest

from fbl_inputs import get_config
from paper_2607_21624_b200 import MAP, Plan, desc_from_config
from paper_2607_21624_b200.tile_chain import IllegalChain, TileChain, expand, permute, reshape


def tiles_of(mat2d, th, tw):
    r, c = mat2d.shape
    return mat2d.reshape(r // th, th, c // tw, tw).transpose(0, 2, 1, 3).reshape(-1, th * tw)


def brute_force(shape, th, tw, np_ops):
    ids = np.arange(int(np.prod(shape))).reshape(shape)
    src = tiles_of(ids.reshape(-1, shape[-1]), th, tw)
    out = ids
    for f in np_ops:
        out = f(out)
    dst = tiles_of(np.ascontiguousarray(out).reshape(-1, out.shape[-1]), th, tw)
    where = {tuple(t): i for i, t in enumerate(dst)}
    return [where[tuple(t)] for t in src]          # KeyError if a source tile is not a destination tile


CASES = [
    # the attention head split (B, S, D) -> (B, S, H, HD) -> (B, H, S, HD), bf16 tiles of 8 x 64
    ((2, 16, 256), 8, 64, [reshape(2, 16, 4, 64), permute(0, 2, 1, 3)],
     [lambda a: a.reshape(2, 16, 4, 64), lambda a: a.transpose(0, 2, 1, 3)]),
    # head_dim 128 = two tiles across
    ((3, 24, 512), 8, 64, [reshape(3, 24, 4, 128), permute(0, 2, 1, 3)],
     [lambda a: a.reshape(3, 24, 4, 128), lambda a: a.transpose(0, 2, 1, 3)]),
    # narrower tiles than the head (tile_w = 8 with head_dim 64: legal, as in the paper's example)
    ((1, 8, 128), 4, 8, [reshape(1, 8, 2, 64), permute(0, 2, 1, 3)],
     [lambda a: a.reshape(1, 8, 2, 64), lambda a: a.transpose(0, 2, 1, 3)]),
    # the merge back, then a batch / head regrouping: five operators collapse into one map
    ((2, 4, 16, 64), 8, 64, [permute(0, 2, 1, 3), reshape(2, 16, 256), reshape(2, 2, 8, 256), permute(1, 0, 2, 3), reshape(4, 8, 256)],
     [lambda a: a.transpose(0, 2, 1, 3), lambda a: a.reshape(2, 16, 256), lambda a: a.reshape(2, 2, 8, 256),
      lambda a: a.transpose(1, 0, 2, 3), lambda a: a.reshape(4, 8, 256)]),
    # cross-attention (Whisper-like): keys of an encoder sequence of 40 frames, queries elsewhere; split of the K side
    ((2, 40, 384), 8, 64, [reshape(2, 40, 6, 64), permute(0, 2, 1, 3)],
     [lambda a: a.reshape(2, 40, 6, 64), lambda a: a.transpose(0, 2, 1, 3)]),
    # fp32 tiles (8 x 32), sequence split into blocks and blocks moved outermost
    ((2, 32, 64), 8, 32, [reshape(2, 4, 8, 64), permute(1, 0, 2, 3)],
     [lambda a: a.reshape(2, 4, 8, 64), lambda a: a.transpose(1, 0, 2, 3)]),
    # no operator at all: the identity
    ((4, 8, 64), 8, 64, [], []),
]


@pytest.mark.parametrize("shape,th,tw,ops,np_ops", CASES)
def test_composed_map_equals_materialised_chain(shape, th, tw, ops, np_ops):
    chain = TileChain(shape, th, tw, ops)
    want = brute_force(shape, th, tw, np_ops)
    assert chain.tiles == len(want)
    assert [chain.map(j) for j in range(chain.tiles)] == want
    # f is a bijection of the tile numbers
    assert sorted(want) == list(range(len(want)))


def test_strength_reduction_merges_digits():
    # (B, S, D) -> (B, H, S, HD): digits of the source tile number are (b, s_tile, h, hd_tile); b stays outermost and
    # hd_tile innermost, so the map needs three terms, not four, and the outermost carries no modulo
    chain = TileChain((2, 16, 256), 8, 64, [reshape(2, 16, 4, 64), permute(0, 2, 1, 3)])
    terms = chain.terms()
    assert terms == [(8, 0, 8), (4, 2, 1), (1, 4, 2)]         # b: j/8*8; s_tile: (j/4)%2; h: j%4 * 2
    # head_dim of two tiles: b | s_tile | h | hd_tile all move separately (s_tile lands between h and hd_tile): four terms
    assert len(TileChain((3, 24, 512), 8, 64, [reshape(3, 24, 4, 128), permute(0, 2, 1, 3)]).terms()) == 4
    # a chain that ends where it began collapses to the identity: one term without any modulo
    ident = TileChain((2, 16, 256), 8, 64, [reshape(2, 16, 4, 64), permute(0, 2, 1, 3), permute(0, 2, 1, 3), reshape(2, 16, 256)])
    assert ident.terms() == [(1, 0, 1)]
    assert all(ident.map(j) == j for j in range(ident.tiles))


def test_matches_the_layer_plans_head_split_map():
    # the attention layer's own split map (fbl_tile_map) is this chain for its shapes
    cfg = get_config(3)
    plan = Plan(desc_from_config(cfg))
    t_pad = 200
    chain = TileChain((cfg.batch, t_pad, cfg.d_q), 8, 64, [reshape(cfg.batch, t_pad, cfg.n_q_heads, 64), permute(0, 2, 1, 3)])
    for j in list(range(0, chain.tiles, 97)) + [chain.tiles - 1]:
        assert chain.map(j) == plan.tile_map(MAP["SPLIT_Q"], j)


def test_the_three_checks():
    # boundary: hidden 768 -> 16 heads of 48 cuts 64-wide tiles (the paper's counter-example); so does head_dim 32
    with pytest.raises(IllegalChain) as e:
        TileChain((1, 8, 768), 8, 64, [reshape(1, 8, 16, 48), permute(0, 2, 1, 3)])
    assert (e.value.failed_op, e.value.check) == (0, "boundary")
    with pytest.raises(IllegalChain) as e:
        TileChain((1, 8, 768), 8, 64, [reshape(1, 8, 24, 32)])
    assert e.value.check == "boundary"
    # boundary: 197 rows are not whole 8-row tiles (the caller pads to 200 first)
    with pytest.raises(IllegalChain) as e:
        TileChain((2, 197, 128), 8, 64, [])
    assert (e.value.failed_op, e.value.check) == (-1, "boundary")
    TileChain((2, 200, 128), 8, 64, [])
    # boundary: splitting the sequence into blocks smaller than a tile's rows
    with pytest.raises(IllegalChain) as e:
        TileChain((2, 32, 64), 8, 64, [reshape(2, 8, 4, 64)])
    assert e.value.check == "boundary"
    # dimension: transposing the last two axes moves the tile's column axis onto the rows (that case is served by
    # operand orientation, not by a tile map)
    with pytest.raises(IllegalChain) as e:
        TileChain((2, 64, 128), 8, 64, [permute(0, 2, 1)])
    assert (e.value.failed_op, e.value.check) == (0, "dimension")
    # continuity: (B, S, H, HD) -> (B, S, HD, H) keeps hd on the column axis but makes H innermost: the elements of a
    # tile row are no longer adjacent
    with pytest.raises(IllegalChain) as e:
        TileChain((2, 16, 256), 8, 64, [reshape(2, 16, 4, 64), permute(0, 1, 3, 2), reshape(2, 16, 256)])
    assert e.value.check == "continuity"
    # continuity on the row axis: (B, S, D) -> (S, B, D) interleaves the rows of a tile with other batches
    with pytest.raises(IllegalChain) as e:
        TileChain((4, 16, 64), 8, 64, [permute(1, 0, 2)])
    assert (e.value.failed_op, e.value.check) == (0, "continuity")
    # dimension: an expansion (grouped-query K/V repeated per query head) changes the element count
    with pytest.raises(IllegalChain) as e:
        TileChain((2, 2, 16, 64), 8, 64, [expand(2, 8, 16, 64)])
    assert (e.value.failed_op, e.value.check) == (0, "dimension")
    # a chain that passes through an illegal arrangement but ends legal is accepted (only the collapsed map matters)
    TileChain((4, 16, 64), 8, 64, [permute(1, 0, 2), permute(1, 0, 2)])
