"""Independent statement of the R-Tile layout and of the tile-index maps (integer oracle).

TEST INFRASTRUCTURE ONLY; shares no code with the library.  Written from the prose
definition, in tile form:

* a matrix [R, C] is cut into storage tiles of tile_h x tile_w elements (section 4.2,
  step 1), each tile stored contiguously, row-major inside (intra-tile mapping, the
  horizontal-strip case of Eq. 1's discussion);
* tiles are numbered with the row-tile coordinate running fastest (inter-tile mapping
  with the token axis as the primary dimension);
* token matrices [B, T, C] use rows b*T_pad + t, T_pad = T rounded up to tile_h;
* reshape/transposes that keep tiles whole are maps between row-major tile numberings
  of the two views (section 4.3, Eq. 3); they are obtained here by brute force:
  materialise the chain on an array of element ids and look where each tile went.
"""
from __future__ import annotations

import numpy as np


def ceil_to(v, m):
    return (v + m - 1) // m * m


def rtile_offset(r, c, r_pad, tile_h, tile_w):
    tiles_r = r_pad // tile_h
    tile_number = (c // tile_w) * tiles_r + (r // tile_h)
    return tile_number * (tile_h * tile_w) + (r % tile_h) * tile_w + (c % tile_w)


def pack_matrix(m2d, tile_h, tile_w, fill=0):
    """Row-major [R, C] -> flat R-Tile buffer (rows padded to tile_h, C must be whole tiles)."""
    R, Cc = m2d.shape
    assert Cc % tile_w == 0
    r_pad = ceil_to(R, tile_h)
    out = np.full(r_pad * Cc, fill, dtype=m2d.dtype)
    rr, cc = np.meshgrid(np.arange(R), np.arange(Cc), indexing="ij")
    out[rtile_offset(rr, cc, r_pad, tile_h, tile_w)] = m2d
    return out


def pack_tokens(x3d, tile_h, tile_w, fill=0):
    """Row-major [B, T, C] -> flat R-Tile buffer with every sequence padded to whole tiles."""
    B, T, Cc = x3d.shape
    t_pad = ceil_to(T, tile_h)
    padded = np.full((B, t_pad, Cc), fill, dtype=x3d.dtype)
    padded[:, :T] = x3d
    return pack_matrix(padded.reshape(B * t_pad, Cc), tile_h, tile_w, fill)


def tile_ids_of_view(view, tile_h, tile_w):
    """For an array whose last two axes are (rows, cols) cut into tiles, return per tile (row-major
    over all leading axes, then tile-row, tile-col) the sorted element ids it holds."""
    *lead, R, Cc = view.shape
    v = view.reshape(-1, R // tile_h, tile_h, Cc // tile_w, tile_w).transpose(0, 1, 3, 2, 4)
    return v.reshape(-1, tile_h * tile_w)


def brute_force_split_map(B, t_pad, heads, hd, tile_h, tile_w):
    """Tile map of (B, S, D) -> (B, S, H, HD) -> (B, H, S, HD), found by moving element ids."""
    D = heads * hd
    ids = np.arange(B * t_pad * D).reshape(B * t_pad, D)
    src_tiles = tile_ids_of_view(ids, tile_h, tile_w)                 # flat view, row-major tile numbering
    moved = ids.reshape(B, t_pad, heads, hd).transpose(0, 2, 1, 3)    # the reshape + transpose chain
    dst_tiles = tile_ids_of_view(moved, tile_h, tile_w)
    key = {tuple(t): i for i, t in enumerate(dst_tiles)}
    return np.array([key[tuple(t)] for t in src_tiles])              # raises if a tile was torn apart
