"""ctypes binding of the tile-propagation entry points (fbl_tile_chain_*): argument marshalling only."""
from __future__ import annotations

import ctypes as C

from .binding import FblError, lib

CHECKS = {0: "ok", 1: "dimension", 2: "boundary", 3: "continuity"}


class FblViewOp(C.Structure):
    _fields_ = [("kind", C.c_int32), ("rank", C.c_int32), ("shape", C.c_int64 * 8), ("perm", C.c_int32 * 8)]


class FblTileTerm(C.Structure):
    _fields_ = [("div", C.c_int64), ("mod", C.c_int64), ("mul", C.c_int64)]


def reshape(*shape):
    op = FblViewOp(kind=0, rank=len(shape))
    for i, v in enumerate(shape):
        op.shape[i] = int(v)
    return op


def permute(*perm):
    op = FblViewOp(kind=1, rank=len(perm))
    for i, v in enumerate(perm):
        op.perm[i] = int(v)
    return op


def expand(*shape):
    op = reshape(*shape)
    op.kind = 2
    return op


class IllegalChain(FblError):
    def __init__(self, failed_op, check):
        self.failed_op, self.check = failed_op, CHECKS[check]
        super().__init__(-2, f"operator {failed_op} breaks the tile structure: {self.check} check")


class TileChain:
    """The composed tile map of a reshape / permute chain; raises IllegalChain where the chain is not a pure tile move."""

    def __init__(self, shape, tile_h, tile_w, ops):
        L = lib()
        vp = C.c_void_p
        L.fbl_tile_chain_create.argtypes = [C.POINTER(C.c_int64), C.c_int, C.c_int, C.c_int, C.POINTER(FblViewOp), C.c_int,
                                            C.POINTER(vp), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.fbl_tile_chain_destroy.argtypes = [vp]
        L.fbl_tile_chain_destroy.restype = None
        L.fbl_tile_chain_tiles.argtypes = [vp]
        L.fbl_tile_chain_tiles.restype = C.c_int64
        L.fbl_tile_chain_terms.argtypes = [vp, C.POINTER(FblTileTerm), C.c_int]
        L.fbl_tile_chain_map.argtypes = [vp, C.c_int64, C.POINTER(C.c_int64)]
        self._h = vp()
        arr = (C.c_int64 * len(shape))(*[int(v) for v in shape])
        oparr = (FblViewOp * max(len(ops), 1))(*ops)
        fo, fc = C.c_int32(), C.c_int32()
        rc = L.fbl_tile_chain_create(arr, len(shape), tile_h, tile_w, oparr, len(ops), C.byref(self._h), C.byref(fo), C.byref(fc))
        if rc == -2:
            raise IllegalChain(fo.value, fc.value)
        if rc != 0:
            raise FblError(rc, "invalid tile chain arguments")

    def __del__(self):
        try:
            if self._h:
                lib().fbl_tile_chain_destroy(self._h)
        except Exception:
            pass

    @property
    def tiles(self):
        return lib().fbl_tile_chain_tiles(self._h)

    def terms(self):
        buf = (FblTileTerm * 32)()
        n = lib().fbl_tile_chain_terms(self._h, buf, 32)
        return [(buf[i].div, buf[i].mod, buf[i].mul) for i in range(n)]

    def map(self, src_tile):
        out = C.c_int64()
        rc = lib().fbl_tile_chain_map(self._h, src_tile, C.byref(out))
        if rc != 0:
            raise FblError(rc, "tile index out of range")
        return out.value
