"""Thin ctypes binding over libfblayout's C ABI: argument marshalling only.

``Plan`` mirrors the C entry points one to one.  ``LayerRunner`` owns the torch
device buffers a caller needs (PyTorch is used for device memory and streams, nothing
else) and offers pack / forward / backward / unpack in terms of them.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libfblayout.so")

DTYPES = {"fp32": 0, "bf16": 1}
NORMS = {"layernorm": 0, "rmsnorm": 1}
TENSOR = {n: i for i, n in enumerate(
    ["X", "Y", "DY", "DX", "WQ", "WK", "WV", "WO", "XN", "Q", "K", "V", "A",
     "Q_HEADS", "K_HEADS", "V_HEADS", "A_HEADS", "WQ_T", "WK_T", "WV_T", "WO_T", "MEM", "DMEM"])}
WS = {n: i for i, n in enumerate(
    ["STATS", "XN", "Q", "K", "V", "A", "LSE", "D", "DA", "DQ", "DK", "DV", "DXN", "PARTIALS"])}
MAP = {n: i for i, n in enumerate(
    ["SPLIT_Q", "MERGE_Q", "SPLIT_KV", "MERGE_KV", "TRANSPOSE_WQ", "TRANSPOSE_WO", "PHYS_Q", "PHYS_WQ"])}


class FblLayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("batch", "seq", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "dtype", "norm", "causal",
                 "has_bias", "residual")] + [("eps", C.c_float), ("softmax_scale", C.c_float)]


class FblError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(what)


_lib = None


def load_library():
    """Load libfblayout.so (built in-tree).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FblError(-100, f"{LIB_PATH} is missing: run `python -m paper_2607_21624_b200.build` first")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
    L.fbl_plan_create.argtypes = [C.POINTER(FblLayerDesc), C.POINTER(vp)]
    L.fbl_plan_destroy.argtypes = [vp]
    L.fbl_plan_destroy.restype = None
    L.fbl_tensor_bytes.argtypes = [vp, C.c_int, C.POINTER(sz)]
    L.fbl_workspace_bytes.argtypes = [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
    L.fbl_workspace_offset.argtypes = [vp, C.c_int, C.POINTER(sz), C.POINTER(sz)]
    L.fbl_selftest_wait_timeout.argtypes = [vp, i64, vp]
    L.fbl_tile_offset.argtypes = [vp, C.c_int, C.POINTER(i32)]
    L.fbl_tile_offset.restype = i64
    L.fbl_tile_map.argtypes = [vp, C.c_int, i64, C.POINTER(i64)]
    L.fbl_pack.argtypes = [vp, C.c_int, vp, vp, vp]
    L.fbl_unpack.argtypes = [vp, C.c_int, vp, vp, vp]
    L.fbl_layer_fwd.argtypes = [vp] * 16
    L.fbl_layer_bwd.argtypes = [vp] * 22
    L.fbl_colsum_scratch_bytes.argtypes = [vp, i64, i64, C.POINTER(sz)]
    L.fbl_colsum.argtypes = [vp, vp, i64, i64, vp, vp, vp]
    L.fbl_colsum_noalloc.argtypes = [vp, vp, i64, i64, vp, vp]
    L.fbl_status_poll.argtypes = [vp, vp, C.POINTER(i32)]
    L.fbl_plan_set_kernel_path.argtypes = [vp, C.c_int]
    L.fbl_plan_enable_rope.argtypes = [vp, C.c_float]
    L.fbl_profile_enable.argtypes = [vp, C.c_int]
    L.fbl_profile_read.argtypes = [vp, C.c_int, C.POINTER(C.c_char_p), C.POINTER(C.c_float)]
    L.fbl_launch_count.argtypes = [vp]
    L.fbl_launch_count.restype = i64
    L.fbl_strerror.argtypes = [C.c_int]
    L.fbl_strerror.restype = C.c_char_p
    L.fbl_last_error_detail.restype = C.c_char_p
    _lib = L
    return L


def lib():
    return load_library()


def _check(code):
    if code != 0:
        L = lib()
        raise FblError(code, f"{L.fbl_strerror(code).decode()} [{L.fbl_last_error_detail().decode()}]")


def desc_from_config(cfg) -> FblLayerDesc:
    return FblLayerDesc(cfg.batch, cfg.seq, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                        DTYPES[cfg.dtype], NORMS[cfg.norm], int(cfg.causal), int(cfg.has_bias), int(cfg.residual),
                        cfg.eps, cfg.softmax_scale)


class Plan:
    """One fbl_plan.  Methods carry the C entry points' names without the ``fbl_`` prefix."""

    def __init__(self, desc: FblLayerDesc, cross=None):
        """``cross`` = (seq_kv, d_mem) makes a cross-attention plan (fbl_xattn_plan_create)."""
        self._h = C.c_void_p()
        self.desc = desc
        if cross is None:
            _check(lib().fbl_plan_create(C.byref(desc), C.byref(self._h)))
        else:
            L = lib()
            L.fbl_xattn_plan_create.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
            _check(L.fbl_xattn_plan_create(C.byref(desc), int(cross[0]), int(cross[1]), C.byref(self._h)))

    def close(self):
        if self._h:
            lib().fbl_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def tensor_bytes(self, tensor_id: int) -> int:
        out = C.c_size_t()
        _check(lib().fbl_tensor_bytes(self._h, tensor_id, C.byref(out)))
        return out.value

    def workspace_bytes(self):
        a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
        _check(lib().fbl_workspace_bytes(self._h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def workspace_offset(self, what: int):
        off, nbytes = C.c_size_t(), C.c_size_t()
        _check(lib().fbl_workspace_offset(self._h, what, C.byref(off), C.byref(nbytes)))
        return off.value, nbytes.value

    def tile_offset(self, tensor_id: int, idx) -> int:
        arr = (C.c_int32 * 4)(*(list(idx) + [0] * (4 - len(idx))))
        return lib().fbl_tile_offset(self._h, tensor_id, arr)

    def tile_map(self, map_id: int, src_tile: int) -> int:
        out = C.c_int64()
        _check(lib().fbl_tile_map(self._h, map_id, src_tile, C.byref(out)))
        return out.value

    def set_kernel_path(self, path: int):
        _check(lib().fbl_plan_set_kernel_path(self._h, path))

    def pack(self, tensor_id, rowmajor_ptr, tiled_ptr, stream):
        _check(lib().fbl_pack(self._h, tensor_id, rowmajor_ptr, tiled_ptr, stream))

    def unpack(self, tensor_id, tiled_ptr, rowmajor_ptr, stream):
        _check(lib().fbl_unpack(self._h, tensor_id, tiled_ptr, rowmajor_ptr, stream))

    def layer_fwd(self, X, gamma, beta, Wq, Wk, Wv, Wo, bq, bk, bv, bo, Y, saved, scratch, stream):
        _check(lib().fbl_layer_fwd(self._h, X, gamma, beta, Wq, Wk, Wv, Wo, bq, bk, bv, bo, Y, saved, scratch, stream))

    def layer_bwd(self, dY, X, gamma, Wq, Wk, Wv, Wo, saved, dX, dWq, dWk, dWv, dWo, dbq, dbk, dbv, dbo, dgamma,
                  dbeta, scratch, stream):
        _check(lib().fbl_layer_bwd(self._h, dY, X, gamma, Wq, Wk, Wv, Wo, saved, dX, dWq, dWk, dWv, dWo, dbq, dbk,
                                   dbv, dbo, dgamma, dbeta, scratch, stream))

    def colsum_scratch_bytes(self, rows, cols) -> int:
        out = C.c_size_t()
        _check(lib().fbl_colsum_scratch_bytes(self._h, rows, cols, C.byref(out)))
        return out.value

    def colsum(self, M, rows, cols, out, scratch, stream):
        _check(lib().fbl_colsum(self._h, M, rows, cols, out, scratch, stream))

    def colsum_noalloc(self, M, rows, cols, out, stream):
        """fbl_colsum with the partial sums kept in the library's own fixed array (allocates nothing)."""
        _check(lib().fbl_colsum_noalloc(self._h, M, rows, cols, out, stream))

    def profile_enable(self, on: bool):
        _check(lib().fbl_profile_enable(self._h, int(on)))

    def profile_read(self):
        names = (C.c_char_p * 32)()
        ms = (C.c_float * 32)()
        n = lib().fbl_profile_read(self._h, 32, names, ms)
        if n < 0:
            _check(n)
        return [(names[i].decode(), float(ms[i])) for i in range(n)]

    def launch_count(self) -> int:
        return lib().fbl_launch_count(self._h)

    def status_poll(self, scratch) -> int:
        out = C.c_int32()
        code = lib().fbl_status_poll(self._h, scratch, C.byref(out))
        if code not in (0, -6):
            _check(code)
        return out.value


def selftest_wait_timeout(scratch_ptr, limit_cycles, stream):
    """fbl_selftest_wait_timeout: enqueue the kernel whose bounded wait is meant to expire."""
    _check(lib().fbl_selftest_wait_timeout(scratch_ptr, limit_cycles, stream))


GUARD_BYTE = 0xA5


def aligned_bytes(torch, nbytes, device, align=1024, zero=True, guard=0):
    """A uint8 device tensor of ``nbytes`` whose data pointer is ``align``-byte aligned (torch only
    promises 512).  With ``guard`` > 0 (a multiple of ``align``) the view sits between two bands of that many
    bytes filled with GUARD_BYTE; ``guard_bands_intact`` checks them."""
    raw = (torch.zeros if zero else torch.empty)(nbytes + align + 2 * guard, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % align
    if guard:
        assert guard % align == 0
        raw[off:off + guard] = GUARD_BYTE
        raw[off + guard + nbytes:off + 2 * guard + nbytes] = GUARD_BYTE
    view = raw[off + guard:off + guard + nbytes]
    view._fbl_guard = (raw, off, guard, nbytes)
    return view


def guard_bands_intact(view) -> bool:
    raw, off, guard, nbytes = view._fbl_guard
    if not guard:
        return True
    lo = raw[off:off + guard]
    hi = raw[off + guard + nbytes:off + 2 * guard + nbytes]
    return bool((lo == GUARD_BYTE).all().item()) and bool((hi == GUARD_BYTE).all().item())


class LayerRunner:
    """Device buffers for one layer plus pack/step/unpack helpers (torch for memory and streams only)."""

    MATS = {"X": "X", "dY": "DY", "Wq": "WQ", "Wk": "WK", "Wv": "WV", "Wo": "WO"}
    OUT_MATS = {"Y": "Y", "dX": "DX", "dWq": "WQ", "dWk": "WK", "dWv": "WV", "dWo": "WO"}

    def __init__(self, cfg, device="cuda:0", guard_bytes=0, tile_choices=None, _before_sizes=None):
        """``tile_choices``: the GEMM launches' compute-tile configurations ({launch name: [tile_n, cta_pair,
        epilogue_sets]}, see rtile.py); None takes the layer's entry of the offline table shipped with the package,
        if it has one, {} leaves every launch to the built-in heuristics.
        ``guard_bytes`` > 0 surrounds every device buffer with bands of a known byte pattern
        (``guards_intact`` checks them): a stand-in for a memory checker when hunting writes past a buffer."""
        import torch
        if not torch.cuda.is_available():
            raise FblError(-101, "no CUDA device: the layer has no CPU path")
        self.torch = torch
        self.cfg = cfg
        self.dev = torch.device(device)
        self.plan = self._make_plan(cfg)
        from . import rtile
        if tile_choices is None:
            tile_choices = rtile.load_table().get(rtile.shape_key(cfg), {}).get("choices", {})
        self.tile_choices = tile_choices
        if tile_choices:
            rtile.apply(self.plan, tile_choices)
        self.tdtype = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
        if getattr(cfg, "rope_base", 0.0) > 0.0:
            _check(lib().fbl_plan_enable_rope(self.plan._h, cfg.rope_base))
        if _before_sizes is not None:
            _before_sizes(self.plan)          # a subclass's plan options that change the work areas
        saved, sf, sb = self.plan.workspace_bytes()
        self.sizes = dict(saved=saved, scratch_fwd=sf, scratch_bwd=sb)
        al = lambda nbytes: aligned_bytes(torch, nbytes, self.dev, guard=guard_bytes)
        self.saved = al(saved)
        # one scratch per pass: each pass clears the status word of its own scratch, so a time-out recorded by a
        # forward kernel is still there after the backward has run
        self.scratch_fwd = al(sf)
        self.scratch = al(sb)
        self.buf = {}
        for name, tid in {**self.MATS, **self.OUT_MATS}.items():
            self.buf[name] = al(self.plan.tensor_bytes(TENSOR[tid]))
        d, dq, dkv = cfg.d_model, cfg.d_q, cfg.d_kv
        fz = lambda n: torch.zeros(n, dtype=torch.float32, device=self.dev)
        lens = {"gamma": d, "beta": d, "bq": dq, "bk": dkv, "bv": dkv, "bo": d,
                "dgamma": d, "dbeta": d, "dbq": dq, "dbk": dkv, "dbv": dkv, "dbo": d}
        if guard_bytes:
            self._vec_raw = {k: al(4 * n) for k, n in lens.items()}
            self.vec = {k: v.view(torch.float32) for k, v in self._vec_raw.items()}
        else:
            self._vec_raw = {}
            self.vec = {k: fz(n) for k, n in lens.items()}

    # -- helpers ---------------------------------------------------------------------------
    def _make_plan(self, cfg):
        return Plan(desc_from_config(cfg))

    def _stream(self):
        return self.torch.cuda.current_stream(self.dev).cuda_stream

    def _shape(self, name):
        c = self.cfg
        return {"X": (c.batch, c.seq, c.d_model), "dY": (c.batch, c.seq, c.d_model), "Y": (c.batch, c.seq, c.d_model),
                "dX": (c.batch, c.seq, c.d_model), "Wq": (c.d_model, c.d_q), "Wk": (c.d_model, c.d_kv),
                "Wv": (c.d_model, c.d_kv), "Wo": (c.d_q, c.d_model), "dWq": (c.d_model, c.d_q),
                "dWk": (c.d_model, c.d_kv), "dWv": (c.d_model, c.d_kv), "dWo": (c.d_q, c.d_model)}[name]

    def to_device_rowmajor(self, arr):
        """numpy float64/float32 array of storage-representable values -> torch tensor in the storage dtype."""
        t = self.torch.from_numpy(arr.astype("float32"))
        return t.to(self.dev).to(self.tdtype).contiguous()

    def load_inputs(self, inp):
        """Pack the row-major inputs of ``fbl_inputs.make_inputs`` into R-Tile device buffers."""
        for name, tid in self.MATS.items():
            rm = self.to_device_rowmajor(inp[name])
            self.plan.pack(TENSOR[tid], rm.data_ptr(), self.buf[name].data_ptr(), self._stream())
        for name in ("gamma", "beta", "bq", "bk", "bv", "bo"):
            if inp.get(name) is not None:
                self.vec[name].copy_(self.torch.from_numpy(inp[name].astype("float32")))
        self.torch.cuda.synchronize(self.dev)

    def forward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        bias = c.has_bias
        self.plan.layer_fwd(ptr(b["X"]), ptr(v["gamma"]), ptr(v["beta"]) if c.norm == "layernorm" else None,
                            ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]), ptr(b["Wo"]),
                            ptr(v["bq"]) if bias else None, ptr(v["bk"]) if bias else None,
                            ptr(v["bv"]) if bias else None, ptr(v["bo"]) if bias else None,
                            ptr(b["Y"]), ptr(self.saved), ptr(self.scratch_fwd), self._stream())

    def backward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        bias = c.has_bias
        self.plan.layer_bwd(ptr(b["dY"]), ptr(b["X"]), ptr(v["gamma"]), ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]),
                            ptr(b["Wo"]), ptr(self.saved), ptr(b["dX"]), ptr(b["dWq"]), ptr(b["dWk"]), ptr(b["dWv"]),
                            ptr(b["dWo"]), ptr(v["dbq"]) if bias else None, ptr(v["dbk"]) if bias else None,
                            ptr(v["dbv"]) if bias else None, ptr(v["dbo"]) if bias else None, ptr(v["dgamma"]),
                            ptr(v["dbeta"]) if c.norm == "layernorm" else None, ptr(self.scratch), self._stream())

    def step(self):
        self.forward()
        self.backward()

    def fetch(self, name):
        """Unpack one output matrix to a row-major float64 numpy array (or copy a vector)."""
        torch = self.torch
        if name in self.OUT_MATS:
            shape = self._shape(name)
            out = torch.empty(shape, dtype=self.tdtype, device=self.dev)
            self.plan.unpack(TENSOR[self.OUT_MATS[name]], self.buf[name].data_ptr(), out.data_ptr(), self._stream())
            torch.cuda.synchronize(self.dev)
            return out.float().cpu().numpy().astype("float64")
        torch.cuda.synchronize(self.dev)
        return self.vec[name].cpu().numpy().astype("float64")

    # intermediates: name -> (workspace id, tensor id whose shape it has, last logical dimension)
    INTERMEDIATES = {"Xn": ("XN", "XN", "d_model"), "Q": ("Q", "Q", "d_q"), "K": ("K", "K", "d_kv"),
                     "V": ("V", "K", "d_kv"), "A": ("A", "Q", "d_q"), "dA": ("DA", "Q", "d_q"),
                     "dQ": ("DQ", "Q", "d_q"), "dK": ("DK", "K", "d_kv"), "dV": ("DV", "K", "d_kv"),
                     "dXn": ("DXN", "XN", "d_model")}

    def saved_view(self, name):
        """An intermediate of the last step as a float64 numpy array in its logical shape: the saved forward
        tensors Xn, Q, K, V, A ([B, T, C]), LSE ([B, Hq, T]), stats ([B, T, 2] = mean, rstd), and from the
        backward scratch D ([B, Hq, T]), dA, dQ, dK, dV, dXn ([B, T, C])."""
        torch, c = self.torch, self.cfg
        torch.cuda.synchronize(self.dev)
        t_pad = (c.seq + 7) // 8 * 8
        if name in ("LSE", "D", "stats"):
            off, nbytes = self.plan.workspace_offset(WS[name.upper()])
            src = self.saved if name != "D" else self.scratch
            flat = src[off:off + nbytes].view(torch.float32)
            if name == "stats":
                return flat.view(c.batch, t_pad, 2)[:, :c.seq].cpu().numpy().astype("float64")
            return flat.view(c.batch, c.n_q_heads, t_pad)[:, :, :c.seq].cpu().numpy().astype("float64")
        ws, tid, dim = self.INTERMEDIATES[name]
        off, nbytes = self.plan.workspace_offset(WS[ws])
        src = self.saved if ws in ("XN", "Q", "K", "V", "A") else self.scratch
        rows = getattr(c, "seq_kv", c.seq) if tid == "K" else c.seq
        out = torch.empty((c.batch, rows, getattr(c, dim)), dtype=self.tdtype, device=self.dev)
        self.plan.unpack(TENSOR[tid], src[off:off + nbytes].data_ptr(), out.data_ptr(), self._stream())
        torch.cuda.synchronize(self.dev)
        return out.float().cpu().numpy().astype("float64")

    def guards_intact(self):
        """Names of the buffers whose guard bands were overwritten (empty list: none)."""
        self.torch.cuda.synchronize(self.dev)
        named = {"saved": self.saved, "scratch_fwd": self.scratch_fwd, "scratch_bwd": self.scratch}
        named.update(self.buf)
        named.update(self._vec_raw)
        return [k for k, v in named.items() if not guard_bands_intact(v)]

    def status(self) -> int:
        """Device status of the last forward and backward (0, or the code of the first bounded wait that expired)."""
        self.torch.cuda.synchronize(self.dev)
        fwd = self.plan.status_poll(self.scratch_fwd.data_ptr())
        return fwd if fwd != 0 else self.plan.status_poll(self.scratch.data_ptr())
