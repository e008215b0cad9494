"""ctypes binding of the feed-forward block's entry points (fbl_mlp_*): argument marshalling only."""
from __future__ import annotations

import ctypes as C

from .binding import DTYPES, NORMS, FblError, _check, aligned_bytes, guard_bands_intact, lib

ACTS = {"gelu": 0, "swiglu": 1}
MLP_TENSOR = {"X": 0, "H": 1, "W1": 2, "W2": 3}
MLP_WS = {n: i for i, n in enumerate(["STATS", "XN", "U", "G", "H", "DU", "DG", "DXN"])}


class FblMlpDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "seq", "d_model", "d_ff", "dtype", "norm", "act", "has_bias",
                                         "residual")] + [("eps", C.c_float)]


_bound = False


def _bind():
    global _bound
    L = lib()
    if _bound:
        return L
    vp, sz, i64 = C.c_void_p, C.c_size_t, C.c_int64
    L.fbl_mlp_plan_create.argtypes = [C.POINTER(FblMlpDesc), C.POINTER(vp)]
    L.fbl_mlp_plan_destroy.argtypes = [vp]
    L.fbl_mlp_plan_destroy.restype = None
    L.fbl_mlp_tensor_bytes.argtypes = [vp, C.c_int, C.POINTER(sz)]
    L.fbl_mlp_workspace_bytes.argtypes = [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
    L.fbl_mlp_workspace_offset.argtypes = [vp, C.c_int, C.POINTER(sz), C.POINTER(sz)]
    L.fbl_mlp_pack.argtypes = [vp, C.c_int, vp, vp, vp]
    L.fbl_mlp_unpack.argtypes = [vp, C.c_int, vp, vp, vp]
    L.fbl_mlp_fwd.argtypes = [vp] * 14
    L.fbl_mlp_bwd.argtypes = [vp] * 19
    L.fbl_mlp_status_poll.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    L.fbl_mlp_set_kernel_path.argtypes = [vp, C.c_int]
    L.fbl_mlp_launch_count.argtypes = [vp]
    L.fbl_mlp_launch_count.restype = i64
    _bound = True
    return L


def mlp_desc_from_config(cfg) -> FblMlpDesc:
    return FblMlpDesc(cfg.batch, cfg.seq, cfg.d_model, cfg.d_ff, DTYPES[cfg.dtype], NORMS[cfg.norm], ACTS[cfg.act],
                      int(cfg.has_bias), int(cfg.residual), cfg.eps)


class MlpPlan:
    """One fbl_mlp_plan; methods carry the C entry points' names without the ``fbl_mlp_`` prefix."""

    def __init__(self, desc: FblMlpDesc):
        self._h = C.c_void_p()
        _check(_bind().fbl_mlp_plan_create(C.byref(desc), C.byref(self._h)))

    def close(self):
        if self._h:
            lib().fbl_mlp_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def tensor_bytes(self, matrix_id):
        out = C.c_size_t()
        _check(lib().fbl_mlp_tensor_bytes(self._h, matrix_id, C.byref(out)))
        return out.value

    def workspace_bytes(self):
        a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
        _check(lib().fbl_mlp_workspace_bytes(self._h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def workspace_offset(self, what):
        off, n = C.c_size_t(), C.c_size_t()
        _check(lib().fbl_mlp_workspace_offset(self._h, what, C.byref(off), C.byref(n)))
        return off.value, n.value

    def pack(self, matrix_id, rowmajor_ptr, tiled_ptr, stream):
        _check(lib().fbl_mlp_pack(self._h, matrix_id, rowmajor_ptr, tiled_ptr, stream))

    def unpack(self, matrix_id, tiled_ptr, rowmajor_ptr, stream):
        _check(lib().fbl_mlp_unpack(self._h, matrix_id, tiled_ptr, rowmajor_ptr, stream))

    def fwd(self, *ptrs):
        _check(lib().fbl_mlp_fwd(self._h, *ptrs))

    def bwd(self, *ptrs):
        _check(lib().fbl_mlp_bwd(self._h, *ptrs))

    def set_kernel_path(self, path):
        _check(lib().fbl_mlp_set_kernel_path(self._h, path))

    def launch_count(self):
        return lib().fbl_mlp_launch_count(self._h)

    def status_poll(self, scratch) -> int:
        out = C.c_int32()
        code = lib().fbl_mlp_status_poll(self._h, scratch, C.byref(out))
        if code not in (0, -6):
            _check(code)
        return out.value


class MlpRunner:
    """Device buffers for one feed-forward block plus pack / step / unpack helpers (torch for memory and streams only)."""

    IN_MATS = {"X": "X", "dY": "X", "W1": "W1", "Wg": "W1", "W2": "W2"}
    OUT_MATS = {"Y": "X", "dX": "X", "dW1": "W1", "dWg": "W1", "dW2": "W2"}
    INTERMEDIATES = {"Xn": ("XN", "X"), "U": ("U", "H"), "G": ("G", "H"), "H": ("H", "H"), "dU": ("DU", "H"),
                     "dG": ("DG", "H"), "dXn": ("DXN", "X")}

    def __init__(self, cfg, device="cuda:0", guard_bytes=0):
        import torch
        if not torch.cuda.is_available():
            raise FblError(-101, "no CUDA device: the block has no CPU path")
        self.torch, self.cfg, self.dev = torch, cfg, torch.device(device)
        self.plan = MlpPlan(mlp_desc_from_config(cfg))
        self.tdtype = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
        saved, sf, sb = self.plan.workspace_bytes()
        self.sizes = dict(saved=saved, scratch_fwd=sf, scratch_bwd=sb)
        al = lambda n: aligned_bytes(torch, n, self.dev, guard=guard_bytes)
        self.saved, self.scratch_fwd, self.scratch = al(saved), al(sf), al(sb)
        self.buf = {}
        for name, tid in {**self.IN_MATS, **self.OUT_MATS}.items():
            if name in ("Wg", "dWg") and not cfg.gated:
                continue
            self.buf[name] = al(self.plan.tensor_bytes(MLP_TENSOR[tid]))
        d, f = cfg.d_model, cfg.d_ff
        lens = {"gamma": d, "beta": d, "b1": f, "bg": f, "b2": d, "dgamma": d, "dbeta": d, "db1": f, "dbg": f, "db2": d}
        self._vec_raw = {k: al(4 * n) for k, n in lens.items()}
        self.vec = {k: v.view(torch.float32) for k, v in self._vec_raw.items()}

    def _stream(self):
        return self.torch.cuda.current_stream(self.dev).cuda_stream

    def _shape(self, tid):
        c = self.cfg
        return {"X": (c.batch, c.seq, c.d_model), "H": (c.batch, c.seq, c.d_ff), "W1": (c.d_model, c.d_ff),
                "W2": (c.d_ff, c.d_model)}[tid]

    def to_device_rowmajor(self, arr):
        return self.torch.from_numpy(arr.astype("float32")).to(self.dev).to(self.tdtype).contiguous()

    def load_inputs(self, inp):
        for name, tid in self.IN_MATS.items():
            if name not in self.buf:
                continue
            rm = self.to_device_rowmajor(inp[name])
            self.plan.pack(MLP_TENSOR[tid], rm.data_ptr(), self.buf[name].data_ptr(), self._stream())
        for name in ("gamma", "beta", "b1", "bg", "b2"):
            if inp.get(name) is not None:
                self.vec[name].copy_(self.torch.from_numpy(inp[name].astype("float32")))
        self.torch.cuda.synchronize(self.dev)

    def _p(self, table, name, cond=True):
        return table[name].data_ptr() if cond and name in table else None

    def forward(self):
        c, b, v = self.cfg, self.buf, self.vec
        bias, ln = c.has_bias, c.norm == "layernorm"
        self.plan.fwd(self._p(b, "X"), self._p(v, "gamma"), self._p(v, "beta", ln), self._p(b, "W1"), self._p(b, "Wg"),
                      self._p(b, "W2"), self._p(v, "b1", bias), self._p(v, "bg", bias and c.gated), self._p(v, "b2", bias),
                      self._p(b, "Y"), self.saved.data_ptr(), self.scratch_fwd.data_ptr(), self._stream())

    def backward(self):
        c, b, v = self.cfg, self.buf, self.vec
        bias, ln = c.has_bias, c.norm == "layernorm"
        self.plan.bwd(self._p(b, "dY"), self._p(b, "X"), self._p(v, "gamma"), self._p(b, "W1"), self._p(b, "Wg"),
                      self._p(b, "W2"), self.saved.data_ptr(), self._p(b, "dX"), self._p(b, "dW1"), self._p(b, "dWg"),
                      self._p(b, "dW2"), self._p(v, "db1", bias), self._p(v, "dbg", bias and c.gated), self._p(v, "db2", bias),
                      self._p(v, "dgamma"), self._p(v, "dbeta", ln), self.scratch.data_ptr(), self._stream())

    def step(self):
        self.forward()
        self.backward()

    def fetch(self, name):
        torch = self.torch
        if name in self.OUT_MATS:
            tid = self.OUT_MATS[name]
            out = torch.empty(self._shape(tid), dtype=self.tdtype, device=self.dev)
            self.plan.unpack(MLP_TENSOR[tid], self.buf[name].data_ptr(), out.data_ptr(), self._stream())
            torch.cuda.synchronize(self.dev)
            return out.float().cpu().numpy().astype("float64")
        torch.cuda.synchronize(self.dev)
        return self.vec[name].cpu().numpy().astype("float64")

    def saved_view(self, name):
        """An intermediate of the last step (Xn, U, G, H from `saved`; dU, dG, dXn from the backward scratch) as a
        float64 numpy array in its logical shape."""
        torch = self.torch
        torch.cuda.synchronize(self.dev)
        ws, tid = self.INTERMEDIATES[name]
        off, n = self.plan.workspace_offset(MLP_WS[ws])
        src = self.saved if ws in ("XN", "U", "G", "H") else self.scratch
        out = torch.empty(self._shape(tid), dtype=self.tdtype, device=self.dev)
        self.plan.unpack(MLP_TENSOR[tid], src[off:off + n].data_ptr(), out.data_ptr(), self._stream())
        torch.cuda.synchronize(self.dev)
        return out.float().cpu().numpy().astype("float64")

    def guards_intact(self):
        self.torch.cuda.synchronize(self.dev)
        named = {"saved": self.saved, "scratch_fwd": self.scratch_fwd, "scratch_bwd": self.scratch}
        named.update(self.buf)
        named.update(self._vec_raw)
        return [k for k, v in named.items() if not guard_bands_intact(v)]

    def status(self) -> int:
        self.torch.cuda.synchronize(self.dev)
        fwd = self.plan.status_poll(self.scratch_fwd.data_ptr())
        return fwd if fwd != 0 else self.plan.status_poll(self.scratch.data_ptr())
