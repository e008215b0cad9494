"""ctypes binding of the adapter entry points (fbl_*lora*): argument marshalling only."""
from __future__ import annotations

import ctypes as C

from .binding import LayerRunner, _check, aligned_bytes, lib

ADAPTER = {"Aq": 0, "Ak": 1, "Av": 2, "Bq": 3, "Bk": 4, "Bv": 5}


class LoraRunner(LayerRunner):
    """LayerRunner for a layer with rank-``rank`` adapters on Q, K, V and frozen base weights."""

    def __init__(self, cfg, rank, device="cuda:0", guard_bytes=0, tile_choices=None):
        L = lib()
        vp, sz = C.c_void_p, C.c_size_t
        L.fbl_plan_enable_lora.argtypes = [vp, C.c_int]
        L.fbl_lora_bytes.argtypes = [vp, C.POINTER(sz), C.POINTER(sz)]
        L.fbl_lora_pack.argtypes = [vp, C.c_int, vp, vp, vp]
        L.fbl_lora_unpack.argtypes = [vp, C.c_int, vp, vp, vp]
        L.fbl_layer_fwd_lora.argtypes = [vp] * 18
        L.fbl_layer_bwd_lora.argtypes = [vp] * 18
        self.rank = rank
        self._guard = guard_bytes
        super().__init__(cfg, device=device, guard_bytes=guard_bytes, tile_choices=tile_choices, _before_sizes=self._enable)
        a, b = sz(), sz()
        _check(L.fbl_lora_bytes(self.plan._h, C.byref(a), C.byref(b)))
        al = lambda n: aligned_bytes(self.torch, n, self.dev, guard=guard_bytes)
        self.buf.update(A_all=al(a.value), B_all=al(b.value), dA_all=al(a.value), dB_all=al(b.value))

    def _enable(self, plan):
        _check(lib().fbl_plan_enable_lora(plan._h, self.rank))

    def _adapter_shape(self, name):
        c = self.cfg
        cols = {"q": c.d_q, "k": c.d_kv, "v": c.d_kv}[name[-1]]
        return (c.d_model, self.rank) if name[-2] == "A" else (self.rank, cols)

    def load_inputs(self, inp):
        super().load_inputs(inp)
        self.buf["A_all"].zero_()
        self.buf["B_all"].zero_()
        for name, which in ADAPTER.items():
            rm = self.to_device_rowmajor(inp[name])
            _check(lib().fbl_lora_pack(self.plan._h, which, rm.data_ptr(), self.buf[name[0] + "_all"].data_ptr(), self._stream()))
        self.torch.cuda.synchronize(self.dev)

    def forward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        bias = c.has_bias
        _check(lib().fbl_layer_fwd_lora(
            self.plan._h, ptr(b["X"]), ptr(v["gamma"]), ptr(v["beta"]) if c.norm == "layernorm" else None,
            ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]), ptr(b["Wo"]),
            ptr(v["bq"]) if bias else None, ptr(v["bk"]) if bias else None, ptr(v["bv"]) if bias else None,
            ptr(v["bo"]) if bias else None, ptr(b["A_all"]), ptr(b["B_all"]), ptr(b["Y"]), ptr(self.saved),
            ptr(self.scratch_fwd), self._stream()))

    def backward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        _check(lib().fbl_layer_bwd_lora(
            self.plan._h, ptr(b["dY"]), ptr(b["X"]), ptr(v["gamma"]), ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]), ptr(b["Wo"]),
            ptr(b["A_all"]), ptr(b["B_all"]), ptr(self.saved), ptr(b["dX"]), ptr(b["dA_all"]), ptr(b["dB_all"]),
            None, None, ptr(self.scratch), self._stream()))

    def fetch(self, name):
        if name[1:] in ADAPTER and name[0] == "d":
            torch = self.torch
            out = torch.empty(self._adapter_shape(name), dtype=self.tdtype, device=self.dev)
            _check(lib().fbl_lora_unpack(self.plan._h, ADAPTER[name[1:]], self.buf["d" + name[1] + "_all"].data_ptr(),
                                         out.data_ptr(), self._stream()))
            torch.cuda.synchronize(self.dev)
            return out.float().cpu().numpy().astype("float64")
        return super().fetch(name)
