"""ctypes binding of the cross-attention entry points (fbl_xattn_*): argument marshalling only."""
from __future__ import annotations

import ctypes as C

from .binding import LayerRunner, Plan, _check, desc_from_config, lib


class XattnRunner(LayerRunner):
    """LayerRunner for a cross-attention layer: ``cfg`` is an ``XattnConfig`` (query side seq / d_model, memory side
    seq_kv / d_mem); buffers gain the memory ``M`` and its gradient ``dM``."""

    MATS = {**LayerRunner.MATS, "M": "MEM"}
    OUT_MATS = {**LayerRunner.OUT_MATS, "dM": "DMEM"}

    def __init__(self, cfg, device="cuda:0", guard_bytes=0):
        L = lib()
        L.fbl_xattn_fwd.argtypes = [C.c_void_p] * 17
        L.fbl_xattn_bwd.argtypes = [C.c_void_p] * 24
        super().__init__(cfg, device=device, guard_bytes=guard_bytes, tile_choices={})

    def _make_plan(self, cfg):
        return Plan(desc_from_config(cfg), cross=(cfg.seq_kv, cfg.d_mem))

    def _shape(self, name):
        c = self.cfg
        mem = {"M": (c.batch, c.seq_kv, c.d_mem), "dM": (c.batch, c.seq_kv, c.d_mem), "Wk": (c.d_mem, c.d_kv),
               "Wv": (c.d_mem, c.d_kv), "dWk": (c.d_mem, c.d_kv), "dWv": (c.d_mem, c.d_kv)}
        return mem[name] if name in mem else super()._shape(name)

    def forward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        bias = c.has_bias
        _check(lib().fbl_xattn_fwd(
            self.plan._h, ptr(b["X"]), ptr(b["M"]), ptr(v["gamma"]), ptr(v["beta"]) if c.norm == "layernorm" else None,
            ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]), ptr(b["Wo"]),
            ptr(v["bq"]) if bias else None, ptr(v["bk"]) if bias else None, ptr(v["bv"]) if bias else None,
            ptr(v["bo"]) if bias else None, ptr(b["Y"]), ptr(self.saved), ptr(self.scratch_fwd), self._stream()))

    def backward(self):
        c, b, v = self.cfg, self.buf, self.vec
        ptr = lambda t: t.data_ptr()
        bias = c.has_bias
        _check(lib().fbl_xattn_bwd(
            self.plan._h, ptr(b["dY"]), ptr(b["X"]), ptr(b["M"]), ptr(v["gamma"]), ptr(b["Wq"]), ptr(b["Wk"]), ptr(b["Wv"]),
            ptr(b["Wo"]), ptr(self.saved), ptr(b["dX"]), ptr(b["dM"]), ptr(b["dWq"]), ptr(b["dWk"]), ptr(b["dWv"]),
            ptr(b["dWo"]), ptr(v["dbq"]) if bias else None, ptr(v["dbk"]) if bias else None,
            ptr(v["dbv"]) if bias else None, ptr(v["dbo"]) if bias else None, ptr(v["dgamma"]),
            ptr(v["dbeta"]) if c.norm == "layernorm" else None, ptr(self.scratch), self._stream()))
