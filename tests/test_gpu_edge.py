"""Edge cases of the layer step on the GPU: degenerate shapes, refusals at the C boundary, repeatability."""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, make_inputs
from tests.test_gpu_layer import run_and_compare

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [
    # one token per sequence: softmax over a single key (P = 1, dS = 0), every tile a ragged tail
    LayerConfig("e1", 3, 1, 128, 2, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 41, 0.02),
    LayerConfig("e2", 2, 1, 64, 2, 1, 32, "fp32", "rmsnorm", False, False, False, 1e-5, 42, 0.02),
    # sequence one short of / one past a 128-row tile, many sequences: tile tails at both ends
    LayerConfig("e3", 5, 127, 256, 4, 4, 64, "bf16", "rmsnorm", True, False, True, 1e-5, 43, 0.02),
    LayerConfig("e4", 5, 129, 256, 2, 1, 128, "bf16", "layernorm", False, True, False, 1e-6, 44, 0.02),
], ids=lambda c: c.name)
def test_degenerate_and_tail_shapes(cfg):
    run_and_compare(cfg, affine_noise=True)


def test_single_token_closed_form():
    # T = 1: attention is the identity on V, so Y = (Xn Wv + bv) Wo + bo (+ X) whatever Q and K are
    from oracle.layer import layer_fwd_bwd
    cfg = LayerConfig("e5", 4, 1, 128, 2, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 45, 0.02)
    inp = make_inputs(cfg, affine_noise=True)
    run = run_and_compare(cfg, affine_noise=True)
    got = run.fetch("Y")
    x = inp["X"][:, 0, :]
    mu = x.mean(-1, keepdims=True)
    xn = (x - mu) / np.sqrt(((x - mu) ** 2).mean(-1, keepdims=True) + cfg.eps) * inp["gamma"] + inp["beta"]
    y = (xn @ inp["Wv"] + inp["bv"]) @ inp["Wo"] + inp["bo"] + x
    assert np.abs(got[:, 0, :] - y).max() <= 1e-2 + 2e-2 * np.abs(y).max()


def test_boundary_refuses_bad_arguments_without_touching_the_device():
    import torch
    from paper_2607_21624_b200 import LayerRunner
    from paper_2607_21624_b200.binding import FblError
    cfg = LayerConfig("e6", 1, 64, 128, 2, 2, 64, "bf16", "layernorm", True, False, False, 1e-5, 46, 0.02)
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg))
    good = run.buf["X"]
    # a matrix pointer that is not 1024-byte aligned
    run.buf["X"] = good[16:]
    with pytest.raises(FblError):
        run.forward()
    run.buf["X"] = good
    # a required vector missing
    gamma = run.vec["gamma"]
    class Null:
        def data_ptr(self):
            return None
    run.vec["gamma"] = Null()
    with pytest.raises(FblError):
        run.forward()
    run.vec["gamma"] = gamma
    run.step()
    assert run.status() == 0
    torch.cuda.synchronize()


def test_two_steps_give_identical_bits_except_dq_order():
    # Everything except the fp32 dQ accumulation (bulk reductions arrive in any order) is order-free; dX, dWq depend
    # on dQ, so they may differ in the last bf16 bit between runs.  Y, dWo, dgamma of the forward-only chain must not.
    from paper_2607_21624_b200 import LayerRunner
    cfg = LayerConfig("e7", 2, 300, 256, 4, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 47, 0.02)
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg, affine_noise=True))
    run.step()
    a = {n: run.fetch(n) for n in ("Y", "dWo", "dbo", "dWv", "dbv")}
    run.step()
    for n, v in a.items():
        assert np.array_equal(v, run.fetch(n)), n


@pytest.mark.parametrize("cfg", [
    LayerConfig("e8", 1, 333, 256, 4, 1, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 48, 0.02),
    LayerConfig("e9", 3, 197, 256, 2, 2, 128, "bf16", "layernorm", False, True, True, 1e-5, 49, 0.02),
], ids=lambda c: c.name)
def test_step_does_not_depend_on_previous_buffer_contents(cfg):
    # `saved` and `scratch` are the caller's memory and arrive holding anything.  The step must establish every
    # value it later reads (zero-filled accumulators, padding rows, the rows of LSE and D that a 128-row copy window
    # takes in beyond the sequence end), and a kernel that requests forward-pass data before waiting for its
    # predecessor must still find the forward pass complete.  Filled with zeros, with NaN bit patterns and with
    # huge finite values before a forward + backward issued back to back, the order-free outputs are identical
    # bit for bit and the others stay within the usual bound of the oracle.
    from paper_2607_21624_b200 import LayerRunner
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg, affine_noise=True))
    names = ("Y", "dWo", "dWk", "dWv")
    ref = None
    for fill in (0x00, 0xFF, 0x7F):
        run.scratch.fill_(fill)
        run.scratch_fwd.fill_(fill)
        run.saved.fill_(fill)
        run.step()
        assert run.status() == 0
        got = {n: run.fetch(n) for n in names + ("dX", "dWq")}
        for n, v in got.items():
            assert np.isfinite(v).all(), (n, hex(fill))
        if ref is None:
            ref = got
            continue
        for n in names:
            assert np.array_equal(ref[n], got[n]), (n, hex(fill))
        for n in ("dX", "dWq"):                       # downstream of the dQ accumulation, whose order is free
            assert np.abs(ref[n] - got[n]).max() <= 2e-2 * np.abs(ref[n]).max() + 1e-6, (n, hex(fill))


@pytest.mark.parametrize("cfg", [
    LayerConfig("e10", 2, 300, 256, 4, 2, 64, "bf16", "layernorm", True, True, True, 1e-5, 56, 0.02),
    LayerConfig("e11", 4, 512, 768, 12, 12, 64, "bf16", "layernorm", True, True, False, 1e-5, 57, 0.02),
    LayerConfig("e12", 1, 640, 512, 4, 4, 128, "bf16", "rmsnorm", True, False, True, 1e-5, 58, 0.02),
], ids=lambda c: c.name)
def test_many_back_to_back_steps_are_identical(cfg):
    # Forty forward + backward passes enqueued without any host synchronisation in between: every kernel is launched
    # so that it may start while its predecessor drains, across the boundary between steps too.  Whatever one step
    # leaves behind (accumulators, staging areas, barriers' worth of in-flight copies) must not reach the next: the
    # order-free outputs of the last step equal those of a lone first step bit for bit.
    import torch
    from paper_2607_21624_b200 import LayerRunner
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg, affine_noise=True))
    names = ("Y", "dWo", "dWk", "dWv")
    run.step()
    torch.cuda.synchronize()
    first = {n: run.fetch(n) for n in names + ("dX", "dWq")}
    for _ in range(40):
        run.step()
    torch.cuda.synchronize()
    assert run.status() == 0
    for n in names:
        assert np.array_equal(first[n], run.fetch(n)), n
    for n in ("dX", "dWq"):
        assert np.abs(first[n] - run.fetch(n)).max() <= 2e-2 * np.abs(first[n]).max() + 1e-6, n


def test_bounded_wait_expires_and_the_context_stays_usable():
    # Failure detection: every barrier wait in the tensor-core kernels is bounded.  The self-test kernel waits,
    # through the same code, on a barrier that nothing signals, with a bound of 2e5 clock cycles (about 0.1 ms).  The
    # wait must run out, the kernel must return normally, the status word must carry the wait's code, and a normal
    # step on the same context must then run and report no error.
    import torch
    from paper_2607_21624_b200 import LayerRunner, aligned_bytes, lib, selftest_wait_timeout
    cfg = LayerConfig("e13", 2, 300, 256, 4, 2, 64, "bf16", "layernorm", True, True, False, 1e-5, 61, 0.02)
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg, affine_noise=True))
    scratch = aligned_bytes(torch, 1024, run.dev)
    scratch.fill_(0xFF)
    selftest_wait_timeout(scratch.data_ptr(), 200_000, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    import ctypes
    word = ctypes.c_int32()
    rc = lib().fbl_status_poll(run.plan._h, scratch.data_ptr(), ctypes.byref(word))
    assert rc == -6 and word.value == 901, (rc, word.value)            # FBL_ERR_TIMEOUT, the self-test's wait code
    assert int(scratch.view(torch.int32)[1].item()) == 1               # the block reached its normal end
    assert lib().fbl_strerror(rc).decode() == "a bounded device-side wait expired"
    run.step()
    assert run.status() == 0
    ref = run.fetch("Y")
    run.step()
    assert run.status() == 0 and np.array_equal(ref, run.fetch("Y"))


def test_forward_timeout_code_survives_the_backward():
    # Each pass clears the status word of its own scratch, so a code left in the forward's scratch is still visible
    # after a backward has been enqueued behind it.
    import torch
    from paper_2607_21624_b200 import LayerRunner, selftest_wait_timeout
    cfg = LayerConfig("e14", 1, 200, 128, 2, 2, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 62, 0.02)
    run = LayerRunner(cfg)
    run.load_inputs(make_inputs(cfg))
    run.forward()
    selftest_wait_timeout(run.scratch_fwd.data_ptr(), 100_000, torch.cuda.current_stream().cuda_stream)
    run.backward()
    assert run.status() == 901
    run.step()
    assert run.status() == 0


def test_offline_tile_choices_sweep_and_apply():
    # The profiling step of the tile chooser on a small layer: every GEMM launch is timed under every configuration
    # (tile width 128 / 256, CTA pair, one or two sets of epilogue warps), Eq. 2 picks one per launch, and a step
    # under the picked table, and under each forced configuration, still matches the oracle.
    from paper_2607_21624_b200 import rtile
    cfg = LayerConfig("t1", 3, 333, 512, 8, 4, 64, "bf16", "layernorm", True, True, True, 1e-5, 63, 0.02)
    res = rtile.sweep(cfg, reps=2)[(0, 0)]
    picked, detail = rtile.choose(cfg, res)
    assert set(picked) == set(rtile.LAUNCHES)
    for name in rtile.LAUNCHES:
        assert len(res[name]) == len(rtile.legal_choices(cfg)) and all(ms > 0 for ms in res[name].values())
    import paper_2607_21624_b200.binding as binding
    for table in [picked] + [{n: list(c) for n in rtile.LAUNCHES} for c in rtile.legal_choices(cfg)]:
        orig = binding.LayerRunner.__init__

        def patched(self, cfg_, device="cuda:0", guard_bytes=0, tile_choices=None, _t=table):
            orig(self, cfg_, device=device, guard_bytes=guard_bytes, tile_choices=_t)
        binding.LayerRunner.__init__ = patched
        try:
            run = run_and_compare(cfg, affine_noise=True, intermediates=False)
            assert run.tile_choices == table
        finally:
            binding.LayerRunner.__init__ = orig
