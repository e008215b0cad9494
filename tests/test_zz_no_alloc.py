"""fbl_colsum_noalloc: the column-sum entry point for callers that cannot allocate device memory
(allocator hooks, out-of-memory handlers, plugins handed only their inputs and outputs).

It must give what fbl_colsum gives, call after call, although every call reuses one fixed array inside
the library.  This file is collected last on purpose: it also has to pass after every other test has
used the device, and alone in a fresh process.
"""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, normal_f64
from paper_2607_21624_b200 import FblError, Plan, aligned_bytes, desc_from_config

from util import FP32_REL, fp32_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tw", [("bf16", 64), ("fp32", 32)])
def test_noalloc_colsum_matches_colsum_on_two_calls_in_a_row(dtype, tw):
    import torch
    cfg = LayerConfig("z", 1, 64, 128, 2, 2, 64, dtype, "layernorm", False, False, False, 1e-5, 0, 0.02)
    plan = Plan(desc_from_config(cfg))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    stream = torch.cuda.current_stream().cuda_stream
    # two different problems back to back: the second is smaller, so stale partials of the first stay in the array
    for call, (rows, cols) in enumerate([(1000, 4 * tw), (264, 2 * tw)]):
        vals = normal_f64(5 + call, 0, 0, rows * cols).astype(np.float32)
        src = torch.from_numpy(vals).cuda().to(tdt).contiguous()        # any values serve: the sum is over tile rows
        M = aligned_bytes(torch, src.numel() * src.element_size(), "cuda").view(tdt)
        M.copy_(src)
        scratch = torch.empty(plan.colsum_scratch_bytes(rows, cols), dtype=torch.uint8, device="cuda")
        want = torch.full((cols,), float("nan"), device="cuda")
        got = torch.full((cols,), float("nan"), device="cuda")
        plan.colsum(M.data_ptr(), rows, cols, want.data_ptr(), scratch.data_ptr(), stream)
        plan.colsum_noalloc(M.data_ptr(), rows, cols, got.data_ptr(), stream)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert fp32_err(g, w) <= FP32_REL
        # and both agree with a plain sum over the tiled buffer's rows
        ref = M.float().view(cols // tw, rows, tw).sum(dim=1).reshape(-1).cpu().numpy().astype(np.float64)
        assert fp32_err(g, ref) <= FP32_REL


def test_noalloc_colsum_refuses_sizes_beyond_its_fixed_area():
    import torch
    cfg = LayerConfig("z", 1, 64, 128, 2, 2, 64, "bf16", "layernorm", False, False, False, 1e-5, 0, 0.02)
    plan = Plan(desc_from_config(cfg))
    M = aligned_bytes(torch, 2048, "cuda").view(torch.bfloat16)
    out = torch.zeros(8192, device="cuda")
    with pytest.raises(FblError) as e:
        plan.colsum_noalloc(M.data_ptr(), 256 * 40, 8192, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert e.value.code == -4
