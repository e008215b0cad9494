"""Element-by-element permutation test of pack/unpack on the device against the layout oracle."""
import numpy as np
import pytest

from fbl_inputs import LayerConfig
from oracle import layout as lo
from paper_2607_21624_b200 import TENSOR, LayerRunner

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,T,D,hq,hkv,hd", [("bf16", 197, 128, 2, 1, 64), ("fp32", 21, 64, 2, 2, 32),
                                                ("bf16", 8, 256, 2, 2, 128)])
def test_pack_is_the_oracle_permutation_and_unpack_inverts_it(dtype, T, D, hq, hkv, hd):
    import torch
    cfg = LayerConfig("p", 3, T, D, hq, hkv, hd, dtype, "layernorm", False, False, False, 1e-5, 0, 0.02)
    run = LayerRunner(cfg)
    tw = 64 if dtype == "bf16" else 32
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    ity = torch.int16 if dtype == "bf16" else torch.int32
    for name, shape, tok in (("X", (3, T, D), True), ("WQ", (D, hq * hd), False), ("WO", (hq * hd, D), False)):
        n = int(np.prod(shape))
        ids = (np.arange(n) % 30011 + 1).astype(np.int32).reshape(shape)      # distinct-ish non-zero bit patterns
        host = torch.from_numpy(ids).to(ity).cuda()
        nbytes = run.plan.tensor_bytes(TENSOR[name])
        tiled = torch.full((nbytes // host.element_size(),), -1, dtype=ity, device="cuda")
        run.plan.pack(TENSOR[name], host.view(tdt).data_ptr(), tiled.view(tdt).data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        want = lo.pack_tokens(ids, 8, tw, fill=0) if tok else lo.pack_matrix(ids, 8, tw, fill=0)
        assert np.array_equal(tiled.cpu().numpy().astype(np.int32), want)          # pad slots are zero, rest bit-exact
        back = torch.zeros_like(host)
        run.plan.unpack(TENSOR[name], tiled.view(tdt).data_ptr(), back.view(tdt).data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert torch.equal(back, host)
