"""The projection kernel on its own, against the CPU oracle's matrix-vector product."""
import numpy as np
import pytest

from oracle import model as OM
from workloads import bf16_bits_from_f32, f32_from_bf16_bits

pytestmark = pytest.mark.gpu


def _case(n_out, k_in, seed):
    rng = np.random.default_rng(seed)
    W = bf16_bits_from_f32((rng.standard_normal((n_out, k_in)) * 0.05).astype(np.float32))
    a = bf16_bits_from_f32(rng.standard_normal((32, k_in)).astype(np.float32))
    return W, a


def _to_dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


# shapes: one tile; several tiles with a ragged last one; k split over several CTAs; wide k
@pytest.mark.parametrize("n_out,k_in", [(128, 64), (200, 256), (1000, 1024), (512, 2816), (4096, 4096)])
def test_gemm_rows32_matches_oracle(n_out, k_in):
    import torch
    from paper_2304_04487_b200 import llma_gemm_rows32_bf16
    W, a = _case(n_out, k_in, seed=n_out + k_in)
    out = torch.full((32, n_out), float("nan"), device="cuda", dtype=torch.float32)
    llma_gemm_rows32_bf16(_to_dev(W), _to_dev(a), out)
    got = out.cpu().numpy()
    af = f32_from_bf16_bits(a)
    rows = range(32) if n_out * k_in <= 1 << 21 else (0, 7, 31)       # sampled rows at the large sizes
    for r in rows:
        want = OM.matvec(W, af[r])
        # fp32 accumulation of k_in products of magnitude ~0.05: error far below 1e-4 of the row's scale
        assert np.abs(got[r] - want).max() <= 1e-4 * max(1.0, np.abs(want).max()), (r, np.abs(got[r] - want).max())
    assert np.isfinite(got).all()
    # same bits on a second run (fixed summation order over the CTAs that share a tile)
    out2 = torch.empty_like(out)
    llma_gemm_rows32_bf16(_to_dev(W), _to_dev(a), out2)
    assert torch.equal(out, out2)


def test_gemm_rejects_bad_arguments():
    import torch
    from paper_2304_04487_b200 import LlmaError, lib
    W, a = _case(128, 64, 0)
    Wd, ad = _to_dev(W), _to_dev(a)
    out = torch.empty((32, 128), device="cuda")
    L = lib()
    assert L.llma_gemm_rows32_bf16(None, ad.data_ptr(), out.data_ptr(), 128, 64, None) == -1
    assert L.llma_gemm_rows32_bf16(Wd.data_ptr(), ad.data_ptr(), out.data_ptr(), 128, 96, None) == -9
    assert L.llma_gemm_rows32_bf16(Wd.data_ptr(), ad.data_ptr(), out.data_ptr(), 0, 64, None) == -9
