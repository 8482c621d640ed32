"""GPU parity of the optimizer tail of Algorithm 1 (sparseAdd, updateSparseMatrix)."""
import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si
from helpers import GpuLayer, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24070_b200 import binding, build

    build.build()                     # no-op when libslope.so is newer than its sources
    binding.lib()
    return binding


def bf16_round(x64):
    """fp64 -> nearest bf16 (ties to even), as float64."""
    return to_f64(si.f32_to_bf16_bits(x64.astype(np.float32)))


@pytest.mark.parametrize("rows,cols", [(512, 512), (384, 1152), (11008, 4096)])
def test_sparse_add(B, oracle, rows, cols):
    import torch

    A = si.gaussian_bf16((rows, cols // 2), 1.0, 51)
    Bv = si.gaussian_bf16((rows, cols // 2), 0.02, 52)
    beta, gamma = 1.0 / 1024.0, 0.01
    out = torch.empty((rows, cols // 2), dtype=torch.bfloat16, device="cuda")
    B.slope_sparse_add(B.bf16_from_bits(A), B.bf16_from_bits(Bv), beta, gamma, out)
    assert B.slope_poll_status() == 0
    got = to_f64(B.bits_from_bf16(out))
    ref = oracle.sparse_add(A, Bv, np.float32(beta), np.float32(gamma))
    # the kernel rounds twice (fp32 arithmetic, then bf16): allow one bf16 ulp on ties, plus the fp32
    # rounding of gamma * b where the two terms cancel (seen among 22 million elements, not among thousands)
    ulp = np.abs(ref) * 2.0 ** -7 + np.abs(np.float64(np.float32(gamma)) * to_f64(Bv)) * 2.0 ** -22
    assert (np.abs(got - ref) <= ulp).all()
    assert (got == bf16_round(ref)).mean() > 0.999
    # identity: 1*A + 0*B is a bit copy
    B.slope_sparse_add(B.bf16_from_bits(A), B.bf16_from_bits(Bv), 1.0, 0.0, out)
    assert np.array_equal(B.bits_from_bf16(out), A)


@pytest.mark.parametrize("d_out,d_in", [(512, 512), (384, 640), (1280, 128), (11008, 4096), (4096, 11008)])
def test_update_sparse_matrix(B, oracle, d_out, d_in):
    import torch

    W = si.gaussian_bf16((d_out, d_in), 0.02, 53)
    layer = GpuLayer(W)
    vals, nib, mask1 = oracle.prune24(W)
    valsT, nibT, mask2 = oracle.double_prune(W, mask1)
    new_vals = si.gaussian_bf16(vals.shape, 0.02, 54)              # what an optimizer step would write
    out = torch.empty_like(layer.WTc_vals)
    B.slope_update_sparse_matrix(B.bf16_from_bits(new_vals), layer.mask1, layer.WTc_meta, out)
    assert B.slope_poll_status() == 0
    assert np.array_equal(B.bits_from_bf16(out), oracle.update_transposed(new_vals, mask1, mask2, nibT))
    # unchanged values reproduce the second pruning pass bit for bit
    B.slope_update_sparse_matrix(layer.Wc_vals, layer.mask1, layer.WTc_meta, out)
    assert np.array_equal(B.bits_from_bf16(out), valsT)
