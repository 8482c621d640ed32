"""The allocation-free dL entry point (for callers that may not allocate GPU memory and have
no workspace to hand over) against the workspace-based entry point.  Collected last on purpose:
a run that stops at the first failure has then already run every other test."""
import ctypes

import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si
from helpers import REL_TOL, parity_error, rel_fro, to_f64

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


def _reference_dl(B, torch, X, dY, L, R, d_out):
    """dT and dL from the existing entry point (caller-provided workspace)."""
    b, d_in = X.shape
    r = L.shape[1]
    bf = torch.bfloat16
    T = torch.empty((b, r), dtype=bf, device="cuda")
    B.slope_adapter_fwd_bwd(0, X, None, L, None, b, d_out, d_in, r, T=T)
    dT = torch.empty((b, r), dtype=bf, device="cuda")
    dL = torch.empty((d_in, r), dtype=bf, device="cuda")
    dR = torch.empty((r, d_out), dtype=bf, device="cuda")
    ws = torch.empty(B.slope_adapter_workspace_bytes(b, d_out, d_in, r), dtype=torch.uint8, device="cuda")
    B.slope_adapter_fwd_bwd(1, X, dY, L, R, b, d_out, d_in, r, T=T, dT=dT, dL=dL, dR=dR, workspace=ws)
    return dT, dL


@pytest.mark.parametrize("shapes", [((2048, 640, 256, 64), (1024, 384, 128, 32))])
def test_noalloc_dl_matches_workspace_path_on_two_calls_in_a_row(B, oracle, shapes):
    """Two different problems back to back: the second call finds the first call's partial
    sums in the shared fixed array and must not be disturbed by them.  Each result is checked
    against the workspace-based entry point and against the CPU oracle."""
    import torch

    for call, (b, d_in, d_out, r) in enumerate(shapes):
        seed = 900 + 10 * call
        Xb, dYb = si.gaussian_bf16((b, d_in), 1.0, seed), si.gaussian_bf16((b, d_out), 1.0, seed + 1)
        Lb, Rb = si.gaussian_bf16((d_in, r), 0.01, seed + 2), si.gaussian_bf16((r, d_out), 0.01, seed + 3)
        X, dY, L, R = (B.bf16_from_bits(a) for a in (Xb, dYb, Lb, Rb))
        dT, dL_ref = _reference_dl(B, torch, X, dY, L, R, d_out)
        dL = torch.full((d_in, r), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.slope_adapter_dl_noalloc(X, dT, dL)
        assert B.slope_poll_status() == 0
        got, ref = to_f64(B.bits_from_bf16(dL)), to_f64(B.bits_from_bf16(dL_ref))
        assert np.isfinite(got).all()
        err = rel_fro(got, ref)
        assert err <= REL_TOL, (call, err)
        # same kernels, same split order: in fact bit-identical
        assert np.array_equal(B.bits_from_bf16(dL), B.bits_from_bf16(dL_ref))
        # and against the oracle's dL = X^T (dY R^T) (dT kept in fp64 there, bf16 here: two roundings)
        err_o = parity_error(got, oracle.adapter_dL_rows(Xb, dYb, Rb, np.arange(d_in)), roundings=2)
        assert err_o <= REL_TOL, (call, err_o)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch(B):
    import torch

    limit = B.slope_adapter_dl_noalloc_max_scratch_bytes()
    assert limit == 16 << 20
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = ctypes.c_void_p(buf.data_ptr())
    launches = B.slope_launch_count()
    # 16512 x 256 x 4 bytes = 16.9 MB > 16 MiB already for a single split, whatever the split
    # heuristic says: refused before any launch (the pointers are never read)
    assert B.lib().slope_adapter_dl_noalloc(p, p, 16384, 16512, 256, p, None) == 2
    assert B.lib().slope_adapter_dl_noalloc(None, p, 1024, 128, 64, p, None) == 1
    assert B.slope_launch_count() == launches
    assert B.slope_poll_status() == 0
