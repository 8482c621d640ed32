"""GPU parity of the general N:M masked-dense pruning passes (bit-exact against the oracle)."""
import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si

pytestmark = pytest.mark.gpu

PATTERNS = [(1, 2), (2, 4), (1, 4), (3, 4), (2, 8), (4, 8), (7, 8), (1, 16), (4, 16), (8, 16)]


@pytest.fixture(scope="module")
def B():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24070_b200 import binding, build

    build.build()                     # no-op when libslope.so is newer than its sources
    binding.lib()
    return binding


def _tie_heavy(shape, seed):
    """Few distinct magnitudes, both signs, zeros, and a block of Inf / NaN / denormal patterns."""
    rng = np.random.Generator(np.random.PCG64(seed))
    alphabet = si.f32_to_bf16_bits(np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 1.5, 3.0], np.float32))
    W = rng.choice(alphabet, size=shape).astype(np.uint16)
    special = np.array([0x7F80, 0xFF80, 0x7FC0, 0x0001, 0x8001, 0x7F7F, 0x0080, 0xFFFF], np.uint16)
    W[: shape[0] // 4] = rng.choice(special, size=(shape[0] // 4, shape[1]))
    return W


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("kind", ["gaussian", "ties"])
def test_nm_passes_bit_exact(B, oracle, n, m, kind):
    import torch

    d_out, d_in = 384, 640
    W = si.gaussian_bf16((d_out, d_in), 0.02, 700 + 10 * m + n) if kind == "gaussian" else _tie_heavy((d_out, d_in), 800 + m + n)
    WR_o, mask1_o = oracle.prune_nm(W, n, m)
    WRC_o, mask2_o = oracle.double_prune_nm(W, mask1_o, n, m)
    Wd = B.bf16_from_bits(W)
    WR = torch.empty_like(Wd)
    WRC = torch.empty_like(Wd)
    mask1 = torch.empty((d_out, d_in // 8), dtype=torch.uint8, device="cuda")
    mask2 = torch.empty_like(mask1)
    B.slope_prune_nm(Wd, n, m, WR, mask1)
    B.slope_double_prune_nm(Wd, mask1, n, m, WRC, mask2)
    assert B.slope_poll_status() == 0
    assert np.array_equal(B.bits_from_bf16(WR), WR_o)
    assert np.array_equal(mask1.cpu().numpy(), mask1_o)
    assert np.array_equal(B.bits_from_bf16(WRC), WRC_o)
    assert np.array_equal(mask2.cpu().numpy(), mask2_o)
    # the second pass reads only what the first-pass mask keeps: the pruned matrix gives the same result
    WRC_b = torch.empty_like(Wd)
    B.slope_double_prune_nm(WR, mask1, n, m, WRC_b, None)
    assert np.array_equal(B.bits_from_bf16(WRC_b), WRC_o)
    # in place, masks optional
    Wi = Wd.clone()
    B.slope_prune_nm(Wi, n, m, Wi, None)
    assert np.array_equal(B.bits_from_bf16(Wi), WR_o)
    B.slope_double_prune_nm(Wi, mask1, n, m, Wi, None)
    assert np.array_equal(B.bits_from_bf16(Wi), WRC_o)
    assert B.slope_poll_status() == 0


def test_nm_2_4_agrees_with_the_compressed_path(B, oracle):
    """slope_prune_nm(2, 4) keeps exactly what slope_prune_24 keeps, likewise the second pass."""
    import torch

    d_out, d_in = 256, 512
    W = si.gaussian_bf16((d_out, d_in), 0.02, 77)
    Wd = B.bf16_from_bits(W)
    vals, meta, mask1 = B.alloc_compressed(d_out, d_in)
    B.slope_prune_24(Wd, vals, meta, mask1)
    valsT, metaT, _ = B.alloc_compressed(d_in, d_out)
    mask2 = torch.empty_like(mask1)
    B.slope_double_prune(Wd, mask1, valsT, metaT, mask2)
    WR = torch.empty_like(Wd)
    m1 = torch.empty_like(mask1)
    m2 = torch.empty_like(mask1)
    B.slope_prune_nm(Wd, 2, 4, WR, m1)
    B.slope_double_prune_nm(Wd, m1, 2, 4, WR, m2)
    assert B.slope_poll_status() == 0
    assert torch.equal(m1, mask1) and torch.equal(m2, mask2)


def test_apply_mask_and_lemma1_density(B, oracle):
    """Masked dense gradient, and the extra zeros of Eq. (sparsity_ratio) measured on the GPU result."""
    import math
    import torch

    d = 2048
    n, m = 2, 8
    W = si.gaussian_bf16((d, d), 0.02, 78)
    G = si.gaussian_bf16((d, d), 1.0, 79)
    Wd, Gd = B.bf16_from_bits(W), B.bf16_from_bits(G)
    WR = torch.empty_like(Wd)
    mask1 = torch.empty((d, d // 8), dtype=torch.uint8, device="cuda")
    mask2 = torch.empty_like(mask1)
    B.slope_prune_nm(Wd, n, m, WR, mask1)
    B.slope_double_prune_nm(WR, mask1, n, m, WR, mask2)
    out = torch.empty_like(Gd)
    B.slope_apply_mask(Gd, mask1, out)
    assert B.slope_poll_status() == 0
    k1 = oracle.mask_to_bool(mask1.cpu().numpy(), d)
    k2 = oracle.mask_to_bool(mask2.cpu().numpy(), d)
    assert np.array_equal(B.bits_from_bf16(out), np.where(k1, G, 0).astype(np.uint16))
    s = n / m
    lemma = sum(math.comb(m, j) * s ** j * (1 - s) ** (m - j) * (j - n) / m for j in range(n + 1, m + 1))
    assert abs((k1.mean() - k2.mean()) - lemma) < 1e-3


def test_nm_argument_errors(B):
    import torch

    W = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    for n, m in [(0, 4), (4, 4), (1, 3), (2, 32)]:
        with pytest.raises(B.SlopeError) as e:
            B.slope_prune_nm(W, n, m, W, None)
        assert e.value.status == 2
    assert B.slope_poll_status() == 0


# ------------------------------------------------------------------ dense layer on the same pipeline
def _dense_dw_from_oracle(oracle, dY, X, d_out, d_in):
    """Dense dW = dY^T X from the masked-gradient oracle: the masks "positions 0,1" and "positions 2,3"
    of every group together cover every entry exactly once."""
    lo = np.full((d_out, d_in // 8), 0x33, np.uint8)          # bits 0,1 and 4,5 of every byte
    hi = np.full((d_out, d_in // 8), 0xCC, np.uint8)
    rows = np.arange(d_out)
    a = oracle.dw_rows(dY, X, lo, rows).reshape(d_out, d_in // 4, 2)
    b = oracle.dw_rows(dY, X, hi, rows).reshape(d_out, d_in // 4, 2)
    return np.concatenate([a, b], axis=-1).reshape(d_out, d_in)


@pytest.mark.parametrize("d_in,d_out,b", [(384, 640, 776), (1024, 256, 264), (128, 128, 8), (256, 384, 77), (384, 256, 1)])
def test_dense_layer_against_oracle(B, oracle, d_in, d_out, b):
    import torch
    from helpers import REL_TOL, parity_error, to_f64

    W = si.gaussian_bf16((d_out, d_in), 0.02, 501)
    X = si.gaussian_bf16((b, d_in), 1.0, 502)
    dY = si.gaussian_bf16((b, d_out), 1.0, 503)
    Wd, Xd, dYd = B.bf16_from_bits(W), B.bf16_from_bits(X), B.bf16_from_bits(dY)
    Y = torch.empty((b, d_out), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((b, d_in), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((d_out, d_in), dtype=torch.bfloat16, device="cuda")
    B.slope_dense_linear_fwd(Xd, Wd, Y)
    B.slope_dense_linear_bwd_dx(dYd, Wd, dX)
    B.slope_dense_linear_bwd_dw(dYd, Xd, dW)
    assert B.slope_poll_status() == 0
    full = np.full((d_out, d_in // 8), 0xFF, np.uint8)        # every entry kept: the dense layer
    rows = np.arange(b)
    errs = {
        "Y": parity_error(to_f64(B.bits_from_bf16(Y)), oracle.fwd_rows(X, W, full, rows)),
        "dX": parity_error(to_f64(B.bits_from_bf16(dX)), oracle.dx_rows(dY, W, full, rows)),
        "dW": parity_error(to_f64(B.bits_from_bf16(dW)), _dense_dw_from_oracle(oracle, dY, X, d_out, d_in)),
    }
    print(errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)


def test_emulated_2_8_layer_matches_oracle_on_the_masks(B, oracle):
    """An N:M-emulated layer (2:8): prune, double prune, dense GEMMs on the masked-dense matrices and the
    masked weight gradient, against the oracle evaluated with the same (oracle-made) masks."""
    import torch
    from helpers import REL_TOL, parity_error, to_f64

    n, m, d_in, d_out, b = 2, 8, 512, 384, 264
    W = si.gaussian_bf16((d_out, d_in), 0.02, 511)
    X = si.gaussian_bf16((b, d_in), 1.0, 512)
    dY = si.gaussian_bf16((b, d_out), 1.0, 513)
    _, mask1 = oracle.prune_nm(W, n, m)
    _, mask2 = oracle.double_prune_nm(W, mask1, n, m)
    Wd, Xd, dYd = B.bf16_from_bits(W), B.bf16_from_bits(X), B.bf16_from_bits(dY)
    WR, WRC = torch.empty_like(Wd), torch.empty_like(Wd)
    m1 = torch.empty((d_out, d_in // 8), dtype=torch.uint8, device="cuda")
    B.slope_prune_nm(Wd, n, m, WR, m1)
    B.slope_double_prune_nm(WR, m1, n, m, WRC, None)
    Y = torch.empty((b, d_out), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((b, d_in), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((d_out, d_in), dtype=torch.bfloat16, device="cuda")
    B.slope_dense_linear_fwd(Xd, WR, Y)
    B.slope_dense_linear_bwd_dx(dYd, WRC, dX)
    B.slope_dense_linear_bwd_dw(dYd, Xd, dW)
    B.slope_apply_mask(dW, m1, dW)
    assert B.slope_poll_status() == 0
    assert np.array_equal(m1.cpu().numpy(), mask1)
    rows = np.arange(b)
    keep1 = oracle.mask_to_bool(mask1, d_in)
    want_dW = np.where(keep1, _dense_dw_from_oracle(oracle, dY, X, d_out, d_in), 0.0)
    errs = {
        "Y": parity_error(to_f64(B.bits_from_bf16(Y)), oracle.fwd_rows(X, W, mask1, rows)),
        "dX": parity_error(to_f64(B.bits_from_bf16(dX)), oracle.dx_rows(dY, W, mask2, rows)),
        "dW": parity_error(to_f64(B.bits_from_bf16(dW)), want_dW),
    }
    print(errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)
    got = B.bits_from_bf16(dW)
    assert not np.any(got[~keep1] & 0x7FFF)                   # exact zeros outside the mask


def test_mask_difference_of_re_selected_masks(B, oracle):
    """A dense weight drifts for a few "steps"; its 2:4 mask is re-selected every step (the dynamic-mask
    variant) and compared with the last one: the GPU count equals the oracle's on the oracle's masks."""
    import torch

    d_out, d_in = 512, 1024
    W0 = si.gaussian_bf16((d_out, d_in), 0.02, 601)
    masks_o, masks_g = [], []
    count = torch.zeros(1, dtype=torch.int64, device="cuda")
    for step in range(4):
        drift = si.gaussian_bf16((d_out, d_in), 0.004 * step, 610 + step)
        W = si.f32_to_bf16_bits((W0.astype(np.uint32) << 16).view(np.float32) + (drift.astype(np.uint32) << 16).view(np.float32))
        _, m_o = oracle.prune_nm(W, 2, 4)
        Wd = B.bf16_from_bits(W)
        m_g = torch.empty((d_out, d_in // 8), dtype=torch.uint8, device="cuda")
        B.slope_prune_nm(Wd, 2, 4, Wd, m_g)
        assert np.array_equal(m_g.cpu().numpy(), m_o)
        masks_o.append(m_o)
        masks_g.append(m_g)
    for step in range(4):
        B.slope_mask_difference(masks_g[step], masks_g[-1], count)
        assert B.slope_poll_status() == 0
        assert int(count.item()) == oracle.mask_difference(masks_o[step], masks_o[-1])
    assert oracle.mask_difference(masks_o[0], masks_o[-1]) > 0
