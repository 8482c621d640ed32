"""GPU parity at the benchmark's full sizes and launch configuration: selection outputs are
compared in full (bit-exact); GEMM outputs on seeded samples of complete output rows, which the
oracle computes one dot product at a time (a sampled sub-tensor is exact)."""
import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si
from helpers import REL_TOL, GpuLayer, check_selection, parity_error, to_f64

pytestmark = pytest.mark.gpu

# every (configuration, layer) pair of the four multi-layer configurations: 3 + 7 + 7 + 7 = 24
CASES = [(key, idx) for key in ("c2_gpt2_small", "c3_llama7b", "c4_llama7b_adapter", "c5_llama13b_block")
         for idx in range(len(si.WORKLOADS[key].layers))]


@pytest.fixture(scope="module")
def B():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24070_b200 import binding, build

    build.build()                     # no-op when libslope.so is newer than its sources
    binding.lib()
    return binding


@pytest.mark.parametrize("key,idx", CASES)
def test_full_size_layer(B, oracle, key, idx):
    import torch

    wl = si.WORKLOADS[key]
    lay = wl.layers[idx]
    b, d_in, d_out, r = wl.tokens, lay.d_in, lay.d_out, wl.rank
    t = si.layer_tensors(wl, idx)
    W, X, dY, L, R = t["W"], t["X"], t["dY"], t.get("L"), t.get("R")
    check_selection(oracle, GpuLayer(W), W)               # the two separate calls
    layer = GpuLayer(W, fused_setup=True)                 # the one-call set-up the benchmark's step uses
    mask1, mask2 = check_selection(oracle, layer, W)
    Xd, dYd = B.bf16_from_bits(X), B.bf16_from_bits(dY)
    if r:
        Ld, Rd = B.bf16_from_bits(L), B.bf16_from_bits(R)
        T = layer.adapter_T(Xd, Ld)
        Y = layer.fwd(Xd, T, Rd)
        dT, dL, dR = layer.adapter_bwd(Xd, dYd, Ld, Rd, T)
        dX = layer.dx(dYd, dT, Ld)
    else:
        Y = layer.fwd(Xd)
        dX = layer.dx(dYd)
    dWc = layer.dw(dYd, Xd)
    layer.poll()

    seed = si.seed_for(wl.config, idx, "X")
    rows = si.sample_indices(b, 64, seed)            # token rows of Y and dX
    orows = si.sample_indices(d_out, 64, seed + 1)   # d_out rows of dWc
    pick = lambda tns, idxs: to_f64(B.bits_from_bf16(tns[torch.as_tensor(idxs, device=tns.device, dtype=torch.long)]))
    errs = {
        "Y": parity_error(pick(Y, rows), oracle.fwd_rows(X, W, mask1, rows, L, R)),
        "dX": parity_error(pick(dX, rows), oracle.dx_rows(dY, W, mask2, rows, L, R)),
        "dWc": parity_error(pick(dWc, orows), oracle.dw_rows(dY, X, mask1, orows)),
    }
    if r:
        jrows = si.sample_indices(d_in, 16, seed + 2)
        icols = si.sample_indices(d_out, 256, seed + 3)
        errs["T"] = parity_error(pick(T, rows), oracle.adapter_T_rows(X, L, rows))
        errs["dT"] = parity_error(pick(dT, rows), oracle.adapter_dT_rows(dY, R, rows))
        errs["dL"] = parity_error(pick(dL, jrows), oracle.adapter_dL_rows(X, dY, R, jrows), roundings=2)
        dR_s = to_f64(B.bits_from_bf16(dR[:, torch.as_tensor(icols, device=dR.device, dtype=torch.long)].contiguous()))
        errs["dR"] = parity_error(dR_s, oracle.adapter_dR_cols(X, L, dY, icols), roundings=2)
    print(key, lay.name, errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)
    # finite everywhere, not just on the sample
    for tns in (Y, dX, dWc):
        assert bool(torch.isfinite(tns.float()).all())


INFERENCE_CASES = [
    ("c4_llama7b_adapter", 0, 8), ("c4_llama7b_adapter", 4, 8), ("c4_llama7b_adapter", 6, 8),
    ("c4_llama7b_adapter", 0, 64), ("c4_llama7b_adapter", 6, 64), ("c5_llama13b_block", 4, 16),
]


@pytest.mark.parametrize("key,idx,tokens", INFERENCE_CASES)
def test_full_size_inference_forward(B, oracle, key, idx, tokens):
    """Forward only at decode sizes on full-size layers (the few-token kernel with its K-split over
    a cluster): every output element against the oracle, without and with the adapters."""
    wl = si.WORKLOADS[key]
    lay = wl.layers[idx]
    t = si.layer_tensors(wl, idx, tokens=tokens)
    W, X, L, R = t["W"], t["X"], t.get("L"), t.get("R")
    layer = GpuLayer(W)
    _, _, mask1 = oracle.prune24(W)
    assert np.array_equal(layer.mask1.cpu().numpy(), mask1)
    Xd = B.bf16_from_bits(X)
    rows = np.arange(tokens)
    Y0 = layer.fwd(Xd)
    errs = {"Y": parity_error(to_f64(B.bits_from_bf16(Y0)), oracle.fwd_rows(X, W, mask1, rows, None, None))}
    if wl.rank:
        Ld, Rd = B.bf16_from_bits(L), B.bf16_from_bits(R)
        T = layer.adapter_T(Xd, Ld)
        Y1 = layer.fwd(Xd, T, Rd)
        errs["T"] = parity_error(to_f64(B.bits_from_bf16(T)), oracle.adapter_T_rows(X, L, rows))
        errs["Y+adapter"] = parity_error(to_f64(B.bits_from_bf16(Y1)), oracle.fwd_rows(X, W, mask1, rows, L, R))
    layer.poll()
    print(key, lay.name, tokens, errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)


def test_more_than_2_31_activation_elements(B, oracle):
    """524296 tokens x 4096 features: activations and outputs of 2^31 + 32768 elements each, so every
    64-bit index path (TMA row coordinates, output offsets, the token reduction of the weight gradient
    over 8193 k-blocks) is exercised.  The activations are a seeded 2048-token block repeated 256 times
    plus 8 more rows, so the oracle needs only the block: row n of the big tensors is block row n % 2048,
    and dY^T X = 256 * (block term) + (term of the first 8 block rows)."""
    import torch

    d, blk, reps, extra = 4096, 2048, 256, 8
    b = blk * reps + extra
    W = si.gaussian_bf16((d, d), 0.02, 901)
    Xb = si.gaussian_bf16((blk, d), 1.0, 902)
    dYb = si.gaussian_bf16((blk, d), 1.0, 903)
    layer = GpuLayer(W)
    _, _, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    assert np.array_equal(layer.mask1.cpu().numpy(), mask1) and np.array_equal(layer.mask2.cpu().numpy(), mask2)

    def tiled(bits):
        small = B.bf16_from_bits(bits)
        big = torch.empty((b, d), dtype=torch.bfloat16, device="cuda")
        big[: blk * reps].view(reps, blk, d).copy_(small.unsqueeze(0).expand(reps, blk, d))
        big[blk * reps:] = small[:extra]
        return big

    X, dY = tiled(Xb), tiled(dYb)
    assert X.numel() > 2 ** 31
    Y = layer.fwd(X)
    dX = layer.dx(dY)
    dWc = layer.dw(dY, X)
    layer.poll()
    rows = np.concatenate([np.arange(3), si.sample_indices(b, 24, 904), np.arange(b - extra - 3, b)])   # incl. the last rows
    pick = lambda t: to_f64(B.bits_from_bf16(t[torch.as_tensor(rows, device="cuda", dtype=torch.long)]))
    errs = {
        "Y": parity_error(pick(Y), oracle.fwd_rows(Xb, W, mask1, rows % blk)),
        "dX": parity_error(pick(dX), oracle.dx_rows(dYb, W, mask2, rows % blk)),
    }
    orows = si.sample_indices(d, 32, 905)
    want = reps * oracle.dw_rows(dYb, Xb, mask1, orows) + oracle.dw_rows(dYb[:extra], Xb[:extra], mask1, orows)
    got = to_f64(B.bits_from_bf16(dWc[torch.as_tensor(orows, device="cuda", dtype=torch.long)]))
    errs["dWc"] = parity_error(got, want)
    print(errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)
    for t in (Y, dX):
        assert bool(torch.isfinite(t[-extra:].float()).all())


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
def test_pruning_a_matrix_of_more_than_2_31_elements(B, oracle, fused):
    """W[65792 x 32768] (2^31 + 8.4 M elements, 4.3 GB): a seeded 256-row block repeated 257 times.  Both
    pruning passes work on groups inside 128 x 128 tiles, so every 256-row slab of the outputs must equal
    the oracle's outputs for the block; the first, a middle and the last slab are compared bit for bit."""
    import torch

    blk, reps, d_in = 256, 257, 32768
    d_out = blk * reps
    Wb = si.gaussian_bf16((blk, d_in), 0.02, 911)
    vals_b, nib_b, mask_b = oracle.prune24(Wb)
    valsT_b, nibT_b, mask2_b = oracle.double_prune(Wb, mask_b)
    meta_b = oracle.canonical_to_hw(oracle.pack_canonical(nib_b))            # 2 row blocks x 256 column blocks
    metaT_b = oracle.canonical_to_hw(oracle.pack_canonical(nibT_b)).reshape(d_in // 128, 2, 2048)
    small = B.bf16_from_bits(Wb)
    W = torch.empty((d_out, d_in), dtype=torch.bfloat16, device="cuda")
    W.view(reps, blk, d_in).copy_(small.unsqueeze(0).expand(reps, blk, d_in))
    assert W.numel() > 2 ** 31
    vals, meta, mask1 = B.alloc_compressed(d_out, d_in)
    valsT, metaT, _ = B.alloc_compressed(d_in, d_out)
    mask2 = torch.empty_like(mask1)
    if fused:
        B.slope_prune_24_double(W, vals, meta, mask1, valsT, metaT, mask2)
    else:
        B.slope_prune_24(W, vals, meta, mask1)
        B.slope_double_prune(W, mask1, valsT, metaT, mask2)
    assert B.slope_poll_status() == 0
    meta_rows = meta.view(d_out // 128, (d_in // 128) * 2048)
    metaT_blocks = metaT.view(d_in // 128, d_out // 128, 2048)
    for t in (0, 131, reps - 1):
        rows = slice(t * blk, (t + 1) * blk)
        assert np.array_equal(B.bits_from_bf16(vals[rows]), vals_b), t
        assert np.array_equal(mask1[rows].cpu().numpy(), mask_b), t
        assert np.array_equal(mask2[rows].cpu().numpy(), mask2_b), t
        assert np.array_equal(meta_rows[2 * t: 2 * t + 2].cpu().numpy().reshape(-1), meta_b.reshape(-1)), t
        assert np.array_equal(B.bits_from_bf16(valsT[:, t * (blk // 2): (t + 1) * (blk // 2)].contiguous()), valsT_b), t
        assert np.array_equal(metaT_blocks[:, 2 * t: 2 * t + 2].contiguous().cpu().numpy(), metaT_b), t
    if fused:
        # the optimizer tail's gather indexes its 8- and 16-byte units with 32 bits: same matrix, same slabs
        # (unchanged forward values must give back the transposed copy)
        del W
        again = torch.zeros_like(valsT)
        B.slope_update_sparse_matrix(vals, mask1, metaT, again)
        assert B.slope_poll_status() == 0
        for t in (0, 131, reps - 1):
            assert np.array_equal(B.bits_from_bf16(again[:, t * (blk // 2): (t + 1) * (blk // 2)].contiguous()), valsT_b), t
