"""GPU parity at the benchmark's full sizes and launch configuration: selection outputs are
compared in full (bit-exact); GEMM outputs on seeded samples of complete output rows, which the
oracle computes one dot product at a time (a sampled sub-tensor is exact)."""
import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si
from helpers import REL_TOL, GpuLayer, check_selection, rel_fro, to_f64

pytestmark = pytest.mark.gpu

CASES = [
    ("c2_gpt2_small", 0), ("c2_gpt2_small", 1), ("c2_gpt2_small", 2),
    ("c3_llama7b", 0), ("c3_llama7b", 4),
    ("c4_llama7b_adapter", 0), ("c4_llama7b_adapter", 6),
    ("c5_llama13b_block", 4),
]


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
    layer = GpuLayer(W)
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
        "Y": rel_fro(pick(Y, rows), oracle.fwd_rows(X, W, mask1, rows, L, R)),
        "dX": rel_fro(pick(dX, rows), oracle.dx_rows(dY, W, mask2, rows, L, R)),
        "dWc": rel_fro(pick(dWc, orows), oracle.dw_rows(dY, X, mask1, orows)),
    }
    if r:
        jrows = si.sample_indices(d_in, 16, seed + 2)
        icols = si.sample_indices(d_out, 256, seed + 3)
        errs["T"] = rel_fro(pick(T, rows), oracle.adapter_T_rows(X, L, rows))
        errs["dT"] = rel_fro(pick(dT, rows), oracle.adapter_dT_rows(dY, R, rows))
        errs["dL"] = rel_fro(pick(dL, jrows), oracle.adapter_dL_rows(X, dY, R, jrows))
        dR_s = to_f64(B.bits_from_bf16(dR[:, torch.as_tensor(icols, device=dR.device, dtype=torch.long)].contiguous()))
        errs["dR"] = rel_fro(dR_s, oracle.adapter_dR_cols(X, L, dY, icols))
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
    errs = {"Y": rel_fro(to_f64(B.bits_from_bf16(Y0)), oracle.fwd_rows(X, W, mask1, rows, None, None))}
    if wl.rank:
        Ld, Rd = B.bf16_from_bits(L), B.bf16_from_bits(R)
        T = layer.adapter_T(Xd, Ld)
        Y1 = layer.fwd(Xd, T, Rd)
        errs["T"] = rel_fro(to_f64(B.bits_from_bf16(T)), oracle.adapter_T_rows(X, L, rows))
        errs["Y+adapter"] = rel_fro(to_f64(B.bits_from_bf16(Y1)), oracle.fwd_rows(X, W, mask1, rows, L, R))
    layer.poll()
    print(key, lay.name, tokens, errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)
