"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same
seeded inputs.  Integer / byte outputs bit-exact; GEMM outputs within 5e-3 relative
Frobenius error (bf16 in, fp32 accumulate, one rounding to bf16)."""
import itertools

import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si
from helpers import REL_TOL, GpuLayer, check_selection, parity_error, rel_fro, to_f64

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


def dev(B, bits):
    return B.bf16_from_bits(bits)


# ------------------------------------------------------------------ selection / compression
@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
@pytest.mark.parametrize("d_out,d_in,seed", [(512, 512, 1), (384, 640, 2), (128, 1152, 3), (1280, 128, 4)])
def test_prune_and_double_prune_bit_exact(B, oracle, d_out, d_in, seed, fused):
    W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
    layer = GpuLayer(W, fused_setup=fused)
    check_selection(oracle, layer, W)


def test_both_passes_in_one_call_without_the_optional_masks(B, oracle):
    """slope_prune_24_double with mask1 / mask2 left out writes the same compressed copies."""
    import torch

    W = si.gaussian_bf16((384, 512), 0.02, 9)
    ref = GpuLayer(W, fused_setup=True)
    check_selection(oracle, ref, W)
    Wd = dev(B, W)
    vals, meta, _ = B.alloc_compressed(384, 512)
    valsT, metaT, _ = B.alloc_compressed(512, 384)
    B.slope_prune_24_double(Wd, vals, meta, None, valsT, metaT, None)
    assert B.slope_poll_status() == 0
    for a, b_ in ((vals, ref.Wc_vals), (valsT, ref.WTc_vals)):
        assert torch.equal(a.view(torch.int16), b_.view(torch.int16))
    assert torch.equal(meta, ref.Wc_meta) and torch.equal(metaT, ref.WTc_meta)


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
def test_prune_ties_zeros_and_specials(B, oracle, fused):
    """All 4-tuples over {+0,-0,+-1,+-2} (ties everywhere), plus inf / nan / denormal patterns."""
    alphabet = si.f32_to_bf16_bits(np.array([0.0, -0.0, 1.0, -1.0, 2.0, -2.0], np.float32))
    groups = np.array(list(itertools.product(alphabet, repeat=4)), np.uint16).reshape(-1)
    W = np.zeros((256, 256), np.uint16)
    W.reshape(-1)[: groups.size] = groups
    special = np.array([0x7F80, 0xFF80, 0x7FC0, 0x0001, 0x8001, 0x7F7F, 0x0080, 0xFFFF], np.uint16)
    rng = np.random.Generator(np.random.PCG64(5))
    W[128:, :] = rng.choice(special, size=(128, 256))
    layer = GpuLayer(W, fused_setup=fused)
    check_selection(oracle, layer, W)


# ------------------------------------------------------------------ exact special cases through the MMAs
def _nibble_pattern_weight(d_out, d_in, seed):
    """Integer-valued weights whose kept pair cycles through all six patterns."""
    rng = np.random.Generator(np.random.PCG64(seed))
    pats = np.array([(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)])
    groups = d_in // 4
    i = np.arange(d_out)[:, None]
    g = np.arange(groups)[None, :]
    which = (i * 7 + g * 5 + (i // 128) + (g // 32)) % 6
    sign = lambda shape: rng.choice(np.array([-1.0, 1.0], np.float32), size=shape)
    Wf = (rng.integers(1, 4, size=(d_out, groups, 4)).astype(np.float32) * sign((d_out, groups, 4)))
    big = rng.integers(8, 64, size=(d_out, groups, 2)).astype(np.float32) * sign((d_out, groups, 2))
    ii, gg = np.meshgrid(np.arange(d_out), np.arange(groups), indexing="ij")
    Wf[ii, gg, pats[which][..., 0]] = big[..., 0]
    Wf[ii, gg, pats[which][..., 1]] = big[..., 1]
    return si.f32_to_bf16_bits(Wf.reshape(d_out, d_in))


@pytest.mark.parametrize("d_out,d_in", [(256, 384), (640, 6144), (6144, 640)])
def test_identity_activations_return_the_pruned_weight_exactly(B, oracle, d_out, d_in):
    """X = I  =>  Y = (W^R)^T bit for bit;  dY = I  =>  dX = W^{R,C};  dY = I  =>  dWc = gather(X).
    The long dimensions reach the 512-row-tile kernel (reduction >= 6144), the short ones the
    256-row-tile kernel, both with partial last tiles."""
    import torch

    W = _nibble_pattern_weight(d_out, d_in, 6)
    layer = GpuLayer(W)
    mask1, mask2 = check_selection(oracle, layer, W)
    m1, m2 = oracle.mask_to_bool(mask1, d_in), oracle.mask_to_bool(mask2, d_in)
    Wf = to_f64(W)

    eye_in = torch.eye(d_in, dtype=torch.bfloat16, device="cuda")
    Y = layer.fwd(eye_in)
    layer.poll()
    assert np.array_equal(to_f64(B.bits_from_bf16(Y)), np.where(m1, Wf, 0.0).T)

    eye_out = torch.eye(d_out, dtype=torch.bfloat16, device="cuda")
    dX = layer.dx(eye_out)
    layer.poll()
    assert np.array_equal(to_f64(B.bits_from_bf16(dX)), np.where(m2, Wf, 0.0))

    Xb = si.gaussian_bf16((d_out, d_in), 1.0, 8)
    dWc = layer.dw(eye_out, dev(B, Xb))
    layer.poll()
    assert np.array_equal(B.bits_from_bf16(dWc), Xb[m1].reshape(d_out, d_in // 2))


# ------------------------------------------------------------------ GEMM parity, full outputs
CASES = [
    # d_in, d_out, tokens, rank, seed
    (512, 512, 256, 0, 11),          # config 1
    (512, 512, 256, 64, 12),
    (384, 640, 776, 32, 13),         # ragged token tail, several tiles in every dimension
    (768, 256, 1000, 128, 14),
    (128, 128, 8, 16, 15),           # smallest legal problem
    (6144, 640, 264, 32, 16),        # long forward reduction (48 k-blocks) on the 256-row tile
    (640, 6144, 264, 0, 17),         # same for the input-gradient GEMM
    (4096, 512, 40, 16, 18),         # few tokens, long reduction on few rows: few-token kernel (64-token tile), K split over a cluster
    (1024, 384, 200, 0, 19),         # 200 tokens: tile kernels with one narrow token tile
    (2048, 256, 64, 64, 20),         # exactly one 64-token tile with adapters
    (256, 2048, 128, 32, 21),        # 128 tokens: forward and dX choose between few-token and tile kernel by estimate
    (1024, 512, 8, 64, 22),          # decode size: 16-token tile with adapters
    (512, 1536, 16, 128, 23),        # 16 tokens, two adapter K-steps
    (1152, 384, 104, 128, 24),       # 104 tokens, ragged, two adapter K-steps, odd number of k-blocks
    (512, 768, 264, 256, 25),        # largest rank (6.25 % of a 4096-wide layer): two adapter column tiles
    (1024, 512, 16, 256, 26),        # largest rank at decode size
    (512, 384, 1, 16, 27),           # one token (decode of a single sequence)
    (1024, 512, 3, 0, 28),           # token counts that are no multiple of 8, on every kernel family:
    (384, 640, 7, 32, 29),
    (512, 512, 17, 64, 30),          #   few-token kernel, 64-token tile
    (640, 384, 100, 32, 31),
    (256, 384, 130, 0, 32),          #   tile kernels
    (384, 512, 250, 16, 33),         #   adapter products still on the few-token kernel
    (512, 256, 1001, 32, 34),        #   one-CTA dense kernels for T / dT, 16 token k-blocks with a tail of 41
    (512, 22016, 8, 16, 35),         # more weight slabs (172) than SMs: few-token kernel with two CTAs per SM
    (256, 19200, 1, 0, 36),          #   same, one token, 150 slabs
]


@pytest.mark.parametrize("d_in,d_out,b,r,seed", CASES)
def test_layer_against_oracle(B, oracle, d_in, d_out, b, r, seed):
    W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
    X = si.gaussian_bf16((b, d_in), 1.0, seed + 100)
    dY = si.gaussian_bf16((b, d_out), 1.0, seed + 200)
    L = si.gaussian_bf16((d_in, r), 0.01, seed + 300) if r else None
    R = si.gaussian_bf16((r, d_out), 0.01, seed + 400) if r else None
    layer = GpuLayer(W)
    mask1, mask2 = check_selection(oracle, layer, W)
    Xd, dYd = dev(B, X), dev(B, dY)
    rows = np.arange(b)
    if r:
        Ld, Rd = dev(B, L), dev(B, R)
        T = layer.adapter_T(Xd, Ld)
        Y = layer.fwd(Xd, T, Rd)
        dT, dL, dR = layer.adapter_bwd(Xd, dYd, Ld, Rd, T)
        dX = layer.dx(dYd, dT, Ld)
    else:
        Y = layer.fwd(Xd)
        dX = layer.dx(dYd)
    dWc = layer.dw(dYd, Xd)
    layer.poll()
    g = lambda t: to_f64(B.bits_from_bf16(t))
    errs = {
        "Y": parity_error(g(Y), oracle.fwd_rows(X, W, mask1, rows, L, R)),
        "dX": parity_error(g(dX), oracle.dx_rows(dY, W, mask2, rows, L, R)),
        "dWc": parity_error(g(dWc), oracle.dw_rows(dY, X, mask1, np.arange(d_out))),
    }
    if r:
        errs["T"] = parity_error(g(T), oracle.adapter_T_rows(X, L, rows))
        errs["dT"] = parity_error(g(dT), oracle.adapter_dT_rows(dY, R, rows))
        errs["dL"] = parity_error(g(dL), oracle.adapter_dL_rows(X, dY, R, np.arange(d_in)), roundings=2)
        errs["dR"] = parity_error(g(dR), oracle.adapter_dR_cols(X, L, dY, np.arange(d_out)), roundings=2)
    print(errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)


@pytest.mark.parametrize("d_in,d_out,b,r", [(4096, 1024, 4104, 32), (1024, 4096, 4104, 0)])
def test_512_row_tile_kernel_on_sampled_rows(B, oracle, d_in, d_out, b, r):
    """Shapes for which the kernel choice takes the 512-row tile (38 tiles fill one wave where 76
    256-row tiles would need two), with a ragged token tail: sampled token rows against the oracle."""
    W = si.gaussian_bf16((d_out, d_in), 0.02, 131)
    X = si.gaussian_bf16((b, d_in), 1.0, 132)
    dY = si.gaussian_bf16((b, d_out), 1.0, 133)
    L = si.gaussian_bf16((d_in, r), 0.01, 134) if r else None
    R = si.gaussian_bf16((r, d_out), 0.01, 135) if r else None
    layer = GpuLayer(W)
    _, _, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    Xd, dYd = dev(B, X), dev(B, dY)
    if r:
        Ld, Rd = dev(B, L), dev(B, R)
        T = layer.adapter_T(Xd, Ld)
        Y = layer.fwd(Xd, T, Rd)
        dT, _, _ = layer.adapter_bwd(Xd, dYd, Ld, Rd, T)
        dX = layer.dx(dYd, dT, Ld)
    else:
        Y = layer.fwd(Xd)
        dX = layer.dx(dYd)
    layer.poll()
    rows = np.concatenate([np.arange(4), si.sample_indices(b, 40, 136), np.arange(b - 4, b)])
    errs = {
        "Y": parity_error(to_f64(B.bits_from_bf16(Y))[rows], oracle.fwd_rows(X, W, mask1, rows, L, R)),
        "dX": parity_error(to_f64(B.bits_from_bf16(dX))[rows], oracle.dx_rows(dY, W, mask2, rows, L, R)),
    }
    print(errs)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)


def test_few_token_forward_in_a_cuda_graph_matches_eager_bitwise(B, oracle):
    """The few-token kernel opts in to programmatic dependent launch; a captured chain of
    launches (each reading the previous one's output) must replay to the eager result."""
    import torch

    d, b = 512, 8
    Ws = [si.gaussian_bf16((d, d), 0.05, 40 + i) for i in range(3)]
    layers = [GpuLayer(W) for W in Ws]
    X = si.gaussian_bf16((b, d), 1.0, 44)
    Xd = dev(B, X)

    def chain(outs):
        h = Xd
        for layer, o in zip(layers, outs):
            B.slope_linear_fwd(h, layer.Wc_vals, layer.Wc_meta, d, o)
            h = o

    eager = [torch.empty((b, d), dtype=torch.bfloat16, device="cuda") for _ in layers]
    chain(eager)
    torch.cuda.synchronize()
    captured = [torch.zeros((b, d), dtype=torch.bfloat16, device="cuda") for _ in layers]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        chain(captured)                       # warm-up outside the capture
        stream.synchronize()
        for o in captured:
            o.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            chain(captured)
    torch.cuda.synchronize()
    for o in captured:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    layers[0].poll()
    for e, c in zip(eager, captured):
        assert np.array_equal(B.bits_from_bf16(e), B.bits_from_bf16(c))
    # and the chain's first link against the oracle
    mask1, _ = check_selection(oracle, layers[0], Ws[0])
    assert parity_error(to_f64(B.bits_from_bf16(eager[0])), oracle.fwd_rows(X, Ws[0], mask1, np.arange(b), None, None)) <= REL_TOL


def test_training_step_of_a_layer_in_a_cuda_graph_matches_eager_bitwise(B, oracle):
    """Every compute call of one layer's step (prune, double prune, adapters, fwd, dX, masked dW) captured
    in one CUDA graph: the replay must reproduce the eager outputs bit for bit."""
    import torch

    d_in, d_out, b, r = 640, 384, 520, 32
    W = si.gaussian_bf16((d_out, d_in), 0.02, 121)
    X, dY = dev(B, si.gaussian_bf16((b, d_in), 1.0, 122)), dev(B, si.gaussian_bf16((b, d_out), 1.0, 123))
    L, R = dev(B, si.gaussian_bf16((d_in, r), 0.01, 124)), dev(B, si.gaussian_bf16((r, d_out), 0.01, 125))
    Wd = dev(B, W)
    bf = torch.bfloat16
    mk = lambda *shape: torch.zeros(shape, dtype=bf, device="cuda")
    vals, meta, mask1 = B.alloc_compressed(d_out, d_in)
    valsT, metaT, _ = B.alloc_compressed(d_in, d_out)
    T, dT, dL, dR = mk(b, r), mk(b, r), mk(d_in, r), mk(r, d_out)
    Y, dX, dWc = mk(b, d_out), mk(b, d_in), mk(d_out, d_in // 2)
    ws = torch.empty(B.slope_adapter_workspace_bytes(b, d_out, d_in, r), dtype=torch.uint8, device="cuda")
    outs = (vals, meta, mask1, valsT, metaT, T, Y, dT, dL, dR, dX, dWc)

    def step():
        B.slope_prune_24(Wd, vals, meta, mask1)
        B.slope_double_prune(Wd, mask1, valsT, metaT, None)
        B.slope_adapter_fwd_bwd(0, X, None, L, None, b, d_out, d_in, r, T=T)
        B.slope_linear_fwd(X, vals, meta, d_out, Y, T, R)
        B.slope_adapter_fwd_bwd(1, X, dY, L, R, b, d_out, d_in, r, T=T, dT=dT, dL=dL, dR=dR, workspace=ws)
        B.slope_linear_bwd_dx(dY, valsT, metaT, d_in, dX, dT, L)
        B.slope_linear_bwd_dw_masked(dY, X, mask1, dWc)

    step()
    torch.cuda.synchronize()
    assert B.slope_poll_status() == 0
    eager = [t.clone() for t in outs]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
    torch.cuda.synchronize()
    for t in outs:
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert B.slope_poll_status() == 0
    for e, t in zip(eager, outs):
        assert torch.equal(e.view(torch.uint8) if e.dtype == torch.uint8 else e.view(torch.int16),
                           t.view(torch.uint8) if t.dtype == torch.uint8 else t.view(torch.int16))
    # the eager step itself against the oracle (forward only; the other outputs have their own tests)
    _, _, m1 = oracle.prune24(W)
    want = oracle.fwd_rows(B.bits_from_bf16(X), W, m1, np.arange(b), B.bits_from_bf16(L), B.bits_from_bf16(R))
    assert parity_error(to_f64(B.bits_from_bf16(eager[6])), want) <= REL_TOL


def test_no_adapter_path_is_bitwise_the_rank0_path_and_deterministic(B, oracle):
    W = si.gaussian_bf16((256, 256), 0.02, 31)
    X = si.gaussian_bf16((512, 256), 1.0, 32)
    layer = GpuLayer(W)
    Xd = dev(B, X)
    a = B.bits_from_bf16(layer.fwd(Xd))
    b = B.bits_from_bf16(layer.fwd(Xd))
    layer.poll()
    assert np.array_equal(a, b)


def test_argument_errors_are_reported_before_launch(B):
    import torch

    W = torch.zeros((100, 128), dtype=torch.bfloat16, device="cuda")
    vals = torch.zeros((100, 64), dtype=torch.bfloat16, device="cuda")
    meta = torch.zeros(100 * 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SlopeError) as e:
        B.slope_prune_24(W, vals, meta)
    assert e.value.status == 2
    W = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    vals = torch.zeros((128, 64 + 4), dtype=torch.bfloat16, device="cuda").view(-1)[1:1 + 128 * 64]
    with pytest.raises(B.SlopeError) as e:
        B.slope_prune_24(W, vals, torch.zeros(2048, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    assert B.lib().slope_prune_24(None, 128, 128, None, None, None, None) == 1
    assert B.slope_poll_status() == 0


def test_bounded_wait_times_out_and_reports_status(B, oracle):
    """A device-side wait that nothing satisfies gives up after its limit, the kernel returns,
    the sticky status reads SLOPE_ERR_TIMEOUT once, and the library keeps working afterwards."""
    import time

    import torch

    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    B.slope_selftest_wait_timeout(2000, flag)                 # 2 ms
    st = B.slope_poll_status()
    dt = time.perf_counter() - t0
    assert st == 6 and B.slope_status_string(st) == "device-side wait timed out"
    assert int(flag.item()) == 1
    assert dt < 1.0
    assert B.slope_poll_status() == 0                          # cleared by the read
    W = si.gaussian_bf16((128, 128), 0.02, 77)
    layer = GpuLayer(W)
    check_selection(oracle, layer, W)                          # context still healthy


def test_optional_masks_and_run_to_run_determinism(B, oracle):
    """The mask outputs are optional and do not change the other outputs; every GEMM is
    bit-identical run to run (no floating-point atomics, split-K reduced in a fixed order)."""
    import torch

    d_out, d_in, b, r = 384, 512, 520, 32
    W = si.gaussian_bf16((d_out, d_in), 0.02, 61)
    layer = GpuLayer(W)
    vals = torch.empty_like(layer.Wc_vals)
    meta = torch.empty_like(layer.Wc_meta)
    B.slope_prune_24(layer.W, vals, meta, None)
    valsT = torch.empty_like(layer.WTc_vals)
    metaT = torch.empty_like(layer.WTc_meta)
    B.slope_double_prune(layer.W, layer.mask1, valsT, metaT, None)
    layer.poll()
    for a, ref in ((vals, layer.Wc_vals), (meta, layer.Wc_meta), (valsT, layer.WTc_vals), (metaT, layer.WTc_meta)):
        assert torch.equal(a.view(torch.uint8), ref.view(torch.uint8))

    X = dev(B, si.gaussian_bf16((b, d_in), 1.0, 62))
    dY = dev(B, si.gaussian_bf16((b, d_out), 1.0, 63))
    L = dev(B, si.gaussian_bf16((d_in, r), 0.01, 64))
    R = dev(B, si.gaussian_bf16((r, d_out), 0.01, 65))

    def run():
        T = layer.adapter_T(X, L)
        Y = layer.fwd(X, T, R)
        dT, dL, dR = layer.adapter_bwd(X, dY, L, R, T)
        dX = layer.dx(dY, dT, L)
        dWc = layer.dw(dY, X)
        layer.poll()
        return [B.bits_from_bf16(t) for t in (T, Y, dT, dL, dR, dX, dWc)]

    first, second = run(), run()
    for a, c in zip(first, second):
        assert np.array_equal(a, c)


def _fuzz_shapes():
    """Seeded shapes that hit every branch of the kernel choice: few-token tiles of all four widths with
    one to eight K-splits, 256-row and 512-row sparse tiles, weight-gradient launches with and without
    halved last-wave tiles, one-CTA weight-gradient tiles, ranks from 16 to 256."""
    rng = np.random.Generator(np.random.PCG64(20260824))
    shapes = []
    for _ in range(20):
        d_in = 128 * int(rng.integers(1, 25))
        d_out = 128 * int(rng.integers(1, 25))
        b = 8 * int(rng.choice([1, 2, 5, 8, 13, 16, 27, 32, 33, 70, 129, 300]))
        r = int(rng.choice([0, 16, 48, 64, 112, 128, 256]))
        shapes.append((d_in, d_out, b, r))
    ragged = np.random.Generator(np.random.PCG64(20260825))          # token counts around every tile boundary
    for b in (1, 5, 9, 31, 63, 65, 127, 129, 255, 257, 999, 2047):
        shapes.append((128 * int(ragged.integers(1, 17)), 128 * int(ragged.integers(1, 17)), b,
                       int(ragged.choice([0, 16, 64, 128]))))
    shapes += [(2560, 5120, 2048, 0),      # dW: 10 x 20 = 200 tiles -> 2 waves + 52 tiles (no halving: more than half the pairs)
               (2304, 2560, 1000, 16),     # dW: 90 tiles -> 1 wave + 16 tiles, halved
               (4096, 1280, 3080, 64)]     # 512-row sparse tiles with a partial last row tile (1280 = 2.5 tiles)
    return shapes


@pytest.mark.parametrize("d_in,d_out,b,r", _fuzz_shapes())
def test_seeded_shape_sweep_on_sampled_outputs(B, oracle, d_in, d_out, b, r):
    seed = 7000 + d_in // 128 * 31 + d_out // 128 * 7 + b + r
    W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
    X = si.gaussian_bf16((b, d_in), 1.0, seed + 1)
    dY = si.gaussian_bf16((b, d_out), 1.0, seed + 2)
    L = si.gaussian_bf16((d_in, r), 0.01, seed + 3) if r else None
    R = si.gaussian_bf16((r, d_out), 0.01, seed + 4) if r else None
    layer = GpuLayer(W)
    _, _, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    assert np.array_equal(layer.mask1.cpu().numpy(), mask1) and np.array_equal(layer.mask2.cpu().numpy(), mask2)
    Xd, dYd = dev(B, X), dev(B, dY)
    if r:
        Ld, Rd = dev(B, L), dev(B, R)
        T = layer.adapter_T(Xd, Ld)
        Y = layer.fwd(Xd, T, Rd)
        dT, dL, dR = layer.adapter_bwd(Xd, dYd, Ld, Rd, T)
        dX = layer.dx(dYd, dT, Ld)
    else:
        Y = layer.fwd(Xd)
        dX = layer.dx(dYd)
    dWc = layer.dw(dYd, Xd)
    layer.poll()
    rows = np.unique(np.concatenate([np.arange(min(b, 3)), si.sample_indices(b, min(b, 24), seed + 5), np.arange(b - min(b, 3), b)]))
    orows = np.unique(np.concatenate([np.arange(2), si.sample_indices(d_out, min(d_out, 24), seed + 6), np.arange(d_out - 2, d_out)]))
    g = lambda t: to_f64(B.bits_from_bf16(t))
    errs = {
        "Y": parity_error(g(Y)[rows], oracle.fwd_rows(X, W, mask1, rows, L, R)),
        "dX": parity_error(g(dX)[rows], oracle.dx_rows(dY, W, mask2, rows, L, R)),
        "dWc": parity_error(g(dWc)[orows], oracle.dw_rows(dY, X, mask1, orows)),
    }
    if r:
        jrows = np.unique(np.concatenate([np.arange(2), si.sample_indices(d_in, min(d_in, 16), seed + 7)]))
        icols = np.unique(np.concatenate([np.arange(2), si.sample_indices(d_out, min(d_out, 32), seed + 8)]))
        errs["T"] = parity_error(g(T)[rows], oracle.adapter_T_rows(X, L, rows))
        errs["dT"] = parity_error(g(dT)[rows], oracle.adapter_dT_rows(dY, R, rows))
        errs["dL"] = parity_error(g(dL)[jrows], oracle.adapter_dL_rows(X, dY, R, jrows), roundings=2)
        errs["dR"] = parity_error(g(dR)[:, icols], oracle.adapter_dR_cols(X, L, dY, icols), roundings=2)
    for k, v in errs.items():
        assert v <= REL_TOL, (k, v, errs)
    import torch

    for t in (Y, dX, dWc):
        assert bool(torch.isfinite(t.float()).all())


def test_two_host_threads_on_two_streams(B, oracle):
    """Two host threads drive two layers on their own CUDA streams at the same time (the library keeps
    per-device caches behind mutexes and per-launch state only): both results match the oracle."""
    import threading

    import torch

    specs = [(1024, 512, 264, 32, 151), (512, 768, 16, 64, 161)]
    results, errors = {}, []

    def work(idx, d_in, d_out, b, r, seed):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
                X = si.gaussian_bf16((b, d_in), 1.0, seed + 1)
                dY = si.gaussian_bf16((b, d_out), 1.0, seed + 2)
                L = si.gaussian_bf16((d_in, r), 0.01, seed + 3)
                R = si.gaussian_bf16((r, d_out), 0.01, seed + 4)
                layer = GpuLayer(W)
                Xd, dYd, Ld, Rd = dev(B, X), dev(B, dY), dev(B, L), dev(B, R)
                outs = None
                for _ in range(10):
                    T = layer.adapter_T(Xd, Ld)
                    Y = layer.fwd(Xd, T, Rd)
                    dT, dL, dR = layer.adapter_bwd(Xd, dYd, Ld, Rd, T)
                    dX = layer.dx(dYd, dT, Ld)
                    dWc = layer.dw(dYd, Xd)
                    outs = (Y, dX, dWc)
                stream.synchronize()
                results[idx] = (W, X, dY, L, R, [B.bits_from_bf16(t) for t in outs], layer.mask1.cpu().numpy(),
                                layer.mask2.cpu().numpy())
        except Exception as ex:                         # noqa: BLE001
            errors.append(ex)

    threads = [threading.Thread(target=work, args=(i, *spec)) for i, spec in enumerate(specs)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert B.slope_poll_status() == 0
    for idx, (d_in, d_out, b, r, seed) in enumerate(specs):
        W, X, dY, L, R, (Y, dX, dWc), m1, m2 = results[idx]
        _, _, mask1 = oracle.prune24(W)
        _, _, mask2 = oracle.double_prune(W, mask1)
        assert np.array_equal(m1, mask1) and np.array_equal(m2, mask2)
        rows = np.arange(b)
        assert parity_error(to_f64(Y), oracle.fwd_rows(X, W, mask1, rows, L, R)) <= REL_TOL
        assert parity_error(to_f64(dX), oracle.dx_rows(dY, W, mask2, rows, L, R)) <= REL_TOL
        assert parity_error(to_f64(dWc), oracle.dw_rows(dY, X, mask1, np.arange(d_out))) <= REL_TOL


@pytest.mark.parametrize("b", [1, 7, 17, 130, 250, 1001])
def test_rows_past_the_last_token_are_never_written(B, oracle, b):
    """Outputs live at the start of larger buffers filled with a sentinel: whatever tile a kernel
    works in, nothing behind row b - 1 may change (forward, input gradient, adapter T and dT)."""
    import torch

    d_in, d_out, r, guard = 384, 512, 32, 96
    W = si.gaussian_bf16((d_out, d_in), 0.02, 9100 + b)
    layer = GpuLayer(W)
    Xd = dev(B, si.gaussian_bf16((b, d_in), 1.0, 9200 + b))
    dYd = dev(B, si.gaussian_bf16((b, d_out), 1.0, 9300 + b))
    Ld = dev(B, si.gaussian_bf16((d_in, r), 0.01, 9400 + b))
    Rd = dev(B, si.gaussian_bf16((r, d_out), 0.01, 9500 + b))
    sentinel = 0x7FC1                                              # a NaN pattern no kernel produces from finite inputs

    def guarded(cols):
        buf = torch.full(((b + guard) * cols,), sentinel, dtype=torch.int16, device="cuda").view(torch.bfloat16)
        return buf, buf[: b * cols].view(b, cols)

    bufs = {}
    bufs["T"], T = guarded(r)
    bufs["dT"], dT = guarded(r)
    bufs["Y"], Y = guarded(d_out)
    bufs["dX"], dX = guarded(d_in)
    dL = torch.empty((d_in, r), dtype=torch.bfloat16, device="cuda")
    dR = torch.empty((r, d_out), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.slope_adapter_workspace_bytes(b, d_out, d_in, r), dtype=torch.uint8, device="cuda")
    B.slope_adapter_fwd_bwd(0, Xd, None, Ld, None, b, d_out, d_in, r, T=T)
    B.slope_linear_fwd(Xd, layer.Wc_vals, layer.Wc_meta, d_out, Y, T, Rd)
    B.slope_adapter_fwd_bwd(1, Xd, dYd, Ld, Rd, b, d_out, d_in, r, T=T, dT=dT, dL=dL, dR=dR, workspace=ws)
    B.slope_linear_bwd_dx(dYd, layer.WTc_vals, layer.WTc_meta, d_in, dX, dT, Ld)
    layer.poll()
    for name, buf in bufs.items():
        cols = {"T": r, "dT": r, "Y": d_out, "dX": d_in}[name]
        tail = buf.view(torch.int16)[b * cols:]
        assert bool((tail == sentinel).all()), name
        assert bool(torch.isfinite(buf[: b * cols].float()).all()), name


def test_dependent_launches_back_to_back_equal_synchronised_launches_bitwise(B, oracle):
    """Every GEMM launch may start its set-up under the previous kernel's tail (programmatic
    dependent launch).  A chain in which each call consumes what the previous one wrote -- three
    layers feeding one another forward, then backward, adapters included -- must give the same bits
    whether the host synchronises after every call or never."""
    import torch

    dims = [384, 640, 256, 512]                      # layer i: dims[i] -> dims[i + 1]
    b, r = 776, 32
    layers, Ls, Rs = [], [], []
    for i in range(3):
        layers.append(GpuLayer(si.gaussian_bf16((dims[i + 1], dims[i]), 0.05, 9600 + i)))
        Ls.append(dev(B, si.gaussian_bf16((dims[i], r), 0.05, 9610 + i)))
        Rs.append(dev(B, si.gaussian_bf16((r, dims[i + 1]), 0.05, 9620 + i)))
    X0 = dev(B, si.gaussian_bf16((b, dims[0]), 1.0, 9630))
    dYlast = dev(B, si.gaussian_bf16((b, dims[3]), 1.0, 9631))

    def run(sync):
        def s():
            if sync:
                torch.cuda.synchronize()
        acts, Ts = [X0], []
        for i, lay in enumerate(layers):
            T = lay.adapter_T(acts[-1], Ls[i]); s()
            Ts.append(T)
            acts.append(lay.fwd(acts[-1], T, Rs[i])); s()
        grads, dY = [], dYlast
        for i in reversed(range(3)):
            dT, dL, dR = layers[i].adapter_bwd(acts[i], dY, Ls[i], Rs[i], Ts[i]); s()
            dX = layers[i].dx(dY, dT, Ls[i]); s()
            dWc = layers[i].dw(dY, acts[i]); s()
            grads += [dL, dR, dWc]
            dY = dX
        torch.cuda.synchronize()
        layers[0].poll()
        return [t.clone() for t in acts[1:] + grads + [dY]]

    ref = run(sync=True)
    for _ in range(3):
        got = run(sync=False)
        for a, g in zip(ref, got):
            assert torch.equal(a.view(torch.int16), g.view(torch.int16))


@pytest.mark.parametrize("d_in,d_out,b,r", [(1024, 512, 1, 16), (4096, 512, 8, 64), (512, 1536, 16, 128),
                                            (2048, 256, 40, 64), (1152, 384, 104, 256), (1024, 512, 16, 256),
                                            (1024, 2816, 64, 64), (256, 2048, 128, 32), (1024, 384, 200, 64),
                                            (512, 5632, 250, 256), (384, 640, 776, 32), (1024, 1024, 1000, 64),
                                            (2048, 512, 2048, 128), (512, 2816, 1544, 16)])
def test_forward_with_adapter_in_one_call_against_the_two_calls(B, oracle, d_in, d_out, b, r):
    """slope_linear_fwd_adapter: at inference sizes a fused pair of launches (the forward runs its
    sparse reduction while T is still being computed), with many tokens the plain two launches.
    T is the same launch as in the separate call: same bits.  Y is the same sum, but the forward of
    a fused pair picks its K-split among the clusters that fit beside the T launch, so fp32 partial
    sums may be grouped differently: a few outputs can land on the neighbouring bf16 value.  The
    call itself is deterministic, and a race with the T launch would not repeat its bits."""
    import torch

    seed = 9700 + b + r
    W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
    X = si.gaussian_bf16((b, d_in), 1.0, seed + 1)
    L = si.gaussian_bf16((d_in, r), 0.01, seed + 2)
    R = si.gaussian_bf16((r, d_out), 0.01, seed + 3)
    layer = GpuLayer(W)
    Xd, Ld, Rd = dev(B, X), dev(B, L), dev(B, R)
    T_ref = layer.adapter_T(Xd, Ld)
    Y_ref = layer.fwd(Xd, T_ref, Rd)
    layer.poll()
    first = None
    for _ in range(3):
        T = torch.full((b, r), float("nan"), dtype=torch.bfloat16, device="cuda")
        Y = torch.full((b, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.slope_linear_fwd_adapter(Xd, layer.Wc_vals, layer.Wc_meta, d_out, Ld, Rd, T, Y)
        layer.poll()
        assert torch.equal(T.view(torch.int16), T_ref.view(torch.int16))
        if first is None:
            first = Y
        assert torch.equal(Y.view(torch.int16), first.view(torch.int16))
    differ = Y.view(torch.int16) != Y_ref.view(torch.int16)
    assert int(differ.sum()) <= max(1, Y.numel() // 500)
    gap = (Y.float() - Y_ref.float()).abs()
    assert bool((gap <= Y_ref.float().abs() * 2.0 ** -6 + 1e-30).all())      # at most the neighbouring bf16 value
    _, _, mask1 = oracle.prune24(W)
    err = parity_error(to_f64(B.bits_from_bf16(Y)), oracle.fwd_rows(X, W, mask1, np.arange(b), L, R))
    assert err <= REL_TOL, err


def test_chain_of_fused_adapter_forwards_in_a_cuda_graph(B, oracle):
    """Four decode-size layers, each through the one-call forward, each fed by the previous one's
    output (so every pair's first launch really has to wait for the pair before it): the eager
    result agrees with the chain of separate calls up to the summation order of the K-split, and
    the captured graph and its replays reproduce the eager bits."""
    import torch

    dims, b, r = [512, 1024, 384, 640, 512], 8, 64
    layers, Ls, Rs = [], [], []
    for i in range(4):
        layers.append(GpuLayer(si.gaussian_bf16((dims[i + 1], dims[i]), 0.05, 9800 + i)))
        Ls.append(dev(B, si.gaussian_bf16((dims[i], r), 0.05, 9810 + i)))
        Rs.append(dev(B, si.gaussian_bf16((r, dims[i + 1]), 0.05, 9820 + i)))
    X0 = dev(B, si.gaussian_bf16((b, dims[0]), 1.0, 9830))
    ref = X0
    for i, lay in enumerate(layers):
        ref = lay.fwd(ref, lay.adapter_T(ref, Ls[i]), Rs[i])
    layers[0].poll()
    Ts = [torch.empty((b, r), dtype=torch.bfloat16, device="cuda") for _ in range(4)]
    acts = [X0] + [torch.empty((b, dims[i + 1]), dtype=torch.bfloat16, device="cuda") for i in range(4)]

    def chain():
        for i, lay in enumerate(layers):
            B.slope_linear_fwd_adapter(acts[i], lay.Wc_vals, lay.Wc_meta, dims[i + 1], Ls[i], Rs[i], Ts[i], acts[i + 1])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        chain()                                                    # eager, also warms up before capture
        side.synchronize()
        eager = acts[4].clone()
        assert rel_fro(eager.double().cpu().numpy(), ref.double().cpu().numpy()) <= 2e-3
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            chain()
        for _ in range(3):
            acts[4].zero_()
            graph.replay()
            side.synchronize()
            assert torch.equal(acts[4].view(torch.int16), eager.view(torch.int16))
    torch.cuda.current_stream().wait_stream(side)
    layers[0].poll()


# ------------------------------------------------------------------ weight gradient with dL, dR riding along
@pytest.mark.parametrize("d_in,d_out,b,r", [
    (3328, 3072, 1100, 64),      # 13 x 12 tiles on 74 pairs: fused launch, ragged tokens, 8 partial sums each way
    (3328, 3072, 200, 16),       # fewer k-blocks (4) than carriers: the split count follows the k-blocks
    (3072, 3328, 520, 128),      # widest rank of the fused launch
    (3200, 2944, 330, 32),       # d_in, d_out not multiples of 256: half-empty last tile row and column
    (4096, 4096, 300, 64),       # 256 tiles: the last wave's tiles are halved, none of them a carrier
    (1024, 1024, 300, 64),       # too few tiles for the 256 x 256 kernel: separate launches
    (3328, 3072, 300, 256),      # rank beyond the fused launch: separate launches
])
def test_weight_gradient_with_adapter_gradients_in_one_call(B, oracle, d_in, d_out, b, r):
    """slope_linear_bwd_dw_adapter against the oracle (dWc, dL, dR) and against the separate calls
    (dWc bit for bit: same kernel arithmetic, same reduction order)."""
    import torch

    W = si.gaussian_bf16((d_out, d_in), 0.02, 701)
    Xb, dYb = si.gaussian_bf16((b, d_in), 1.0, 702), si.gaussian_bf16((b, d_out), 1.0, 703)
    Lb, Rb = si.gaussian_bf16((d_in, r), 0.01, 704), si.gaussian_bf16((r, d_out), 0.01, 705)
    layer = GpuLayer(W, fused_setup=True)
    X, dY, L, R = dev(B, Xb), dev(B, dYb), dev(B, Lb), dev(B, Rb)
    T = layer.adapter_T(X, L)
    bf = torch.bfloat16
    dT = torch.empty((b, r), dtype=bf, device="cuda")
    B.slope_adapter_fwd_bwd(2, None, dY, None, R, b, d_out, d_in, r, dT=dT)
    dT_ref, dL_ref, dR_ref = layer.adapter_bwd(X, dY, L, R, T)
    assert torch.equal(dT.view(torch.int16), dT_ref.view(torch.int16))
    dWc_ref = layer.dw(dY, X)
    nan = float("nan")
    dWc = torch.full((d_out, d_in // 2), nan, dtype=bf, device="cuda")
    dL = torch.full((d_in, r), nan, dtype=bf, device="cuda")
    dR = torch.full((r, d_out), nan, dtype=bf, device="cuda")
    ws = torch.empty(B.slope_bwd_dw_adapter_workspace_bytes(b, d_out, d_in, r), dtype=torch.uint8, device="cuda")
    launches = B.slope_launch_count()
    for _ in range(2):                       # twice: stale partial sums in the workspace must not matter
        B.slope_linear_bwd_dw_adapter(dY, X, T, dT, layer.mask1, dWc, dL, dR, ws)
    layer.poll()
    # one GEMM launch + the reduction when the shape takes the fused launch, else dW, partial products, reduction
    fused = r <= 128 and d_in >= 2048
    assert B.slope_launch_count() - launches == 2 * (2 if fused else 3)
    assert torch.equal(dWc.view(torch.int16), dWc_ref.view(torch.int16))
    g = lambda t: to_f64(B.bits_from_bf16(t))
    _, _, mask1 = oracle.prune24(W)
    orows = si.sample_indices(d_out, 48, 11)
    jrows = si.sample_indices(d_in, 48, 12)
    icols = si.sample_indices(d_out, 96, 13)
    errs = {
        "dWc": parity_error(g(dWc)[orows], oracle.dw_rows(dYb, Xb, mask1, orows)),
        "dL": parity_error(g(dL)[jrows], oracle.adapter_dL_rows(Xb, dYb, Rb, jrows), roundings=2),
        "dR": parity_error(g(dR)[:, icols], oracle.adapter_dR_cols(Xb, Lb, dYb, icols), roundings=2),
        # against the separate launches: the same sums cut into other slices
        "dL_vs_separate": rel_fro(g(dL), g(dL_ref)),
        "dR_vs_separate": rel_fro(g(dR), g(dR_ref)),
    }
    print(errs)
    for k, v in errs.items():
        assert v <= (REL_TOL if "separate" not in k else 2.5e-3), (k, v, errs)
    assert np.isfinite(g(dL)).all() and np.isfinite(g(dR)).all()


def test_kernel_clock_diagnostic_reports_a_plausible_sm_clock(B, oracle):
    """slope_kernel_clock_mhz: the SM clock measured inside the sparse / dense tile-kernel launches
    since the previous call."""
    import torch

    W = si.gaussian_bf16((1024, 1024), 0.02, 801)
    layer = GpuLayer(W, fused_setup=True)
    X = dev(B, si.gaussian_bf16((2048, 1024), 1.0, 802))
    dY = dev(B, si.gaussian_bf16((2048, 1024), 1.0, 803))
    B.slope_kernel_clock_mhz(0), B.slope_kernel_clock_mhz(1)          # forget earlier launches
    assert B.slope_kernel_clock_mhz(0) == 0.0                          # nothing ran in between
    layer.fwd(X)                               # a CTA-pair sparse tile kernel
    layer.dw(dY, X)                            # the CTA-pair dense kernel
    layer.poll()
    for kind in (0, 1):
        mhz = B.slope_kernel_clock_mhz(kind)
        assert 300.0 < mhz < 2100.0, (kind, mhz)        # B200: at most 1965 MHz, ~1.1-1.5 GHz under tensor load
    with pytest.raises(B.SlopeError):
        B.slope_kernel_clock_mhz(2)
