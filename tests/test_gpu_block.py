"""GPU: one decoder-block training step with real data flow through the seven sparse linears,
against the float64 block oracle.

Tolerance: unlike a single layer (one fp32 -> bf16 rounding, 1.7e-3 relative), a block output or
gradient has passed 10-15 bf16 roundings in sequence (every linear output, T / dT, every torch
glue op, the bf16 attention probabilities), each ~2e-3 relative and independent: their
root-sum-square is 6-8e-3 (measured on this case: 2.4e-3 for the output and the input gradient,
which the residual path dominates, 3.9-5.7e-3 for the weight and adapter gradients).  The
bound is 1.5e-2; a wrong mask, a dropped adapter term or the wrong pruned copy in the input
gradient moves these tensors by 1e-1 or more.
"""
import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si

pytestmark = pytest.mark.gpu

TOL = 1.5e-2


@pytest.fixture(scope="module")
def H():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24070_b200 import binding, block_harness, build

    build.build()
    binding.lib()
    return block_harness


def rel(a, ref):
    a = np.asarray(a, np.float64)
    return float(np.linalg.norm(a - ref) / np.linalg.norm(ref))


def compress_rows(dense, mask_bool):
    rows, cols = dense.shape
    return dense[mask_bool].reshape(rows, cols // 2)


@pytest.mark.parametrize("r", [0, 64])
def test_block_step_matches_block_oracle(H, oracle, r):
    import torch
    from oracle import block as OB
    from paper_2608_24070_b200 import binding as B

    d, ffn, batch, seq, heads = 512, 1408, 2, 128, 4
    tokens = batch * seq
    shapes = {"q": (d, d), "k": (d, d), "v": (d, d), "o": (d, d), "gate": (ffn, d), "up": (ffn, d), "down": (d, ffn)}
    gpu_layers, cpu_layers, masks = {}, {}, {}
    for i, (name, (d_out, d_in)) in enumerate(shapes.items()):
        W = si.gaussian_bf16((d_out, d_in), 0.02, 4000 + 10 * i)
        L = si.gaussian_bf16((d_in, r), 0.01, 4003 + 10 * i) if r else None
        Rm = si.gaussian_bf16((r, d_out), 0.01, 4004 + 10 * i) if r else None
        cpu_layers[name] = OB.make_layer(W, L, Rm)
        masks[name] = cpu_layers[name].mask1.numpy().astype(bool)
        gpu_layers[name] = H.SlopeLinear(B.bf16_from_bits(W), None if L is None else B.bf16_from_bits(L),
                                         None if Rm is None else B.bf16_from_bits(Rm))
    x = si.gaussian_bf16((tokens, d), 1.0, 4101)
    dout = si.gaussian_bf16((tokens, d), 1.0, 4102)

    out_o, dx_o, grads_o = OB.block_fwd_bwd(x, dout, cpu_layers, batch, seq, heads)
    out_g, dx_g = H.block_step(B.bf16_from_bits(x), B.bf16_from_bits(dout), gpu_layers, batch, seq, heads)
    torch.cuda.synchronize()
    assert B.slope_poll_status() == 0

    errs = {"out": rel(out_g.float().cpu().numpy(), out_o), "dx": rel(dx_g.float().cpu().numpy(), dx_o)}
    for name in H.LAYER_NAMES:
        lay = gpu_layers[name]
        errs[f"dWc.{name}"] = rel(lay.dWc.float().cpu().numpy(), compress_rows(grads_o[name]["dW"], masks[name]))
        if r:
            errs[f"dL.{name}"] = rel(lay.dL.float().cpu().numpy(), grads_o[name]["dL"])
            errs[f"dR.{name}"] = rel(lay.dR.float().cpu().numpy(), grads_o[name]["dR"])
    print({k: round(v, 5) for k, v in errs.items()})
    bad = {k: v for k, v in errs.items() if not v <= TOL}
    assert not bad, bad


def test_dense_block_on_torch_runs_the_same_graph(H):
    """The all-dense comparison block (cuBLAS linears) used by the benchmark: shapes and gradients exist."""
    import torch
    from paper_2608_24070_b200 import binding as B

    d, ffn, batch, seq, heads = 256, 512, 2, 64, 2
    shapes = {"q": (d, d), "k": (d, d), "v": (d, d), "o": (d, d), "gate": (ffn, d), "up": (ffn, d), "down": (d, ffn)}
    layers = {n: H.DenseLinear(B.bf16_from_bits(si.gaussian_bf16(s, 0.02, 4200 + i))) for i, (n, s) in enumerate(shapes.items())}
    timers = []
    for lay in layers.values():
        lay.timers = timers
    x = B.bf16_from_bits(si.gaussian_bf16((batch * seq, d), 1.0, 4301))
    dout = B.bf16_from_bits(si.gaussian_bf16((batch * seq, d), 1.0, 4302))
    out, dx = H.block_step(x, dout, layers, batch, seq, heads)
    torch.cuda.synchronize()
    assert out.shape == x.shape and dx.shape == x.shape
    assert all(lay.W.grad is not None and lay.W.grad.shape == lay.W.shape for lay in layers.values())
    assert len(timers) == 14 and H.elapsed_ms(timers) > 0
