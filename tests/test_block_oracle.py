"""Pins of the float64 decoder-block oracle (no GPU needed).

B1  its linear-layer function against the C oracle's per-row routines (forward, input
    gradient with the doubly pruned matrix, masked weight gradient, adapter gradients);
B2  the whole block against plain torch autograd when the second pruning pass removes
    nothing: then the layer's hand-written backward is the derivative of its forward;
B3  closed form: with one position per sequence causal attention returns v.
"""
import numpy as np
import pytest
import torch

from paper_2608_24070_b200 import inputs as si


@pytest.fixture(scope="module")
def blk():
    from oracle import block
    return block


def compress_rows(dense, mask_bool):
    """Kept entries of every row in ascending column order -> [rows, cols/2]."""
    rows, cols = dense.shape
    return dense[mask_bool].reshape(rows, cols // 2)


def small_block_inputs(d, ffn, tokens, r, seed):
    shapes = {"q": (d, d), "k": (d, d), "v": (d, d), "o": (d, d), "gate": (ffn, d), "up": (ffn, d), "down": (d, ffn)}
    W, L, R = {}, {}, {}
    for i, (name, (d_out, d_in)) in enumerate(shapes.items()):
        W[name] = si.gaussian_bf16((d_out, d_in), 0.05, seed + 10 * i)
        L[name] = si.gaussian_bf16((d_in, r), 0.05, seed + 10 * i + 3) if r else None
        R[name] = si.gaussian_bf16((r, d_out), 0.05, seed + 10 * i + 4) if r else None
    x = si.gaussian_bf16((tokens, d), 1.0, seed + 101)
    dout = si.gaussian_bf16((tokens, d), 1.0, seed + 102)
    return W, L, R, x, dout


def test_b1_layer_function_matches_c_oracle(oracle, blk):
    d_in, d_out, b, r = 64, 48, 24, 8
    W = si.gaussian_bf16((d_out, d_in), 0.02, 11)
    X = si.gaussian_bf16((b, d_in), 1.0, 12)
    dY = si.gaussian_bf16((b, d_out), 1.0, 13)
    L = si.gaussian_bf16((d_in, r), 0.1, 14)
    R = si.gaussian_bf16((r, d_out), 0.1, 15)
    _, _, m1 = oracle.prune24(W)
    _, _, m2 = oracle.double_prune(W, m1)
    lay = blk.make_layer(W, L, R)
    Xt = torch.from_numpy(oracle.bf16_to_f64(X)).requires_grad_(True)
    Y = blk.slope_linear(Xt, lay)
    Y.backward(torch.from_numpy(oracle.bf16_to_f64(dY)))
    rows = np.arange(b)
    close = lambda a, ref: np.testing.assert_allclose(a, ref, rtol=1e-11, atol=1e-12)
    close(Y.detach().numpy(), oracle.fwd_rows(X, W, m1, rows, L, R))
    close(Xt.grad.numpy(), oracle.dx_rows(dY, W, m2, rows, L, R))
    close(compress_rows(lay.WR.grad.numpy(), oracle.mask_to_bool(m1, d_in)), oracle.dw_rows(dY, X, m1, np.arange(d_out)))
    close(lay.L.grad.numpy(), oracle.adapter_dL_rows(X, dY, R, np.arange(d_in)))
    close(lay.R.grad.numpy(), oracle.adapter_dR_cols(X, L, dY, np.arange(d_out)))
    # the doubly pruned matrix really differs from the pruned one here, so the two gradients differ
    assert (lay.WRC != lay.WR).any()


def test_b2_block_equals_plain_autograd_when_second_pass_removes_nothing(oracle, blk):
    d, ffn, batch, seq, heads, r = 32, 48, 2, 6, 2, 4
    W, L, R, x, dout = small_block_inputs(d, ffn, batch * seq, r, 500)
    layers = {}
    for name in blk.LAYER_NAMES:
        _, _, m1 = oracle.prune24(W[name])
        _, _, m2 = oracle.double_prune(W[name], m1)
        keep = oracle.mask_to_bool(m2, W[name].shape[1])
        W2 = np.where(keep, W[name], np.uint16(0))          # already 2:4 along rows and along columns
        layers[name] = blk.make_layer(W2, L[name], R[name])
        assert torch.equal(layers[name].WR.detach(), layers[name].WRC)

    out, dx, grads = blk.block_fwd_bwd(x, dout, layers, batch, seq, heads)

    def plain_linear(X, lay):
        return X @ lay.WR.t() + (X @ lay.L) @ lay.R

    out_p, dx_p, grads_p = blk.block_fwd_bwd(x, dout, layers, batch, seq, heads, linear=plain_linear)
    close = lambda a, ref: np.testing.assert_allclose(a, ref, rtol=1e-10, atol=1e-12)
    close(out, out_p)
    close(dx, dx_p)
    for name in blk.LAYER_NAMES:
        close(grads[name]["dW"], grads_p[name]["dW"] * layers[name].mask1.numpy())
        close(grads[name]["dL"], grads_p[name]["dL"])
        close(grads[name]["dR"], grads_p[name]["dR"])
    # and the masked weight gradient is not the full one: the mask matters
    assert any((grads_p[n]["dW"] * (1 - layers[n].mask1.numpy()) != 0).any() for n in blk.LAYER_NAMES)


def test_b3_single_position_block_has_a_closed_form(oracle, blk):
    d, ffn, batch, seq, heads = 16, 32, 5, 1, 2
    W, _, _, x, dout = small_block_inputs(d, ffn, batch * seq, 0, 900)
    layers = {name: blk.make_layer(W[name]) for name in blk.LAYER_NAMES}
    out, _, _ = blk.block_fwd_bwd(x, dout, layers, batch, seq, heads)
    X = oracle.bf16_to_f64(x)
    WR = {n: layers[n].WR.detach().numpy() for n in blk.LAYER_NAMES}
    rms = lambda t: t / np.sqrt((t * t).mean(axis=-1, keepdims=True) + 1e-5)
    n1 = rms(X)
    h = X + (n1 @ WR["v"].T) @ WR["o"].T                      # softmax over one position is 1: attention returns v
    n2 = rms(h)
    gate = n2 @ WR["gate"].T
    ref = h + ((gate / (1 + np.exp(-gate))) * (n2 @ WR["up"].T)) @ WR["down"].T
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)
