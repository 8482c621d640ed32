"""One LLaMA-style decoder block, forward and backward, in float64 on the CPU -- TEST INFRASTRUCTURE ONLY.

The seven linear layers follow the sparse layer's equations on masked dense matrices
(masks from ``oracle.prune24`` / ``oracle.double_prune``):

    forward            Y  = X (W^R)^T + (X L) R                       Eq. (sparse_forward), Eq. (concat)
    input gradient     dX = dY W^{R,C} + (dY R^T) L^T                 Eq. (sparse_backward_input)
    weight gradient    dW = mask1 (.) (dY^T X)                        Eq. (sparse_backward_weight), Alg. 1
    adapter gradients  dL = X^T (dY R^T),  dR = (X L)^T dY            chain rule on the forward

Because the input gradient uses the doubly pruned matrix it is not the derivative of the
forward; the layer is therefore a ``torch.autograd.Function`` with exactly these four
formulas as its backward.  Everything between the linears (RMS normalisation without gain,
causal softmax attention without positional rotation, SiLU gate, residual adds) is the
textbook definition, differentiated by torch autograd in float64.  No intermediate is
rounded to bf16.

Pins (``tests/test_block_oracle.py``): the layer function against the C oracle's per-row
routines, and the whole block against plain torch autograd for weights on which the second
pruning pass removes nothing (then the backward above IS the derivative).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

from . import bf16_to_f64, double_prune, mask_to_bool, prune24

LAYER_NAMES = ("q", "k", "v", "o", "gate", "up", "down")


@dataclass
class LayerF64:
    """Masked dense matrices of one layer as float64 leaf tensors."""
    WR: torch.Tensor            # [d_out, d_in]  W (.) mask1, requires grad (its grad is mask1 (.) dY^T X)
    WRC: torch.Tensor           # [d_out, d_in]  W (.) mask2
    mask1: torch.Tensor         # [d_out, d_in]  float64 0/1
    L: Optional[torch.Tensor]   # [d_in, r]
    R: Optional[torch.Tensor]   # [r, d_out]


def make_layer(W_bits: np.ndarray, L_bits: Optional[np.ndarray] = None, R_bits: Optional[np.ndarray] = None) -> LayerF64:
    """Prune a bf16 weight (raw bit patterns) twice and widen everything to float64."""
    d_out, d_in = W_bits.shape
    _, _, m1 = prune24(W_bits)
    _, _, m2 = double_prune(W_bits, m1)
    W = bf16_to_f64(W_bits)
    b1 = mask_to_bool(m1, d_in)
    b2 = mask_to_bool(m2, d_in)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))
    return LayerF64(
        WR=t(W * b1).requires_grad_(True), WRC=t(W * b2), mask1=t(b1.astype(np.float64)),
        L=None if L_bits is None else t(bf16_to_f64(L_bits)).requires_grad_(True),
        R=None if R_bits is None else t(bf16_to_f64(R_bits)).requires_grad_(True))


class _SlopeLinearF64(torch.autograd.Function):
    @staticmethod
    def forward(ctx, X, WR, WRC, mask1, L, R):
        ctx.save_for_backward(X, WRC, mask1, L, R)
        Y = X @ WR.t()
        if L is not None:
            Y = Y + (X @ L) @ R
        return Y

    @staticmethod
    def backward(ctx, dY):
        X, WRC, mask1, L, R = ctx.saved_tensors
        dX = dY @ WRC
        dW = (dY.t() @ X) * mask1
        dL = dR = None
        if L is not None:
            dT = dY @ R.t()
            dX = dX + dT @ L.t()
            dL = X.t() @ dT
            dR = (X @ L).t() @ dY
        return dX, dW, None, None, dL, dR


def slope_linear(X: torch.Tensor, layer: LayerF64) -> torch.Tensor:
    return _SlopeLinearF64.apply(X, layer.WR, layer.WRC, layer.mask1, layer.L, layer.R)


def rms_norm(x: torch.Tensor, eps: float) -> torch.Tensor:
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps)


def causal_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, batch: int, seq: int, heads: int) -> torch.Tensor:
    """softmax(q k^T / sqrt(head_dim) + causal mask) v per (batch, head); inputs [batch*seq, heads*head_dim]."""
    hd = q.shape[1] // heads
    split = lambda t: t.reshape(batch, seq, heads, hd).permute(0, 2, 1, 3)         # [B, H, S, hd]
    qh, kh, vh = split(q), split(k), split(v)
    scores = (qh @ kh.transpose(-1, -2)) / math.sqrt(hd)
    future = torch.triu(torch.ones(seq, seq, dtype=torch.bool), diagonal=1)
    scores = scores.masked_fill(future, float("-inf"))
    out = torch.softmax(scores, dim=-1) @ vh
    return out.permute(0, 2, 1, 3).reshape(batch * seq, heads * hd)


def decoder_block(x: torch.Tensor, layers: Dict[str, LayerF64], batch: int, seq: int, heads: int, eps: float = 1e-5,
                  linear=slope_linear) -> torch.Tensor:
    """x [batch*seq, d] -> block output [batch*seq, d]."""
    n1 = rms_norm(x, eps)
    a = causal_attention(linear(n1, layers["q"]), linear(n1, layers["k"]), linear(n1, layers["v"]), batch, seq, heads)
    h = x + linear(a, layers["o"])
    n2 = rms_norm(h, eps)
    g = torch.nn.functional.silu(linear(n2, layers["gate"])) * linear(n2, layers["up"])
    return h + linear(g, layers["down"])


def block_fwd_bwd(x_bits: np.ndarray, dout_bits: np.ndarray, layers: Dict[str, LayerF64], batch: int, seq: int,
                  heads: int, eps: float = 1e-5, linear=slope_linear):
    """Forward and backward of the block for the loss <out, dOut>.

    Returns (out, dx, grads) as float64 numpy arrays; grads[name] = dict(dW=mask1 (.) dY^T X [d_out, d_in],
    dL, dR).  Clears the gradients held by ``layers`` first.
    """
    for lay in layers.values():
        for t in (lay.WR, lay.L, lay.R):
            if t is not None:
                t.grad = None
    x = torch.from_numpy(bf16_to_f64(x_bits)).requires_grad_(True)
    dout = torch.from_numpy(bf16_to_f64(dout_bits))
    out = decoder_block(x, layers, batch, seq, heads, eps, linear)
    out.backward(dout)
    grads = {}
    for name, lay in layers.items():
        grads[name] = {"dW": lay.WR.grad.numpy().copy(),
                       "dL": None if lay.L is None else lay.L.grad.numpy().copy(),
                       "dR": None if lay.R is None else lay.R.grad.numpy().copy()}
    return out.detach().numpy(), x.grad.numpy().copy(), grads
