"""LLaMA-style decoder block around the library's linear layer: integration and timing harness.

The seven linear layers (q, k, v, o, gate, up, down) run through the C-ABI calls, wired into
torch autograd by a ``torch.autograd.Function`` whose backward issues the adapter backward, the
input gradient with the doubly pruned weight and the masked compressed weight gradient
(Eq. (sparse_forward), Eq. (sparse_backward_input), Eq. (sparse_backward_weight), Eq. (concat)).
Everything between them -- RMS normalisation without gain, causal attention without positional
rotation, the SiLU gate, the residual adds -- is plain torch in bf16 and is NOT part of the
library: it is there so that the linears see a real data flow, each one fed by the previous
one's output and its gradient by the next one's.  ``DenseLinear`` is the same block on
``torch.nn.functional.linear`` (cuBLAS) for the all-dense comparison.

Every linear call is bracketed by CUDA events when ``timers`` is given, so the time spent in
the linears can be summed separately from the torch glue.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import torch
import torch.nn.functional as F

from . import binding as B

LAYER_NAMES = ("q", "k", "v", "o", "gate", "up", "down")
Timers = List[Tuple[torch.cuda.Event, torch.cuda.Event]]


def _timed(timers: Optional[Timers], fn):
    if timers is None:
        return fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    out = fn()
    e1.record()
    timers.append((e0, e1))
    return out


def elapsed_ms(timers: Timers) -> float:
    """Sum of the bracketed intervals; synchronise the device first."""
    return sum(a.elapsed_time(b) for a, b in timers)


class SlopeLinear:
    """One 2:4-sparse layer: compressed weight and its doubly pruned transposed copy, static masks,
    optional lazy adapters, and the gradient buffers the backward fills (dWc compressed, dL, dR)."""

    def __init__(self, W: torch.Tensor, L: Optional[torch.Tensor] = None, R: Optional[torch.Tensor] = None,
                 max_tokens: int = 0):
        self.d_out, self.d_in = W.shape
        self.Wc_vals, self.Wc_meta, self.mask1 = B.alloc_compressed(self.d_out, self.d_in)
        self.WTc_vals, self.WTc_meta, _ = B.alloc_compressed(self.d_in, self.d_out)
        B.slope_prune_24_double(W, self.Wc_vals, self.Wc_meta, self.mask1, self.WTc_vals, self.WTc_meta, None)
        self.L, self.R = L, R
        self.r = 0 if L is None else L.shape[1]
        self.dWc = torch.empty_like(self.Wc_vals)
        self.dL = None if L is None else torch.empty_like(L)
        self.dR = None if R is None else torch.empty_like(R)
        self.workspace = None
        if self.r and max_tokens:
            n = B.slope_adapter_workspace_bytes(max_tokens, self.d_out, self.d_in, self.r)
            self.workspace = torch.empty(max(n, 16), dtype=torch.uint8, device=W.device)
        self.timers: Optional[Timers] = None

    def __call__(self, X: torch.Tensor) -> torch.Tensor:
        return _SlopeLinearFn.apply(X, self)


class _SlopeLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, X, layer: SlopeLinear):
        X = X.contiguous()
        b = X.shape[0]
        Y = torch.empty(b, layer.d_out, dtype=torch.bfloat16, device=X.device)
        T = None

        def run():
            nonlocal T
            if layer.r:
                T = torch.empty(b, layer.r, dtype=torch.bfloat16, device=X.device)
                B.slope_linear_fwd_adapter(X, layer.Wc_vals, layer.Wc_meta, layer.d_out, layer.L, layer.R, T, Y)
            else:
                B.slope_linear_fwd(X, layer.Wc_vals, layer.Wc_meta, layer.d_out, Y)

        _timed(layer.timers, run)
        ctx.layer = layer
        ctx.save_for_backward(X, T) if T is not None else ctx.save_for_backward(X)
        return Y

    @staticmethod
    def backward(ctx, dY):
        layer: SlopeLinear = ctx.layer
        saved = ctx.saved_tensors
        X, T = saved[0], (saved[1] if len(saved) > 1 else None)
        dY = dY.contiguous()
        b = X.shape[0]
        dX = torch.empty(b, layer.d_in, dtype=torch.bfloat16, device=X.device)

        def run():
            dT = None
            if layer.r:
                dT = torch.empty(b, layer.r, dtype=torch.bfloat16, device=X.device)
                need = B.slope_adapter_workspace_bytes(b, layer.d_out, layer.d_in, layer.r)
                if layer.workspace is None or layer.workspace.numel() < need:
                    layer.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=X.device)
                B.slope_adapter_fwd_bwd(1, X, dY, layer.L, layer.R, b, layer.d_out, layer.d_in, layer.r, T=T, dT=dT,
                                        dL=layer.dL, dR=layer.dR, workspace=layer.workspace)
            B.slope_linear_bwd_dx(dY, layer.WTc_vals, layer.WTc_meta, layer.d_in, dX, dT, layer.L)
            B.slope_linear_bwd_dw_masked(dY, X, layer.mask1, layer.dWc)

        _timed(layer.timers, run)
        return dX, None


class DenseLinear:
    """The dense bf16 layer on torch (cuBLAS): Y = X W^T, gradients by autograd."""

    def __init__(self, W: torch.Tensor):
        self.W = W.clone().requires_grad_(True)
        self.timers: Optional[Timers] = None

    def __call__(self, X: torch.Tensor) -> torch.Tensor:
        return _DenseLinearFn.apply(X, self.W, self)


class _DenseLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, X, W, layer: DenseLinear):
        ctx.layer = layer
        ctx.save_for_backward(X, W)
        return _timed(layer.timers, lambda: F.linear(X, W))

    @staticmethod
    def backward(ctx, dY):
        X, W = ctx.saved_tensors
        dX, dW = _timed(ctx.layer.timers, lambda: (dY @ W, dY.t() @ X))
        return dX, dW, None


def rms_norm(x: torch.Tensor, eps: float) -> torch.Tensor:
    xf = x.float()
    return (xf * torch.rsqrt((xf * xf).mean(dim=-1, keepdim=True) + eps)).to(x.dtype)


def causal_attention(q, k, v, batch: int, seq: int, heads: int) -> torch.Tensor:
    hd = q.shape[1] // heads
    split = lambda t: t.reshape(batch, seq, heads, hd).permute(0, 2, 1, 3)
    out = F.scaled_dot_product_attention(split(q), split(k), split(v), is_causal=True)
    return out.permute(0, 2, 1, 3).reshape(batch * seq, heads * hd)


def decoder_block(x: torch.Tensor, layers: Dict[str, object], batch: int, seq: int, heads: int,
                  eps: float = 1e-5) -> torch.Tensor:
    """x [batch*seq, d] bf16 -> block output [batch*seq, d] bf16; ``layers`` maps the seven names to callables."""
    n1 = rms_norm(x, eps)
    a = causal_attention(layers["q"](n1), layers["k"](n1), layers["v"](n1), batch, seq, heads)
    h = x + layers["o"](a)
    n2 = rms_norm(h, eps)
    g = F.silu(layers["gate"](n2)) * layers["up"](n2)
    return h + layers["down"](g)


def block_step(x: torch.Tensor, dout: torch.Tensor, layers: Dict[str, object], batch: int, seq: int, heads: int,
               eps: float = 1e-5):
    """One training step of the block for the loss <out, dOut> (no optimizer): returns (out, dx)."""
    x = x.detach().requires_grad_(True)
    out = decoder_block(x, layers, batch, seq, heads, eps)
    out.backward(dout)
    return out.detach(), x.grad
