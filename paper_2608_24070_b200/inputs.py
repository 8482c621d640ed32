"""Seeded synthetic inputs shaped like the LLM-pretraining linear layers.

This module holds no arithmetic of the method: it only draws Gaussian tensors,
rounds them to bf16 (round-to-nearest-even) and names the workload shapes.  The
same bytes are handed to the CPU oracle and to the CUDA library.

bf16 tensors are numpy ``uint16`` arrays of raw bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np

BASE_SEED = 260824070
_ROLE = {"W": 0, "X": 1, "dY": 2, "L": 3, "R": 4}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def seed_for(config: int, layer: int, role: str) -> int:
    return BASE_SEED + 1000 * config + 10 * layer + _ROLE[role]


def gaussian_bf16(shape: Tuple[int, ...], sigma: float, seed: int) -> np.ndarray:
    """N(0, sigma^2) drawn in float32 with PCG64(seed), rounded to bf16."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.standard_normal(shape, dtype=np.float32) * np.float32(sigma)
    return f32_to_bf16_bits(x)


@dataclass(frozen=True)
class Layer:
    name: str
    d_in: int
    d_out: int


@dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration: a set of linear layers and a token count."""
    key: str
    config: int
    tokens: int
    layers: Tuple[Layer, ...]
    rank: int = 0           # adapter rank (0 = no adapter phase)
    sigma_w: float = 0.02   # std of W (GPT-2 style init)
    sigma_a: float = 0.01   # std of the adapter factors
    note: str = ""


WORKLOADS: Dict[str, Workload] = {
    "c1_single_512": Workload("c1_single_512", 1, 256, (Layer("lin", 512, 512),),
                              note="single layer 512->512, 256 tokens"),
    "c2_gpt2_small": Workload("c2_gpt2_small", 2, 8 * 1024,
                              (Layer("qkv", 768, 2304), Layer("fc", 768, 3072), Layer("proj", 3072, 768)),
                              note="GPT-2-small MLP pair + QKV, tokens 8x1024"),
    "c3_llama7b": Workload("c3_llama7b", 3, 16384,
                           (Layer("q", 4096, 4096), Layer("k", 4096, 4096), Layer("v", 4096, 4096),
                            Layer("o", 4096, 4096), Layer("gate", 4096, 11008), Layer("up", 4096, 11008),
                            Layer("down", 11008, 4096)),
                           note="LLaMA-7B projections, 16384 tokens"),
    "c4_llama7b_adapter": Workload("c4_llama7b_adapter", 4, 16384,
                                   (Layer("q", 4096, 4096), Layer("k", 4096, 4096), Layer("v", 4096, 4096),
                                    Layer("o", 4096, 4096), Layer("gate", 4096, 11008),
                                    Layer("up", 4096, 11008), Layer("down", 11008, 4096)),
                                   rank=64, note="LLaMA-7B projections + rank-64 lazy adapters"),
    "c5_llama13b_block": Workload("c5_llama13b_block", 5, 4 * 2048,
                                  (Layer("q", 5120, 5120), Layer("k", 5120, 5120), Layer("v", 5120, 5120),
                                   Layer("o", 5120, 5120), Layer("gate", 5120, 13824),
                                   Layer("up", 5120, 13824), Layer("down", 13824, 5120)),
                                  rank=128, note="LLaMA-13B-width block linears, seq 2048 x batch 4, rank-128"),
}


def layer_tensors(wl: Workload, layer_idx: int, tokens: int | None = None,
                  want: Tuple[str, ...] = ("W", "X", "dY", "L", "R")) -> Dict[str, np.ndarray]:
    """Draw the tensors of one layer of a workload (bf16 bit patterns).

    W [d_out, d_in] ~ N(0, sigma_w^2); X [b, d_in], dY [b, d_out] ~ N(0, 1);
    L [d_in, r], R [r, d_out] ~ N(0, sigma_a^2) when the workload has adapters.
    """
    lay = wl.layers[layer_idx]
    b = wl.tokens if tokens is None else tokens
    out: Dict[str, np.ndarray] = {}
    if "W" in want:
        out["W"] = gaussian_bf16((lay.d_out, lay.d_in), wl.sigma_w, seed_for(wl.config, layer_idx, "W"))
    if "X" in want:
        out["X"] = gaussian_bf16((b, lay.d_in), 1.0, seed_for(wl.config, layer_idx, "X"))
    if "dY" in want:
        out["dY"] = gaussian_bf16((b, lay.d_out), 1.0, seed_for(wl.config, layer_idx, "dY"))
    if wl.rank > 0:
        if "L" in want:
            out["L"] = gaussian_bf16((lay.d_in, wl.rank), wl.sigma_a, seed_for(wl.config, layer_idx, "L"))
        if "R" in want:
            out["R"] = gaussian_bf16((wl.rank, lay.d_out), wl.sigma_a, seed_for(wl.config, layer_idx, "R"))
    return out


def sample_indices(n: int, count: int, seed: int) -> np.ndarray:
    """Seeded sample of row indices in [0, n): always the first and last row and one
    row on each side of every 128-boundary that fits, the rest uniform."""
    must: List[int] = [0, n - 1]
    if n > 256:
        must += [127, 128, n - 129, n - 128]
    rng = np.random.Generator(np.random.PCG64(seed))
    extra = rng.choice(n, size=min(n, max(0, count)), replace=False).tolist()
    seen: List[int] = []
    for v in must + extra:
        if 0 <= v < n and v not in seen:
            seen.append(v)
        if len(seen) >= min(count, n):
            break
    return np.array(sorted(seen), dtype=np.int32)
