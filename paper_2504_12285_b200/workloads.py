"""Seeded synthetic inputs shaped like the 2B BitNet b1.58 model's BitLinear layers.

This module only draws random numbers and casts dtypes.  It holds none of the
method's arithmetic (no quantiser, no norm, no packing), so both the CPU oracle's
tests and the CUDA path's tests / benchmark can feed on the very same bytes
without sharing any code of the method itself.

Shapes follow the paper's "2B" model (Section 2: BitLinear replaces every linear
layer; no bias): hidden 2560, FFN 6912, 20 query / 5 KV heads of 128, 30 layers.
Everything is generated on the host CPU so the bytes do not depend on the device.
"""
from __future__ import annotations

import numpy as np
import torch

HIDDEN = 2560
FFN = 6912
N_LAYERS = 30
HEAD_DIM = 128
N_Q_HEADS = 20
N_KV_HEADS = 5

# name -> (N out features, K in features); order is the order inside one layer.
LAYER_SHAPES = (
    ("q", HIDDEN, HIDDEN),
    ("k", N_KV_HEADS * HEAD_DIM, HIDDEN),
    ("v", N_KV_HEADS * HEAD_DIM, HIDDEN),
    ("o", HIDDEN, HIDDEN),
    ("gate", FFN, HIDDEN),
    ("up", FFN, HIDDEN),
    ("down", HIDDEN, FFN),
)
SHAPE_INDEX = {name: i for i, (name, _, _) in enumerate(LAYER_SHAPES)}
SHAPE_NK = {name: (n, k) for name, n, k in LAYER_SHAPES}

BASE_SEED = 20250412
WEIGHT_STD = 0.02
RMS_EPS = 1e-5
WEIGHT_EPS = 1e-5


def seed_for(config: int, shape_index: int = 0, trial: int = 0) -> int:
    """One seed per (benchmark configuration, layer shape, trial)."""
    return BASE_SEED + 1000 * config + 10 * shape_index + trial


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def latent_weights(n: int, k: int, seed: int) -> torch.Tensor:
    """fp32 [n, k] master weights ~ N(0, 0.02^2)."""
    return torch.randn(n, k, generator=_gen(seed), dtype=torch.float32).mul_(WEIGHT_STD)


def activations_normal(m: int, k: int, seed: int) -> torch.Tensor:
    """bf16 [m, k] activations ~ N(0, 1)."""
    return torch.randn(m, k, generator=_gen(seed), dtype=torch.float32).to(torch.bfloat16)


def activations_outlier(m: int, k: int, seed: int, frac: float = 0.01, scale: float = 20.0) -> torch.Tensor:
    """bf16 [m, k] ~ N(0, 1) with a seeded random 1% of the channels multiplied by 20."""
    g = _gen(seed)
    x = torch.randn(m, k, generator=g, dtype=torch.float32)
    n_out = max(1, int(round(frac * k)))
    chans = torch.randperm(k, generator=g)[:n_out]
    x[:, chans] *= scale
    return x.to(torch.bfloat16)


def activations_student_t(m: int, k: int, seed: int, dof: float = 3.0) -> torch.Tensor:
    """bf16 [m, k] ~ Student-t(3): heavy tails, so absmax scaling leaves most codes near 0."""
    rng = np.random.default_rng(int(seed))
    x = rng.standard_t(dof, size=(m, k)).astype(np.float32)
    return torch.from_numpy(x).to(torch.bfloat16)


def gain_ones(k: int) -> torch.Tensor:
    return torch.ones(k, dtype=torch.bfloat16)


def gain_random(k: int, seed: int) -> torch.Tensor:
    """bf16 [k] gains around 1 (used by tests so that the gain multiply is exercised)."""
    return (1.0 + 0.25 * torch.randn(k, generator=_gen(seed), dtype=torch.float32)).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """View a CPU bf16 tensor as a numpy uint16 array of the same shape (no copy of values)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    """Inverse of bf16_bits."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def layer_seed(config: int, layer: int, name: str) -> int:
    """Seed of one matrix of the 30-layer stack (independent per layer and per shape)."""
    return seed_for(config, SHAPE_INDEX[name], 0) + 100_000 * (layer + 1)
