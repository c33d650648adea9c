"""CPU oracle of the rest of a decode step around the BitLinear layers (paper Section 2: rotary position embeddings;
a Transformer decoder, hence causal attention - here with grouped queries as in the 2B configuration, 20 query heads
on 5 key/value heads; tokenizer with a vocabulary of 128,256, hence an embedding table and an output head of that
many rows).  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Everything here is the plain textbook definition evaluated in fp64 on the bf16 / fp32 inputs as given.  The paper
states none of the formulas; the readings (rotation base, pairing of the rotated coordinates, score scale, dtypes of
the cache) are listed in the design notes and are arguments where cheap.
"""
from __future__ import annotations

import numpy as np

from . import bf16_to_f32


def rope_angles(positions: np.ndarray, head_dim: int, base: float) -> np.ndarray:
    """theta[m, i] = pos[m] * base ** (-2 i / head_dim), i = 0 .. head_dim / 2 - 1 (fp64)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / head_dim)
    return np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]


def rope(x: np.ndarray, positions: np.ndarray, n_heads: int, head_dim: int, base: float = 500000.0) -> np.ndarray:
    """Rotary position embedding of x [M, n_heads * head_dim] (any float dtype, taken exactly): coordinate i of a head
    is paired with coordinate i + head_dim / 2;  (x_i, x_j) -> (x_i cos - x_j sin, x_j cos + x_i sin).  Returns fp64."""
    M = x.shape[0]
    xs = np.asarray(x, dtype=np.float64).reshape(M, n_heads, head_dim)
    th = rope_angles(positions, head_dim, base)
    c, s = np.cos(th)[:, None, :], np.sin(th)[:, None, :]
    half = head_dim // 2
    lo, hi = xs[..., :half], xs[..., half:]
    out = np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)
    return out.reshape(M, n_heads * head_dim)


def attention_decode(q_bits: np.ndarray, k_cache_bits: np.ndarray, v_cache_bits: np.ndarray, length: int, n_q_heads: int,
                     n_kv_heads: int, head_dim: int) -> np.ndarray:
    """One query token against the first `length` positions of a bf16 key / value cache.

    q_bits: uint16 [n_q_heads * head_dim]; caches: uint16 [T, n_kv_heads * head_dim].  Query head h reads key/value head
    h // (n_q_heads // n_kv_heads).  scores = q . k / sqrt(head_dim); softmax over the positions; output = sum p v (fp64)."""
    q = bf16_to_f32(q_bits).astype(np.float64).reshape(n_q_heads, head_dim)
    k = bf16_to_f32(k_cache_bits[:length]).astype(np.float64).reshape(length, n_kv_heads, head_dim)
    v = bf16_to_f32(v_cache_bits[:length]).astype(np.float64).reshape(length, n_kv_heads, head_dim)
    group = n_q_heads // n_kv_heads
    out = np.empty((n_q_heads, head_dim), np.float64)
    for h in range(n_q_heads):
        g = h // group
        s = k[:, g, :] @ q[h] / np.sqrt(float(head_dim))
        p = np.exp(s - s.max())
        p /= p.sum()
        out[h] = p @ v[:, g, :]
    return out.reshape(-1)


def lm_head(x_bits: np.ndarray, table_bits: np.ndarray) -> np.ndarray:
    """logits[m, v] = sum_k x[m, k] * E[v, k] on bf16 inputs, fp64."""
    x = bf16_to_f32(x_bits).astype(np.float64)
    e = bf16_to_f32(table_bits).astype(np.float64)
    return x @ e.T


def embed(ids: np.ndarray, table_bits: np.ndarray) -> np.ndarray:
    """Rows of the embedding table (bf16 bit patterns) for the given token ids."""
    return table_bits[np.asarray(ids, dtype=np.int64)]
