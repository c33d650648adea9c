"""CPU oracle of the chained decode benchmark: a stack of decoder layers in which every linear map is a
BitLinear (paper Section 2) and everything between them is written out step by step.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Per layer, for a hidden state h (bf16, [M, H]):

    q, k, v = BitLinear_q(h), BitLinear_k(h), BitLinear_v(h)              fp32 outputs
    a       = bf16( q + v[matching KV head] )                              stand-in for attention (attention is not
                                                                           a BitLinear; this keeps the dependence)
    h       = bf16( float(h) + BitLinear_o(a) )                            residual
    g, u    = BitLinear_gate(h), BitLinear_up(h)
    f       = bf16( (max(g, 0) * max(g, 0)) * u )                          squared ReLU gate (Section 2)
    h       = bf16( float(h) + BitLinear_down(f) )                         residual

Each BitLinear applies its own RMSNorm (subln) + absmax int8 quantiser to its input, as everywhere in this oracle.
Every arithmetic step is one fp32 operation; bf16() is round-to-nearest-even.
"""
from __future__ import annotations

import numpy as np

from . import bitlinear_forward, glue_attn_standin, glue_relu2, glue_residual


def _bitlinear(x_bits, mat, rms_eps):
    return bitlinear_forward(x_bits, mat.get("gain"), rms_eps, mat["wq"], mat["s_w"])["y"]


def decode_chain(h_bits: np.ndarray, layers, n_q_heads: int, n_kv_heads: int, head_dim: int, rms_eps: float):
    """h_bits: uint16 [M, H] bf16 bit patterns.  layers: list of dicts name -> dict(wq, s_w[, gain]) for the names
    q, k, v, o, gate, up, down.  Returns dict(h=final hidden bits, k=last layer's k projection fp32)."""
    h = np.array(h_bits, dtype=np.uint16, copy=True)
    k_last = None
    for layer in layers:
        q = _bitlinear(h, layer["q"], rms_eps)
        k_last = _bitlinear(h, layer["k"], rms_eps)
        v = _bitlinear(h, layer["v"], rms_eps)
        a_bits = glue_attn_standin(q, v, n_q_heads, n_kv_heads, head_dim)
        h = glue_residual(h, _bitlinear(a_bits, layer["o"], rms_eps))
        g = _bitlinear(h, layer["gate"], rms_eps)
        u = _bitlinear(h, layer["up"], rms_eps)
        f_bits = glue_relu2(g, u)
        h = glue_residual(h, _bitlinear(f_bits, layer["down"], rms_eps))
    return dict(h=h, k=k_last)
