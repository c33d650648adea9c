"""Chained decode over a stack of decoder layers: argument marshalling for the benchmark's 30-layer configuration.

Every step runs in the library's kernels: per layer four batched BitLinear calls (q/k/v, o, gate/up, down - the
problems of a call share their input and are independent of each other) and four element-wise glue launches
(attention stand-in, residual, squared-ReLU gate, residual).  This module only owns the buffers and the call order.
"""
from __future__ import annotations

import torch

from . import binding as bl


class DecodeChain:
    def __init__(self, layers, M: int, hidden: int, ffn: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 rms_eps: float = 1e-5, device="cuda:0"):
        """layers: list of dicts name -> (packed uint8, s_w fp32 [1], gain bf16 [K] or None) for q,k,v,o,gate,up,down."""
        dev = torch.device(device)
        self.M, self.dims = M, (n_q_heads, n_kv_heads, head_dim)
        kv = n_kv_heads * head_dim
        f32 = dict(dtype=torch.float32, device=dev)
        self.h = torch.zeros(M, hidden, dtype=torch.bfloat16, device=dev)
        self.q, self.k, self.v = torch.empty(M, hidden, **f32), torch.empty(M, kv, **f32), torch.empty(M, kv, **f32)
        self.a = torch.empty(M, hidden, dtype=torch.bfloat16, device=dev)
        self.o = torch.empty(M, hidden, **f32)
        self.g, self.u = torch.empty(M, ffn, **f32), torch.empty(M, ffn, **f32)
        self.f = torch.empty(M, ffn, dtype=torch.bfloat16, device=dev)
        self.dn = torch.empty(M, hidden, **f32)
        self.calls = []  # per layer: four (ProblemBatch, workspace)
        for layer in layers:
            def item(name, x, y):
                packed, s_w, gain = layer[name]
                return (x, gain, packed, s_w, y)
            groups = [[item("q", self.h, self.q), item("k", self.h, self.k), item("v", self.h, self.v)],
                      [item("o", self.a, self.o)],
                      [item("gate", self.h, self.g), item("up", self.h, self.u)],
                      [item("down", self.f, self.dn)]]
            per_layer = []
            for grp in groups:
                batch = bl.ProblemBatch(grp, rms_eps)
                ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
                bl.bitlinear_forward_batch(batch, ws)  # uploads the plan; results are overwritten by step()
                per_layer.append((batch, ws))
            self.calls.append(per_layer)
        torch.cuda.synchronize(dev)

    launches_per_layer = 12  # 4 x (quantiser + weight stream) + 4 glue kernels

    def step(self, h0: torch.Tensor | None = None) -> torch.Tensor:
        """One pass over all layers, starting from h0 (bf16 [M, hidden]) or from the current hidden state."""
        if h0 is not None:
            self.h.copy_(h0)
        nq, nkv, hd = self.dims
        for qkv, o, gu, down in self.calls:
            bl.bitlinear_forward_batch(qkv[0], qkv[1], reuse_plan=True)
            bl.bitlinear_glue_attn_standin(self.q, self.v, self.a, nq, nkv, hd)
            bl.bitlinear_forward_batch(o[0], o[1], reuse_plan=True)
            bl.bitlinear_glue_residual_add(self.h, self.o)
            bl.bitlinear_forward_batch(gu[0], gu[1], reuse_plan=True)
            bl.bitlinear_glue_relu2_mul(self.g, self.u, self.f)
            bl.bitlinear_forward_batch(down[0], down[1], reuse_plan=True)
            bl.bitlinear_glue_residual_add(self.h, self.dn)
        return self.h


class PersistentChain:
    """The same chain at one token through bitlinear_decode_chain: one cooperative kernel per token."""

    def __init__(self, layers, hidden: int, ffn: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 rms_eps: float = 1e-5, device="cuda:0"):
        """layers: list of dicts q,k,v,o,gate,up,down -> (packed, s_w) and "gains" -> 4 x (bf16 [K] or None)."""
        dev = torch.device(device)
        self.dims = (hidden, ffn, n_q_heads, n_kv_heads, head_dim)
        self.eps = rms_eps
        self.table = bl.ChainLayers(layers)
        self.h = torch.zeros(1, hidden, dtype=torch.bfloat16, device=dev)
        self.k = torch.empty(n_kv_heads * head_dim, dtype=torch.float32, device=dev)
        self.ws = torch.empty(bl.bitlinear_decode_chain_workspace_bytes(len(layers), *self.dims), dtype=torch.uint8, device=dev)
        self.uploaded = False

    def step(self, h0: torch.Tensor | None = None) -> torch.Tensor:
        if h0 is not None:
            self.h.copy_(h0)
        bl.bitlinear_decode_chain(self.table, *self.dims, self.h, self.ws, self.eps, k_out=self.k, reuse_plan=self.uploaded)
        self.uploaded = True
        return self.h
