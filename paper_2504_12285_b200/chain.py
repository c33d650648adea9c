"""Chained decode over a stack of decoder layers: argument marshalling for the benchmark's 30-layer configuration.

Every step runs in the library's kernels: per layer four batched BitLinear calls (q/k/v, o, gate/up, down - the
problems of a call share their input and are independent of each other), each with the element-wise step in front of
it (residual, attention stand-in, residual, squared-ReLU gate) fused into its quantiser - which at one token is part
of the same launch as the weight stream.  This module only owns
the buffers and the call order.
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
        bf = dict(dtype=torch.bfloat16, device=dev)
        # the hidden state alternates between two buffers: a fused residual step reads one and writes the other
        self.h_in, self.h_mid = torch.zeros(M, hidden, **bf), torch.zeros(M, hidden, **bf)
        self.q, self.k, self.v = torch.empty(M, hidden, **f32), torch.empty(M, kv, **f32), torch.empty(M, kv, **f32)
        self.o = torch.empty(M, hidden, **f32)
        self.g, self.u = torch.empty(M, ffn, **f32), torch.empty(M, ffn, **f32)
        self.dn = torch.empty(M, hidden, **f32)
        group = n_q_heads // n_kv_heads
        self.calls = []  # per layer: four (ProblemBatch, workspace)
        for li, layer in enumerate(layers):
            def item(name, x, y, step=None):
                packed, s_w, gain = layer[name]
                return (x, gain, packed, s_w, y) if step is None else (x, gain, packed, s_w, y, step)
            # the element-wise step in front of each level is fused into that level's quantiser launch:
            #   q,k,v : h = h_mid(previous layer) + down output  (plain input in the first layer)
            #   o     : attention stand-in on q and v
            #   gate,up: h_mid = h + o output
            #   down  : squared-ReLU gate
            res_in = None if li == 0 else (bl.X_RESIDUAL, self.dn, self.h_in, 0, 0)
            x_qkv = self.h_in if li == 0 else self.h_mid
            standin = (bl.X_ATTN_STANDIN, self.v, None, head_dim, group)
            res_mid = (bl.X_RESIDUAL, self.o, self.h_mid, 0, 0)
            relu2 = (bl.X_RELU2, self.u, None, 0, 0)
            groups = [[item("q", x_qkv, self.q, res_in), item("k", x_qkv, self.k, res_in), item("v", x_qkv, self.v, res_in)],
                      [item("o", self.q, self.o, standin)],
                      [item("gate", self.h_in, self.g, res_mid), item("up", self.h_in, self.u, res_mid)],
                      [item("down", self.g, self.dn, relu2)]]
            per_layer = []
            for grp in groups:
                batch = bl.ProblemBatch(grp, rms_eps)
                ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
                bl.bitlinear_forward_batch(batch, ws)  # uploads the plan; results are overwritten by step()
                per_layer.append((batch, ws))
            self.calls.append(per_layer)
        self.h = self.h_mid  # where the hidden state is after step()
        torch.cuda.synchronize(dev)

    @property
    def launches_per_layer(self) -> int:
        """One token: each of the four levels is one launch (the kernel quantises its input row itself); more tokens:
        4 x (quantiser with its fused element-wise step + weight stream)."""
        return 4 if self.M == 1 else 8

    def step(self, h0: torch.Tensor | None = None) -> torch.Tensor:
        """One pass over all layers, starting from h0 (bf16 [M, hidden]) or from the current hidden state."""
        self.h_in.copy_(self.h_mid if h0 is None else h0)
        for qkv, o, gu, down in self.calls:
            for batch, ws in (qkv, o, gu, down):
                bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
        bl.bitlinear_glue_residual_add(self.h_mid, self.dn)  # the last layer's residual
        return self.h_mid


class DecodeStep:
    """One whole decoded token for M sequences: embedding gather, per layer {q/k/v BitLinear, rotary embedding + cache
    append, grouped-query attention over the cache, o BitLinear, gate/up BitLinear, down BitLinear} with the residual
    adds and the squared-ReLU gate fused into the quantiser launches, then the output head.  Sequence m owns row m of
    every layer's cache."""

    def __init__(self, layers, embedding: torch.Tensor, M: int, t_max: int, hidden: int, ffn: int, n_q_heads: int,
                 n_kv_heads: int, head_dim: int, rms_eps: float = 1e-5, rope_base: float = 500000.0, device="cuda:0",
                 append_in_attention: bool = True):
        """layers: as for DecodeChain; embedding: bf16 [V, hidden], used for the gather and as the output head.
        append_in_attention: rotary embedding and cache append run inside the attention launches (same bits, one launch
        per layer fewer); False keeps them a launch of their own, which also leaves the rotated q in q_rot."""
        dev = torch.device(device)
        self.append_in_attention = append_in_attention
        self.rope_table = bl.bitlinear_rope_table(head_dim, t_max, rope_base, device=dev) if append_in_attention else None
        self.M, self.dims, self.rope_base, self.table = M, (n_q_heads, n_kv_heads, head_dim), rope_base, embedding
        kv = n_kv_heads * head_dim
        f32 = dict(dtype=torch.float32, device=dev)
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.h_in, self.h_mid = torch.zeros(M, hidden, **bf), torch.zeros(M, hidden, **bf)
        self.q, self.k, self.v = torch.empty(M, hidden, **f32), torch.empty(M, kv, **f32), torch.empty(M, kv, **f32)
        self.q_rot, self.attn = torch.empty(M, hidden, **bf), torch.empty(M, hidden, **bf)
        self.o = torch.empty(M, hidden, **f32)
        self.g, self.u = torch.empty(M, ffn, **f32), torch.empty(M, ffn, **f32)
        self.dn = torch.empty(M, hidden, **f32)
        self.logits = torch.empty(M, embedding.shape[0], **f32)
        self.k_cache = [torch.zeros(M, n_kv_heads, t_max, head_dim, **bf) for _ in layers]
        self.v_cache = [torch.zeros(M, n_kv_heads, t_max, head_dim, **bf) for _ in layers]
        self.seq_ids = torch.arange(M, dtype=torch.int32, device=dev)
        self.positions = torch.zeros(M, dtype=torch.int32, device=dev)  # where this token goes in its sequence
        self.lengths = torch.ones(M, dtype=torch.int32, device=dev)     # cache rows attended to: positions + 1
        self.attn_ws = torch.empty(bl.bitlinear_attention_workspace_bytes(M, n_q_heads, n_kv_heads, head_dim, t_max),
                                   dtype=torch.uint8, device=dev)
        self.calls = []
        for li, layer in enumerate(layers):
            def item(name, x, y, step=None):
                packed, s_w, gain = layer[name]
                return (x, gain, packed, s_w, y) if step is None else (x, gain, packed, s_w, y, step)
            res_in = None if li == 0 else (bl.X_RESIDUAL, self.dn, self.h_in, 0, 0)
            x_qkv = self.h_in if li == 0 else self.h_mid
            res_mid = (bl.X_RESIDUAL, self.o, self.h_mid, 0, 0)
            relu2 = (bl.X_RELU2, self.u, None, 0, 0)
            groups = [[item("q", x_qkv, self.q, res_in), item("k", x_qkv, self.k, res_in), item("v", x_qkv, self.v, res_in)],
                      [item("o", self.attn, self.o)],
                      [item("gate", self.h_in, self.g, res_mid), item("up", self.h_in, self.u, res_mid)],
                      [item("down", self.g, self.dn, relu2)]]
            per_layer = []
            for grp in groups:
                batch = bl.ProblemBatch(grp, rms_eps)
                ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
                bl.bitlinear_forward_batch(batch, ws)  # uploads the plan; results are overwritten by step()
                per_layer.append((batch, ws))
            self.calls.append(per_layer)
        torch.cuda.synchronize(dev)

    @property
    def launches_per_layer(self) -> int:
        """Four levels (one launch each at one token, quantiser + weight stream otherwise), attention slices, attention
        merge, and rotary/append where that is a launch of its own."""
        return (4 if self.M == 1 else 8) + (2 if self.append_in_attention else 3)

    def set_positions(self, positions: torch.Tensor) -> None:
        """positions: int32 [M] (device): where the next token of each sequence goes; it attends to rows 0 .. position."""
        self.positions.copy_(positions)
        torch.add(self.positions, 1, out=self.lengths)

    def step(self, ids: torch.Tensor) -> torch.Tensor:
        """ids: int32 [M] (device) -> logits fp32 [M, V]; appends this token's keys and values to every layer's cache."""
        n_q, n_kv, hd = self.dims
        bl.bitlinear_embed(ids, self.table, out=self.h_in)
        for li, (qkv, o, gu, down) in enumerate(self.calls):
            bl.bitlinear_forward_batch(*qkv, reuse_plan=True)
            if self.append_in_attention:
                bl.bitlinear_attention_decode_append(self.q, self.k, self.v, self.rope_table, self.k_cache[li], self.v_cache[li],
                                                     self.lengths, n_q, n_kv, hd, seq_ids=self.seq_ids, out=self.attn, ws=self.attn_ws)
            else:
                bl.bitlinear_rope_kv(self.q, self.k, self.v, self.positions, self.k_cache[li], self.v_cache[li], n_q, n_kv, hd,
                                     rope_base=self.rope_base, seq_ids=self.seq_ids, q_out=self.q_rot)
                bl.bitlinear_attention_decode(self.q_rot, self.k_cache[li], self.v_cache[li], self.lengths, n_q, n_kv, hd,
                                              seq_ids=self.seq_ids, out=self.attn, ws=self.attn_ws)
            for batch, ws in (o, gu, down):
                bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
        bl.bitlinear_glue_residual_add(self.h_mid, self.dn)  # the last layer's residual
        return bl.bitlinear_lm_head(self.h_mid, self.table, out=self.logits)

    def capture(self) -> None:
        """Record the launches of step() once into a CUDA graph; step_graph() then replays them without the host cost of
        a few hundred calls.  Token ids, positions and lengths are read from device buffers (ids_buf, positions, lengths), so one
        recording serves every later token: fill ids_buf and call set_positions() before each replay."""
        self.ids_buf = torch.zeros(self.M, dtype=torch.int32, device=self.h_in.device)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.step(self.ids_buf)  # every kernel has run once outside the recording
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=side):
                self.step(self.ids_buf)
        torch.cuda.current_stream().wait_stream(side)

    def step_graph(self) -> torch.Tensor:
        """Replay the recorded step on the current ids_buf / positions / lengths -> logits fp32 [M, V]."""
        self.graph.replay()
        return self.logits


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
