#!/usr/bin/env python
"""Benchmark of the B200 BitLinear library.

Headline line (one JSON object on stdout, rank 0): decode throughput in GB/s of packed-weight
bytes at M = 1 over the seven BitLinear shapes of a 2B-style layer, rotated over 30 independently
seeded layers (210 matmuls, 521 MB of packed weights > L2, so every weight byte comes from HBM).
The same line carries the prefill result (int8 TOPS at M = 2048), the roofline of the dominant
kernel, the end-to-end number with host buffers, and the CPU oracle timed on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_12285_b200 import replicas  # noqa: E402
from paper_2504_12285_b200 import workloads as wl  # noqa: E402

METRIC = "bitlinear_decode_packed_weight_bandwidth_m1"
UNIT = "GB/s"
CONFIG_ID = 2  # seed family of the headline workload: a decode step over all 7 BitLinear shapes of a 2B-style layer, 30 layers
WORKLOAD = ("configs[1] at M=1: decode step over the 7 BitLinear shapes of a 2B-style layer "
            "(q,k,v,o,gate,up,down), rotated over 30 independently seeded layers = 210 forwards, "
            "521,011,200 packed-weight bytes per step")
PREFILL_M = 2048


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


def cuda_time_ms(fn, stream=None):
    """Device time of fn() on torch's current stream, with a synchronise on both sides."""
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def measure_int8_peak(bl):
    """tcgen05.mma kind::i8 on shared-memory-resident operands, every SM, no global traffic: TOP/s, best of 3."""
    bl.bitlinear_probe_int8_mma_rate(1000)
    best = 0.0
    for _ in range(3):
        ops = [0.0]
        ms = cuda_time_ms(lambda: ops.__setitem__(0, bl.bitlinear_probe_int8_mma_rate(100000)))
        best = max(best, ops[0] / ms / 1e9)
    return best


def avg_call_us(calls, warm=3):
    """Average device time per call of a back-to-back sequence (the list is run once after `warm` untimed calls)."""
    for c in calls[:warm]:
        c()
    return cuda_time_ms(lambda: [c() for c in calls]) * 1e3 / len(calls)


# --------------------------------------------------------------------------------------------- ours


def build_decode_pool(bl, dev, n_layers):
    """Packs n_layers x 7 seeded weight matrices on the GPU.  Returns list of dicts per matmul."""
    pool = []
    for layer in range(n_layers):
        for name, n, k in wl.LAYER_SHAPES:
            W = wl.latent_weights(n, k, wl.layer_seed(CONFIG_ID, layer, name)).to(dev, non_blocking=False)
            packed, s_w = bl.bitlinear_pack_weights(W, wl.WEIGHT_EPS)
            del W
            pool.append(dict(name=name, N=n, K=k, packed=packed, s_w=s_w))
    torch.cuda.synchronize()
    return pool


def run_ours(args):
    from paper_2504_12285_b200 import binding as bl

    rank, local_rank, world = replicas.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bl.lib()  # fail loudly here if the library cannot be built / loaded
    peaks = load_peaks()
    M = 1
    n_layers = wl.N_LAYERS

    pool = build_decode_pool(bl, dev, n_layers)
    packed_bytes = sum(p["packed"].numel() for p in pool)
    assert packed_bytes == 521_011_200
    gains = {k: wl.gain_ones(k).to(dev) for k in (wl.HIDDEN, wl.FFN)}
    # activations and outputs live in two arenas (one slot per forward) so that the end-to-end leg can
    # move them with one copy each way
    x_off, y_off, xo, yo = [], [], 0, 0
    for p in pool:
        x_off.append(xo)
        y_off.append(yo)
        xo += (M * p["K"] * 2 + 255) // 256 * 256
        yo += (M * p["N"] * 4 + 255) // 256 * 256
    x_host = torch.empty(xo, dtype=torch.uint8).pin_memory()
    y_host = torch.empty(yo, dtype=torch.uint8).pin_memory()
    x_dev = torch.empty(xo, dtype=torch.uint8, device=dev)
    y_dev = torch.empty(yo, dtype=torch.uint8, device=dev)
    shape_x = {name: wl.activations_normal(M, k, wl.seed_for(CONFIG_ID, i)) for i, (name, n, k) in enumerate(wl.LAYER_SHAPES)}
    items = []
    for p, xo_, yo_ in zip(pool, x_off, y_off):
        nb = M * p["K"] * 2
        x_host[xo_:xo_ + nb] = shape_x[p["name"]].view(torch.uint8).reshape(-1)
        xv = x_dev[xo_:xo_ + nb].view(torch.bfloat16).view(M, p["K"])
        yv = y_dev[yo_:yo_ + M * p["N"] * 4].view(torch.float32).view(M, p["N"])
        items.append((xv, gains[p["K"]], p["packed"], p["s_w"], yv))
    x_dev.copy_(x_host)
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
    bl.bitlinear_forward_batch(batch, ws)  # uploads the plan once

    def step():
        bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)

    launches_per_step = 2  # one quantiser launch over all tokens + one persistent weight-streaming launch

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    replicas.barrier()
    with ClockSampler(local_rank) as clocks:
        ms = cuda_time_ms(lambda: [step() for _ in range(args.steps)])
    replicas.barrier()
    sec = ms / 1e3
    value, slowest = replicas.aggregate_throughput(packed_bytes * args.steps / 1e9, sec, device=str(dev))
    ms_per_step = slowest * 1e3 / args.steps

    # ---- roofline of the dominant kernel: the persistent weight-streaming kernel, timed alone ----
    n_alone = max(5, args.steps)
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True)
    stream_s = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True)
                                     for _ in range(n_alone)]) / n_alone / 1e3
    achieved = packed_bytes / stream_s / 1e9
    roofline = {"bound": "hbm", "kernel": "decode_stream_kernel (persistent decode contraction, 210 matmuls per launch)",
                "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4), "algorithmic_bytes_per_launch": packed_bytes,
                "avg_launch_us": round(stream_s * 1e6, 2),
                # dram__bytes_read.sum + dram__bytes_write.sum of this kernel on 10 of the 30 layers (173.96 MB + 4.00 MB,
                # profiles/decode_stream_10layers_m1.md), times 3: it streams every packed byte once
                "traffic": 3 * (173959936 + 4003584),
                "traffic_source": "ncu capture of a 10-layer launch (profiles/decode_stream_10layers_m1.md) scaled x3, not measured in this run"}

    # ---- sustained leg: the same step repeated for at least half a second, with the SM clock sampled meanwhile ----
    sustained = None
    if rank == 0:
        n_sus = max(200, int(0.6 / max(ms_per_step * 1e-3, 1e-6)))
        with ClockSampler(local_rank) as clk_s:
            ms_sus = cuda_time_ms(lambda: [step() for _ in range(n_sus)])
        cs = clk_s.summary()
        sustained = {"steps": n_sus, "seconds": round(ms_sus / 1e3, 3), "ms_per_step": round(ms_sus / n_sus, 4),
                     "value": round(packed_bytes * n_sus / ms_sus / 1e6, 1), "unit": UNIT,
                     "frac_of_hbm_peak": round(packed_bytes * n_sus / ms_sus / 1e6 / peaks["hbm_gbs"], 4), "clocks": cs,
                     "us_per_step_x_sm_ghz": None if not cs["sm_mhz"] else round(ms_sus / n_sus * cs["sm_mhz"], 1)}

    # ---- the same 210 forwards as separate bitlinear_forward calls (two launches each), for comparison ----
    ws_call = torch.empty(max(bl.bitlinear_workspace_bytes(M, n, k) for _, n, k in wl.LAYER_SHAPES), dtype=torch.uint8,
                          device=dev)

    def step_calls():
        for xv, g, packed, s_w, yv in items:
            bl.bitlinear_forward(xv, g, packed, s_w, yv.shape[1], wl.RMS_EPS, ws=ws_call, out=yv)

    step_calls()
    ms_calls = cuda_time_ms(lambda: [step_calls() for _ in range(3)]) / 3
    per_call = {"api": "bitlinear_forward, one call per BitLinear", "ms_per_step": round(ms_calls, 4),
                "value": round(packed_bytes / ms_calls / 1e6, 1), "unit": UNIT}

    # ---- end to end with host buffers through bitlinear_forward_batch_host ----
    e2e = None
    if True:
        # a workspace of its own: the call may run as three segments (copies beside kernels), each with its own plan
        ws_host = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
        bl.bitlinear_forward_batch_host(batch, x_host, x_dev, y_dev, y_host, ws_host)

        def step_host():
            bl.bitlinear_forward_batch_host(batch, x_host, x_dev, y_dev, y_host, ws_host, reuse_plan=True)

        for _ in range(3):
            step_host()
        replicas.barrier()
        t0 = time.perf_counter()
        ms_h = cuda_time_ms(lambda: [step_host() for _ in range(args.steps)])
        wall_h = (time.perf_counter() - t0) * 1e3
        replicas.barrier()
        # the call synchronises, so host wall clock and device events bracket the same work; the slower one counts
        v_h, _ = replicas.aggregate_throughput(packed_bytes * args.steps / 1e9, max(ms_h, wall_h) / 1e3, device=str(dev))
        e2e = {"value": round(v_h, 2), "unit": UNIT, "ms_per_step": round(max(ms_h, wall_h) / args.steps, 4),
               "device_ms_per_step": round(ms_h / args.steps, 4), "wall_ms_per_step": round(wall_h / args.steps, 4),
               "h2d_bytes_per_step": int(x_host.numel()), "d2h_bytes_per_step": int(y_host.numel()),
               "api": "bitlinear_forward_batch_host: pinned x arena -> device, quantiser + stream launches, y arena -> pinned host, "
                      "sync; run as three segments so that one segment's copies overlap another's kernels"}

    # ---- the same step at M = 4, 8 and 16 tokens per forward (rank 0 only): the tensor-core decode kernels ----
    decode_m = {}
    if rank == 0:
        for m in (4, 8, 16):
            its = [(wl.activations_normal(m, p["K"], wl.seed_for(CONFIG_ID, i % 7, m)).to(dev), gains[p["K"]], p["packed"],
                    p["s_w"], torch.empty(m, p["N"], dtype=torch.float32, device=dev)) for i, p in enumerate(pool)]
            bm = bl.ProblemBatch(its, wl.RMS_EPS)
            wm = torch.empty(bm.workspace_bytes(), dtype=torch.uint8, device=dev)
            bl.bitlinear_forward_batch(bm, wm)
            for _ in range(2):
                bl.bitlinear_forward_batch(bm, wm, reuse_plan=True)
            n_m = max(3, args.steps // 4)
            ms_m = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(bm, wm, reuse_plan=True) for _ in range(n_m)]) / n_m
            ms_k = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(bm, wm, reuse_plan=True, reuse_act=True)
                                         for _ in range(n_m)]) / n_m
            decode_m[f"M={m}"] = {"ms_per_step": round(ms_m, 4), "value": round(packed_bytes / ms_m / 1e6, 1), "unit": UNIT,
                                  "frac_of_hbm_peak": round(packed_bytes / ms_m / 1e6 / peaks["hbm_gbs"], 4),
                                  "kernel": "decode_stream_mma_kernel (the one-token weight stream feeding int8 mma.sync)" if m <= 8 else
                                            "decode_mma_kernel (weights unpacked into tensor memory, tcgen05 kind::i8)",
                                  "kernel_alone_ms": round(ms_k, 4),
                                  "kernel_alone_frac_of_hbm_peak": round(packed_bytes / ms_k / 1e6 / peaks["hbm_gbs"], 4)}
            del its, bm, wm

    # ---- configs[0]: one q-projection forward at M = 1: isolated call latency and steady state over rotating copies ----
    config1 = None
    if rank == 0:
        config1 = run_config1(bl, dev, peaks)

    # ---- the same step with the weights in the dense layout, five values per byte (rank 0 only) ----
    dense = None
    if rank == 0:
        dense = run_dense(bl, dev, peaks, items, ms_per_step, reps=max(5, args.steps))

    # ---- configs[4]: batch sweep on the FFN down projection, every legal path forced (rank 0 only) ----
    sweep = None
    int8_peak = None
    if rank == 0:
        int8_peak = measure_int8_peak(bl)
        sweep = run_sweep(bl, dev, peaks, int8_peak)

    # ---- the 30-layer stack as a dependent chain (configs[2]): 210 matmuls, glue in between, M = 1 (rank 0 only) ----
    chain = None
    if rank == 0:
        chain = run_chain(bl, dev, pool, gains, peaks, packed_bytes, reps=max(5, args.steps))

    # ---- a whole decoded token: the chain plus rotary embedding, attention over a 4096-token cache, output head ----
    decode_step = None
    if rank == 0:
        decode_step = run_decode_step(bl, dev, pool, gains, peaks, packed_bytes, reps=max(5, args.steps))
        # the same with 16 sequences: attention then streams 168 MB per layer and is bound by bandwidth, not latency
        decode_step["sixteen_sequences"] = run_decode_step(bl, dev, pool, gains, peaks, packed_bytes, reps=5, M=16)
        torch.cuda.empty_cache()

    # ---- prefill: int8 tensor-core path at M = 2048 on the 7 shapes (rank 0 only) ----
    prefill = None
    if rank == 0:
        prefill = run_prefill(bl, dev, pool, gains, peaks, int8_peak, reps=max(3, min(args.steps, 10)))

    # ---- CPU oracle on the host cores (rank 0, N = 1 only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_decode_baseline(budget_s=15.0)

    if rank == 0:
        out = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "s8 x ternary -> s32 (fp32 epilogue)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "matmuls_per_step": len(pool),
                       "packed_bytes_per_step": packed_bytes,
                       "l2": "inputs larger than L2: 521 MB of packed weights per step, each byte read once",
                       "parallelism": "replicas only (no collective)" if world > 1 else "single GPU"},
            "frac_of_hbm_peak": round(value / world / peaks["hbm_gbs"], 4),
            "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "sustained": sustained, "per_call": per_call, "config1": config1,
            "decode_more_tokens": decode_m, "dense_layout": dense, "chain": chain, "decode_step": decode_step,
            "prefill": prefill, "sweep": sweep,
            "cpu_baseline": cpu,
        }
        print(json.dumps(out))
    replicas.finalize()


def run_chain(bl, dev, pool, gains, peaks, packed_bytes, reps):
    """configs[2]: every matmul of the 30-layer stack depends on the one before (RMSNorm + quantiser per BitLinear
    input, squared-ReLU gate, residuals, attention stand-in); one pass = one decoded token at M = 1."""
    from paper_2504_12285_b200 import chain as gpu_chain

    layers = []
    for layer in range(wl.N_LAYERS):
        mats = pool[layer * 7:(layer + 1) * 7]
        layers.append({m["name"]: (m["packed"], m["s_w"], gains[m["K"]]) for m in mats})
    ch = gpu_chain.DecodeChain(layers, 1, wl.HIDDEN, wl.FFN, wl.N_Q_HEADS, wl.N_KV_HEADS, wl.HEAD_DIM, wl.RMS_EPS, dev)
    h0 = wl.activations_normal(1, wl.HIDDEN, wl.seed_for(3)).to(dev)
    ch.step(h0)
    eager_ms = cuda_time_ms(lambda: [ch.step(h0) for _ in range(reps)]) / reps
    out = {"workload": "configs[2]: 30 layers x 7 BitLinear as a dependent chain at M=1 (210 matmuls, 120 fused "
                       "RMSNorm+quantiser inputs, glue kernels in between)",
           "launches_per_token": wl.N_LAYERS * ch.launches_per_layer + 1,
           "eager_us_per_token": round(eager_ms * 1e3, 1),
           "eager_value": round(packed_bytes / eager_ms / 1e6, 1), "unit": UNIT}
    try:  # the same launches replayed from a CUDA graph (no host launch cost)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            ch.step(h0)
            with torch.cuda.graph(graph, stream=side):
                ch.step(h0)
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        graph_ms = cuda_time_ms(lambda: [graph.replay() for _ in range(reps)]) / reps
        out.update({"graph_us_per_token": round(graph_ms * 1e3, 1), "graph_value": round(packed_bytes / graph_ms / 1e6, 1),
                    "graph_frac_of_hbm_peak": round(packed_bytes / graph_ms / 1e6 / peaks["hbm_gbs"], 4)})
    except Exception as exc:  # capture refused: keep the eager number
        out["graph"] = f"not captured: {type(exc).__name__}"
    # the same token through ONE persistent cooperative kernel (grid barriers instead of kernel boundaries)
    pl = [dict({m["name"]: (m["packed"], m["s_w"]) for m in pool[layer * 7:(layer + 1) * 7]},
               gains=[gains[wl.HIDDEN], gains[wl.HIDDEN], gains[wl.HIDDEN], gains[wl.FFN]]) for layer in range(wl.N_LAYERS)]
    pc = gpu_chain.PersistentChain(pl, wl.HIDDEN, wl.FFN, wl.N_Q_HEADS, wl.N_KV_HEADS, wl.HEAD_DIM, wl.RMS_EPS, dev)
    h_ref = ch.step(h0).clone()
    h_p = pc.step(h0).clone()
    torch.cuda.synchronize()
    pers_ms = cuda_time_ms(lambda: [pc.step(h0) for _ in range(reps)]) / reps
    out.update({"persistent_us_per_token": round(pers_ms * 1e3, 1), "persistent_value": round(packed_bytes / pers_ms / 1e6, 1),
                "persistent_frac_of_hbm_peak": round(packed_bytes / pers_ms / 1e6 / peaks["hbm_gbs"], 4),
                "persistent_launches_per_token": 1,
                "persistent_equals_per_level_calls": bool(torch.equal(h_ref, h_p))})
    return out


def graph_time_ms(fn, reps):
    """fn's launches captured once into a CUDA graph; mean device time of a replay.  None if the capture is refused."""
    try:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        return cuda_time_ms(lambda: [graph.replay() for _ in range(reps)]) / reps
    except Exception:
        return None


def run_decode_step(bl, dev, pool, gains, peaks, packed_bytes, reps, M=1, context=4096):
    """One whole decoded token of the 2B configuration at M sequences with `context` - 1 tokens already in the cache:
    embedding gather, 30 x {q/k/v, rotary embedding + cache append, grouped-query attention, o, gate/up, down}, output
    head over the 128,256-row table.  The cache and the table are bf16; the parts that are not BitLinear are timed on
    their own as well (the 30 attention calls read 30 different caches, 315 MB at M = 1: larger than L2)."""
    from paper_2504_12285_b200 import chain as gpu_chain

    vocab = 128256
    layers = []
    for layer in range(wl.N_LAYERS):
        layers.append({m["name"]: (m["packed"], m["s_w"], gains[m["K"]]) for m in pool[layer * 7:(layer + 1) * 7]})
    gen = torch.Generator(device=dev).manual_seed(wl.seed_for(5))
    table = (torch.randn(vocab, wl.HIDDEN, generator=gen, device=dev) * 0.02).to(torch.bfloat16)
    st = gpu_chain.DecodeStep(layers, table, M, context, wl.HIDDEN, wl.FFN, wl.N_Q_HEADS, wl.N_KV_HEADS, wl.HEAD_DIM, wl.RMS_EPS,
                              device=dev)
    for kc, vc in zip(st.k_cache, st.v_cache):
        kc.copy_(torch.randn(kc.shape, generator=gen, device=dev))
        vc.copy_(torch.randn(vc.shape, generator=gen, device=dev))
    st.set_positions(torch.full((M,), context - 1, dtype=torch.int32, device=dev))
    ids = torch.randint(0, vocab, (M,), generator=gen, device=dev, dtype=torch.int32)
    n_q, n_kv, hd = st.dims
    st.step(ids)
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0 and bool(torch.isfinite(st.logits).all())
    eager_ms = cuda_time_ms(lambda: [st.step(ids) for _ in range(reps)]) / reps
    graph_ms = graph_time_ms(lambda: st.step(ids), reps)

    def attention_all():
        for kc, vc in zip(st.k_cache, st.v_cache):
            bl.bitlinear_attention_decode_append(st.q, st.k, st.v, st.rope_table, kc, vc, st.lengths, n_q, n_kv, hd,
                                                 seq_ids=st.seq_ids, out=st.attn, ws=st.attn_ws)

    attn_ms = graph_time_ms(attention_all, reps)  # rotary embedding and cache append included
    # the table (657 MB) is larger than L2: back-to-back calls each stream it from HBM
    head_ms = cuda_time_ms(lambda: [bl.bitlinear_lm_head(st.h_mid, table, out=st.logits) for _ in range(reps)]) / reps
    cache_bytes = 2 * wl.N_LAYERS * M * context * n_kv * hd * 2
    table_bytes = table.numel() * 2
    us = lambda ms: None if ms is None else round(ms * 1e3, 1)  # noqa: E731
    gbs = lambda b, ms: None if ms is None else round(b / ms / 1e6, 1)  # noqa: E731
    total = graph_ms if graph_ms is not None else eager_ms
    return {"workload": f"one decoded token, M={M}, {context - 1} tokens in a bf16 KV cache, 30 layers, bf16 output head of {vocab} rows",
            "launches_per_token": wl.N_LAYERS * st.launches_per_layer + 3,
            "eager_us_per_token": us(eager_ms), "graph_us_per_token": us(graph_ms),
            "bytes_per_token": {"packed_weights": packed_bytes, "kv_cache": cache_bytes, "output_head": table_bytes},
            "frac_of_hbm_peak": round((packed_bytes + cache_bytes + table_bytes) / total / 1e6 / peaks["hbm_gbs"], 4),
            "rope_append_attention_30_layers": {"us": us(attn_ms), "GBps": gbs(cache_bytes, attn_ms),
                                    "frac_of_hbm_peak": None if attn_ms is None else round(cache_bytes / attn_ms / 1e6 / peaks["hbm_gbs"], 4)},
            "output_head": {"us": us(head_ms), "GBps": gbs(table_bytes, head_ms),
                            "frac_of_hbm_peak": round(table_bytes / head_ms / 1e6 / peaks["hbm_gbs"], 4)}}


def timed_sequence(calls, blocker):
    """Device time of each call of a back-to-back sequence.  `blocker` enqueues enough GPU work for the host to
    run ahead, so that no call waits for its launch; an event is recorded between consecutive calls."""
    torch.cuda.synchronize()
    blocker()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
    for ev, call in zip(evs, calls):
        ev.record()
        call()
    evs[-1].record()
    torch.cuda.synchronize()
    return [evs[i].elapsed_time(evs[i + 1]) for i in range(len(calls))]


def run_config1(bl, dev, peaks):
    """configs[0]: a single q-projection forward (N = K = 2560) at one token."""
    name, n, k = wl.LAYER_SHAPES[0]
    copies = 256  # 256 x 1.6 MB = 419 MB of distinct packed weights: every call finds its weights in HBM, not in L2
    W = wl.latent_weights(n, k, wl.seed_for(1, 0)).to(dev)
    packed0, s_w = bl.bitlinear_pack_weights(W, wl.WEIGHT_EPS)
    del W
    packs = [packed0] + [packed0.clone() for _ in range(copies - 1)]
    x = wl.activations_normal(1, k, wl.seed_for(1, 0, 1)).to(dev)
    gain = wl.gain_ones(k).to(dev)
    ys = [torch.empty(1, n, dtype=torch.float32, device=dev) for _ in range(copies)]
    ws = torch.empty(bl.bitlinear_workspace_bytes(1, n, k), dtype=torch.uint8, device=dev)
    lib, st = bl.lib(), torch.cuda.current_stream().cuda_stream

    def single(j):
        rc = lib.bitlinear_forward(x.data_ptr(), gain.data_ptr(), wl.RMS_EPS, packs[j].data_ptr(), s_w.data_ptr(), 1, n, k,
                                   ys[j].data_ptr(), 0, ws.data_ptr(), ws.numel(), st)
        assert rc == 0, rc

    # isolated: each call alone on an idle GPU (synchronised before and after), cold weights
    iso = []
    for j in range(8, 40):
        iso.append(cuda_time_ms(lambda j=j: single(j)) * 1e3)
    iso_us = statistics.median(iso)
    # back to back single calls (two launches each)
    seq_us = avg_call_us([lambda j=j: single(j) for j in range(copies)])
    # steady state: all 256 forwards in one batched call (two launches in all)
    batch = bl.ProblemBatch([(x, gain, packs[j], s_w, ys[j]) for j in range(copies)], wl.RMS_EPS)
    wsb = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
    bl.bitlinear_forward_batch(batch, wsb)
    n_rep = 10
    ms_b = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, wsb, reuse_plan=True) for _ in range(n_rep)]) / n_rep
    pb = n * k // 4
    return {"workload": "configs[0]: q projection, M=1, K=N=2560, 1,638,400 packed bytes per forward",
            "isolated_us_per_forward": round(iso_us, 2), "isolated_GBps": round(pb / iso_us / 1e3, 1),
            "isolated_note": "one bitlinear_forward (a single launch that quantises the row and streams the weights) on an idle GPU, weights not in L2: "
                             "latency-bound, a 1.6 MB matmul is far below the bandwidth-delay product of HBM",
            "back_to_back_us_per_forward": round(seq_us, 2), "back_to_back_GBps": round(pb / seq_us / 1e3, 1),
            "steady_us_per_forward": round(ms_b * 1e3 / copies, 3), "steady_GBps": round(pb * copies / ms_b / 1e6, 1),
            "steady_frac_of_hbm_peak": round(pb * copies / ms_b / 1e6 / peaks["hbm_gbs"], 4),
            "steady_note": f"{copies} forwards on {copies} distinct copies of the packed matrix in one bitlinear_forward_batch call"}


def run_dense(bl, dev, peaks, items2, ms_two_bit, reps):
    """The headline step with every matrix stored five ternary values per byte (Table 1's 1.58-bit budget)."""
    items, nbytes = [], 0
    for layer in range(wl.N_LAYERS):
        for (name, n, k), it in zip(wl.LAYER_SHAPES, items2[layer * 7:(layer + 1) * 7]):
            W = wl.latent_weights(n, k, wl.layer_seed(CONFIG_ID, layer, name)).to(dev)
            packed5, s_w = bl.bitlinear_pack_weights5(W, wl.WEIGHT_EPS)
            del W
            nbytes += packed5.numel()
            items.append((it[0], it[1], packed5, s_w, torch.empty_like(it[4])))
    batch = bl.ProblemBatch(items, wl.RMS_EPS, w_format=bl.WEIGHTS_DENSE5)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
    bl.bitlinear_forward_batch(batch, ws)
    same = all(torch.equal(a[4], b[4]) for a, b in zip(items, items2))  # outputs of the 2-bit step, computed before
    for _ in range(3):
        bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
    ms = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_plan=True) for _ in range(reps)]) / reps
    ms_k = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True) for _ in range(reps)]) / reps
    out = {"layout": "five ternary values per byte (1.6 bit per weight), K padded to multiples of 320",
           "packed_bytes_per_step": nbytes, "bytes_vs_two_bit": round(nbytes / 521_011_200, 4),
           "us_per_step": round(ms * 1e3, 2), "kernel_alone_us": round(ms_k * 1e3, 2),
           "value_actual_bytes": round(nbytes / ms / 1e6, 1), "unit": UNIT,
           "kernel_frac_of_hbm_peak_actual_bytes": round(nbytes / ms_k / 1e6 / peaks["hbm_gbs"], 4),
           "two_bit_us_per_step": round(ms_two_bit * 1e3, 2), "outputs_equal_two_bit_step": bool(same),
           "note": "same kernel structure as the headline step; the base-3 digits are peeled off in registers (multiply by 3, "
                   "mask, byte permute per digit), which makes this kernel bound by instruction issue, not by HBM: it "
                   "saves 20 % of the memory, not time"}
    del items, batch, ws
    return out


def run_sweep(bl, dev, peaks, int8_peak):
    """configs[4]: FFN down projection (N = 2560, K = 6912), M in {1, 8, 32, 64, 256, 1024, 4096}, Student-t inputs.

    Every path that accepts the shape is forced.  Two regimes: a SINGLE matmul per call (4.4 MB of weights: far below
    the bandwidth-delay product, so the time is launch latency) and the STEADY state, 32 such matmuls on 32 distinct
    copies of the packed matrix in one batched call (141 MB > L2), reported per matmul."""
    n, k = wl.SHAPE_NK["down"]
    copies = 32
    W = wl.latent_weights(n, k, wl.seed_for(5, 0) + 1).to(dev)
    packed0, s_w = bl.bitlinear_pack_weights(W, wl.WEIGHT_EPS)
    del W
    packs = [packed0] + [packed0.clone() for _ in range(copies - 1)]
    gain = wl.gain_ones(k).to(dev)
    lib, st = bl.lib(), torch.cuda.current_stream().cuda_stream
    pb = n * k // 4
    rows = {}

    def batch_us(items, reps):
        b = bl.ProblemBatch(items, wl.RMS_EPS)
        w = torch.empty(b.workspace_bytes(), dtype=torch.uint8, device=dev)
        bl.bitlinear_forward_batch(b, w)
        bl.bitlinear_forward_batch(b, w, reuse_plan=True, reuse_act=True)
        return cuda_time_ms(lambda: [bl.bitlinear_forward_batch(b, w, reuse_plan=True, reuse_act=True) for _ in range(reps)]) * 1e3 / reps

    for M in (1, 8, 32, 64, 256, 1024, 4096):
        x = wl.activations_student_t(M, k, wl.seed_for(5, 0, M % 10)).to(dev)
        xq, d, xsum = bl.bitlinear_quant_act(x, gain, wl.RMS_EPS)
        y = torch.empty(M, n, dtype=torch.float32, device=dev)
        ws_mm = torch.empty(max(16, bl.bitlinear_matmul_workspace_bytes(M, n, k, bl.PATH_GEMM)), dtype=torch.uint8, device=dev)
        single, steady = {}, {}

        def mm(j, path):
            rc = lib.bitlinear_matmul_q(xq.data_ptr(), d.data_ptr(), xsum.data_ptr(), packs[j % copies].data_ptr(), s_w.data_ptr(),
                                        M, n, k, y.data_ptr(), 0, None, path, ws_mm.data_ptr(), ws_mm.numel(), st)
            assert rc == 0, rc

        reps = copies if M <= 256 else 8
        if M <= 256:  # the streaming kernel of the single-call API takes any M in chunks of 16 tokens
            single["streaming_dp4a"] = avg_call_us([lambda j=j: mm(j, bl.PATH_GEMV) for j in range(reps)])
        single["tcgen05_gemm"] = avg_call_us([lambda j=j: mm(j, bl.PATH_GEMM) for j in range(reps)])
        # steady state, contraction only (quantised activations reused): outputs of the 32 problems share one buffer
        n_rep = 5 if M <= 256 else 2
        if M <= 64:
            # decode kernels: one problem per copy and per chunk of at most 16 tokens (M = 1: dot-products-of-four;
            # 2..8 tokens: the same stream feeding mma.sync; 9..16: tcgen05 decode kernel); for M > 16 this is the decode path forced
            chunks = [(c0, min(16, M - c0)) for c0 in range(0, M, 16)]
            items = [(x[c0:c0 + m], gain, packs[j], s_w, y[c0:c0 + m]) for j in range(copies) for c0, m in chunks]
            steady["streaming_dp4a" if M == 1 else "streaming_mma_sync" if M <= 8 else "tensor_core_decode_16_token_chunks"] = batch_us(items, n_rep) / copies
        if M > 16:
            items = [(x, gain, packs[j], s_w, y) for j in range(copies)]
            steady["grouped_tcgen05_gemm"] = batch_us(items, n_rep) / copies
        best = min(steady, key=steady.get)
        us = steady[best]
        rows[f"M={M}"] = {"single_call_us": {kk: round(v, 2) for kk, v in single.items()},
                          "steady_us_per_matmul": {kk: round(v, 3) for kk, v in steady.items()}, "steady_best": best,
                          "GBps_packed": round(pb / us / 1e3, 1), "frac_of_hbm_peak": round(pb / us / 1e3 / peaks["hbm_gbs"], 4),
                          "tops": round(2.0 * M * n * k / us / 1e6, 1),
                          "frac_of_int8_peak": round(2.0 * M * n * k / us / 1e6 / int8_peak, 4)}
        del x, xq, y, ws_mm
    cross = [M for M in (32, 64) if rows[f"M={M}"]["steady_best"] == "grouped_tcgen05_gemm"]
    return {"workload": "configs[4]: FFN down projection K=6912, N=2560, Student-t(3) activations, 4,423,680 packed bytes",
            "per_M": rows,
            "crossover_M": cross[0] if cross else ">64",
            "crossover_note": "smallest M of the sweep at which the grouped tcgen05 GEMM (weights expanded to byte codes, 256 x 256 "
                              "tiles) beats streaming the packed weights once per 16 tokens through the decode kernels, steady state",
            "dispatch_threshold": 16,
            "dispatch_note": "M <= 16 goes to the streaming decode kernels (M = 1 dot-products-of-four, 2..16 tokens tensor-core "
                             "decode), M > 16 to the tcgen05 GEMM; a caller with 17..64 tokens may split them into 16-token "
                             "problems of one batched call where the table above says that is faster",
            "int8_peak_tops": round(int8_peak, 1)}


def run_prefill(bl, dev, pool, gains, peaks, int8_peak, reps):
    """Forward at M = 2048 on the 7 shapes: per-shape contraction TOPS and the layer aggregate.

    Every call of a timed sequence uses another layer's packed weights and another activation / output buffer, so
    that the sequence touches far more than the 126 MB L2 (outputs alone are 21-57 MB per call)."""
    M = PREFILL_M
    # Denominator: the measured rate of the int8 tensor-core instruction itself (bitlinear_probe_int8_mma_rate, operands in
    # shared memory, no global traffic).  Beside it: 2 x the measured bf16 GEMM burst (nominal ratio 4.5 / 2.25) and the
    # datasheet's dense int8 figure.
    proxy_peak = 2.0 * peaks["bf16_tflops"]
    int8_peak = int8_peak or proxy_peak
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    n_sets = 6
    per_shape, t_gemm_total, t_fwd_total, ops_total = {}, 0.0, 0.0, 0.0
    for i, (name, n, k) in enumerate(wl.LAYER_SHAPES):
        mats = [pool[layer * 7 + i] for layer in range(n_sets)]
        xs = [wl.activations_outlier(M, k, wl.seed_for(4, i, j)).to(dev) for j in range(n_sets)]
        ys = [torch.empty(M, n, dtype=torch.float32, device=dev) for _ in range(n_sets)]
        ws = torch.empty(bl.bitlinear_workspace_bytes(M, n, k), dtype=torch.uint8, device=dev)
        ws_mm = torch.empty(bl.bitlinear_matmul_workspace_bytes(M, n, k), dtype=torch.uint8, device=dev)
        quant = [bl.bitlinear_quant_act(x, gains[k], wl.RMS_EPS) for x in xs]
        lib, st = bl.lib(), torch.cuda.current_stream().cuda_stream

        def mm(j):
            xq, d, xsum = quant[j]
            rc = lib.bitlinear_matmul_q(xq.data_ptr(), d.data_ptr(), xsum.data_ptr(), mats[j]["packed"].data_ptr(),
                                        mats[j]["s_w"].data_ptr(), M, n, k, ys[j].data_ptr(), 0, None, 0,
                                        ws_mm.data_ptr(), ws_mm.numel(), st)
            assert rc == 0, rc

        def fwd(j):
            rc = lib.bitlinear_forward(xs[j].data_ptr(), gains[k].data_ptr(), wl.RMS_EPS, mats[j]["packed"].data_ptr(),
                                       mats[j]["s_w"].data_ptr(), M, n, k, ys[j].data_ptr(), 0, ws.data_ptr(),
                                       ws.numel(), st)
            assert rc == 0, rc

        n_calls = n_sets * max(2, reps // 2)
        t_mm = timed_sequence([lambda j=j: mm(j % n_sets) for j in range(n_calls)], flush.zero_)[n_sets:]
        t_fw = timed_sequence([lambda j=j: fwd(j % n_sets) for j in range(n_calls)], flush.zero_)[n_sets:]
        ops = 2.0 * M * n * k
        mm_s, fw_s = statistics.median(t_mm) / 1e3, statistics.median(t_fw) / 1e3
        per_shape[name] = {"N": n, "K": k, "matmul_us": round(mm_s * 1e6, 2), "matmul_tops": round(ops / mm_s / 1e12, 1),
                           "forward_us": round(fw_s * 1e6, 2), "forward_tops": round(ops / fw_s / 1e12, 1)}
        t_gemm_total += mm_s
        t_fwd_total += fw_s
        ops_total += ops
        del xs, ys, quant
    # ---- the 7 matmuls of a layer as ONE grouped call (3 launches: unpack, quantise beside it, every tile of every matmul) ----
    group_sets = []
    shared_input = {"k": "q", "v": "q", "up": "gate"}  # as in the layer: q/k/v read one tensor, gate/up another
    for j in range(3):
        items, xs_by_name = [], {}
        for i, (name, n, k) in enumerate(wl.LAYER_SHAPES):
            src = shared_input.get(name)
            x = xs_by_name[src] if src else wl.activations_outlier(M, k, wl.seed_for(4, i, j)).to(dev)
            xs_by_name[name] = x
            mat = pool[j * 7 + i]
            items.append((x, gains[k], mat["packed"], mat["s_w"], torch.empty(M, n, dtype=torch.float32, device=dev)))
        group_sets.append(bl.ProblemBatch(items, wl.RMS_EPS))
    ws_g = torch.empty(group_sets[0].workspace_bytes(), dtype=torch.uint8, device=dev)
    n_calls = 3 * max(2, reps // 2)
    t_g = timed_sequence([lambda j=j: bl.bitlinear_forward_batch(group_sets[j % 3], ws_g) for j in range(n_calls)],
                         flush.zero_)[3:]
    g_s = statistics.median(t_g) / 1e3
    t_gm = timed_sequence([lambda j=j: bl.bitlinear_forward_batch(group_sets[j % 3], ws_g, reuse_act=True)
                           for j in range(n_calls)], flush.zero_)[3:]
    gm_s = statistics.median(t_gm) / 1e3  # activations of the last full call stay quantised: unpack + GEMM only
    grouped = {"api": "bitlinear_forward_batch on the 7 shapes of a layer at M=2048, q/k/v and gate/up sharing their input "
                      "(3 launches: unpack, quantiser beside it, every tile of every matmul following the unpack tile by tile)",
               "forward_us_per_layer": round(g_s * 1e6, 2), "forward_tops": round(ops_total / g_s / 1e12, 1),
               "forward_frac": round(ops_total / g_s / 1e12 / int8_peak, 4),
               "matmul_us_per_layer": round(gm_s * 1e6, 2), "matmul_tops": round(ops_total / gm_s / 1e12, 1),
               "matmul_frac": round(ops_total / gm_s / 1e12 / int8_peak, 4)}
    del group_sets, ws_g
    tops = ops_total / t_gemm_total / 1e12
    return {"metric": "bitlinear_prefill_int8_tops_m2048", "M": M, "value": grouped["matmul_tops"], "unit": "TOP/s",
            "frac": grouped["matmul_frac"], "forward_value": grouped["forward_tops"],
            "what": "value = 2MNK of the 7 matmuls of a layer / device time of ONE grouped call that unpacks the packed "
                    "weights and runs every tile of every matmul (activations already quantised); forward_value also "
                    "counts the fused RMSNorm+quantiser launch; fp32 outputs",
            "peak": round(int8_peak, 1), "peak_source": "measured: tcgen05.mma kind::i8 on shared-memory-resident operands, all SMs",
            "other_peaks": {"two_x_bf16_gemm_burst": round(proxy_peak, 1), "datasheet_dense_int8": 4500.0},
            "frac_of_two_x_bf16_burst": round(grouped["matmul_tops"] / proxy_peak, 4),
            "frac_of_datasheet": round(grouped["matmul_tops"] / 4500.0, 4),
            "forward_frac": grouped["forward_frac"], "grouped": grouped,
            "single_calls": {"value": round(tops, 1), "frac": round(tops / int8_peak, 4),
                             "forward_value": round(ops_total / t_fwd_total / 1e12, 1),
                             "note": "one bitlinear_matmul_q / bitlinear_forward call per shape (unpack pass + tcgen05 "
                                     "GEMM; forward adds the quantiser); median device time per call between CUDA events",
                             "per_shape": per_shape},
            "l2": "back-to-back calls rotate over several layers' weights and activation/output buffers "
                  "(footprint > 2 x L2)"}


# --------------------------------------------------------------------------------------------- oracle


def oracle_decode_baseline(budget_s: float):
    """Times the CPU oracle, as it stands, on a bounded sample of the decode workload."""
    import oracle

    M = 1
    n_layers = 2
    mats = []
    for layer in range(n_layers):
        for name, n, k in wl.LAYER_SHAPES:
            W = wl.latent_weights(n, k, wl.layer_seed(CONFIG_ID, layer, name)).numpy()
            s_w, _ = oracle.weight_scale(W, wl.WEIGHT_EPS)
            mats.append((name, n, k, oracle.weight_quant(W, s_w), s_w))
    xs = {name: wl.bf16_bits(wl.activations_normal(M, k, wl.seed_for(CONFIG_ID, i)))
          for i, (name, n, k) in enumerate(wl.LAYER_SHAPES)}
    gains = {k: wl.bf16_bits(wl.gain_ones(k)) for k in (wl.HIDDEN, wl.FFN)}

    def one_pass():
        for name, n, k, wq, s_w in mats:
            oracle.bitlinear_forward(xs[name], gains[k], wl.RMS_EPS, wq, s_w)

    one_pass()
    t0 = time.perf_counter()
    passes = 0
    while True:
        one_pass()
        passes += 1
        el = time.perf_counter() - t0
        if el > budget_s or passes >= 5000:
            break
    packed = sum(n * k // 4 for _, n, k, _, _ in mats)
    return {"value": round(packed * passes / el / 1e9, 3), "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(el, 2),
            "sample": f"{n_layers} of 30 layers x 7 shapes at M=1 ({len(mats)} forwards, {packed} packed-equivalent "
                      f"bytes per pass), {passes} passes; weights pre-quantised by the oracle outside the timed region"}


def run_reference(args):
    """The reference arm of this build is the CPU oracle on the host cores (no released GPU code exists)."""
    rank, _, world = replicas.world()
    if rank != 0:
        return
    per_step_budget = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    for _ in range(min(args.warmup, 1)):
        oracle_decode_baseline(budget_s=1.0)
    res, t_all = [], time.perf_counter()
    for _ in range(args.steps):
        res.append(oracle_decode_baseline(budget_s=per_step_budget))
    v = statistics.median(r["value"] for r in res)
    last = res[-1]
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": round((time.perf_counter() - t_all) * 1e3 / args.steps, 2),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "s8 x ternary -> s32 (fp32 epilogue)",
           "data": "synthetic", "config": {"workload": WORKLOAD, "M": 1, "note": "each step is a bounded sample"},
           "cpu_baseline": {"value": v, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def run_case_batch(args, bl, dev):
    """The batched decode call on --layers layers of the 7 shapes at --m tokens (a smaller copy of the headline step)."""
    M = args.m
    pool = build_decode_pool(bl, dev, args.layers)
    packed_bytes = sum(p["packed"].numel() for p in pool)
    gains = {k: wl.gain_ones(k).to(dev) for k in (wl.HIDDEN, wl.FFN)}
    items = []
    for i, p in enumerate(pool):
        x = wl.activations_normal(M, p["K"], wl.seed_for(CONFIG_ID, i % 7, M)).to(dev)
        items.append((x, gains[p["K"]], p["packed"], p["s_w"], torch.empty(M, p["N"], dtype=torch.float32, device=dev)))
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
    bl.bitlinear_forward_batch(batch, ws)
    for _ in range(args.warmup):
        bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
    ms = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_plan=True) for _ in range(args.steps)]) / args.steps
    ms_s = statistics.median(cuda_time_ms(lambda: bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True))
                             for _ in range(max(3, args.steps)))
    print(json.dumps({"case": "batch", "M": M, "layers": args.layers, "forwards": len(pool), "packed_bytes": packed_bytes,
                      "us_per_step": round(ms * 1e3, 2), "packed_GBps": round(packed_bytes / ms / 1e6, 1),
                      "stream_kernel_us": round(ms_s * 1e3, 2), "stream_kernel_GBps": round(packed_bytes / ms_s / 1e6, 1),
                      "hbm_peak": load_peaks()["hbm_gbs"]}))


def run_case_chain(args, bl, dev):
    """The dependent chain of --layers layers at one token through the persistent kernel (a smaller copy of configs[2])."""
    from paper_2504_12285_b200 import chain as gpu_chain

    pool = build_decode_pool(bl, dev, args.layers)
    packed_bytes = sum(p["packed"].numel() for p in pool)
    gains = {k: wl.gain_ones(k).to(dev) for k in (wl.HIDDEN, wl.FFN)}
    pl = [dict({m["name"]: (m["packed"], m["s_w"]) for m in pool[layer * 7:(layer + 1) * 7]},
               gains=[gains[wl.HIDDEN], gains[wl.HIDDEN], gains[wl.HIDDEN], gains[wl.FFN]]) for layer in range(args.layers)]
    pc = gpu_chain.PersistentChain(pl, wl.HIDDEN, wl.FFN, wl.N_Q_HEADS, wl.N_KV_HEADS, wl.HEAD_DIM, wl.RMS_EPS, dev)
    h0 = wl.activations_normal(1, wl.HIDDEN, wl.seed_for(3)).to(dev)
    for _ in range(args.warmup):
        pc.step(h0)
    ms = cuda_time_ms(lambda: [pc.step(h0) for _ in range(args.steps)]) / args.steps
    assert bl.bitlinear_poll_status() == 0
    print(json.dumps({"case": "chain", "layers": args.layers, "packed_bytes": packed_bytes, "us_per_token": round(ms * 1e3, 1),
                      "us_per_level": round(ms * 1e3 / (4 * args.layers), 3), "packed_GBps": round(packed_bytes / ms / 1e6, 1)}))


def run_case_step(args, bl, dev):
    """A whole decoded token at --m sequences with --context cache rows (see run_decode_step)."""
    pool = build_decode_pool(bl, dev, wl.N_LAYERS)
    gains = {k: wl.gain_ones(k).to(dev) for k in (wl.HIDDEN, wl.FFN)}
    out = run_decode_step(bl, dev, pool, gains, load_peaks(), sum(p["packed"].numel() for p in pool), max(3, args.steps),
                          M=args.m, context=args.context)
    print(json.dumps(dict(out, case="step")))


def run_case_group(args, bl, dev):
    """The 7 shapes of a layer at --m tokens as one grouped call (quantiser + unpack + grouped GEMM)."""
    M = args.m
    pool = build_decode_pool(bl, dev, 1)
    gains = {k: wl.gain_ones(k).to(dev) for k in (wl.HIDDEN, wl.FFN)}
    ydt = torch.bfloat16 if args.ydtype == "bf16" else torch.float32
    items = []
    for i, p in enumerate(pool):
        x = wl.activations_outlier(M, p["K"], wl.seed_for(4, i)).to(dev)
        items.append((x, gains[p["K"]], p["packed"], p["s_w"], torch.empty(M, p["N"], dtype=ydt, device=dev)))
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=dev)
    for _ in range(args.warmup):
        bl.bitlinear_forward_batch(batch, ws)
    ms = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws) for _ in range(args.steps)]) / args.steps
    ms_mm = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_act=True) for _ in range(args.steps)]) / args.steps
    ms_g = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_act=True, reuse_weights=True) for _ in range(args.steps)]) / args.steps
    ms_qg = cuda_time_ms(lambda: [bl.bitlinear_forward_batch(batch, ws, reuse_weights=True) for _ in range(args.steps)]) / args.steps
    ops = sum(2.0 * M * p["N"] * p["K"] for p in pool)
    print(json.dumps({"case": "group", "M": M, "us_forward": round(ms * 1e3, 2), "forward_tops": round(ops / ms / 1e9, 1),
                      "us_unpack_gemm": round(ms_mm * 1e3, 2), "unpack_gemm_tops": round(ops / ms_mm / 1e9, 1),
                      "us_gemm_only": round(ms_g * 1e3, 2), "gemm_only_tops": round(ops / ms_g / 1e9, 1),
                      "us_quant_gemm": round(ms_qg * 1e3, 2)}))


def run_case(args):
    """One kernel on one shape (for profiling and sweeps): --case gemv|gemm|quant|pack --shape q --m 1,
    or --case batch --layers L --m M.

    Distinct copies of the packed weights (--copies) are cycled so that the footprint exceeds L2."""
    from paper_2504_12285_b200 import binding as bl

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    if args.case == "batch":
        return run_case_batch(args, bl, dev)
    if args.case == "group":
        return run_case_group(args, bl, dev)
    if args.case == "step":
        return run_case_step(args, bl, dev)
    if args.case == "chain":
        return run_case_chain(args, bl, dev)
    n, k = wl.SHAPE_NK[args.shape]
    M = args.m
    peaks = load_peaks()
    W = wl.latent_weights(n, k, wl.seed_for(CONFIG_ID, wl.SHAPE_INDEX[args.shape])).to(dev)
    packed0, s_w = bl.bitlinear_pack_weights(W, wl.WEIGHT_EPS)
    copies = [packed0] + [packed0.clone() for _ in range(args.copies - 1)]
    x = wl.activations_normal(M, k, wl.seed_for(CONFIG_ID, 0, 1)).to(dev)
    gain = wl.gain_ones(k).to(dev)
    xq, d, xsum = bl.bitlinear_quant_act(x, gain, wl.RMS_EPS)
    path = {"gemv": bl.PATH_GEMV, "gemm": bl.PATH_GEMM}.get(args.case, bl.PATH_AUTO)
    ws = torch.empty(max(16, bl.bitlinear_matmul_workspace_bytes(M, n, k, path)), dtype=torch.uint8, device=dev)
    ws_p = torch.empty(bl.bitlinear_pack_workspace_bytes(n, k), dtype=torch.uint8, device=dev)
    ydt = torch.bfloat16 if args.ydtype == "bf16" else torch.float32
    y = torch.empty(M, n, dtype=ydt, device=dev)
    lib, st = bl.lib(), torch.cuda.current_stream().cuda_stream

    def one(i):
        p = copies[i % len(copies)]
        if args.case in ("gemv", "gemm"):
            rc = lib.bitlinear_matmul_q(xq.data_ptr(), d.data_ptr(), xsum.data_ptr(), p.data_ptr(), s_w.data_ptr(), M, n, k,
                                        y.data_ptr(), 1 if args.ydtype == "bf16" else 0, None, path, ws.data_ptr(),
                                        ws.numel(), st)
        elif args.case == "quant":
            rc = lib.bitlinear_quant_act(x.data_ptr(), gain.data_ptr(), wl.RMS_EPS, M, k, xq.data_ptr(), d.data_ptr(),
                                         xsum.data_ptr(), st)
        else:
            rc = lib.bitlinear_pack_weights(W.data_ptr(), 0, n, k, wl.WEIGHT_EPS, p.data_ptr(), s_w.data_ptr(),
                                            ws_p.data_ptr(), ws_p.numel(), st)
        assert rc == 0, rc

    for i in range(args.warmup):
        one(i)
    calls = args.steps * len(copies)
    ms = cuda_time_ms(lambda: [one(i) for i in range(calls)])
    us = ms * 1e3 / calls
    out = {"case": args.case, "shape": args.shape, "M": M, "N": n, "K": k, "copies": len(copies), "calls": calls,
           "us_per_call": round(us, 3), "packed_GBps": round(n * k / 4 / us / 1e3, 1),
           "tops": round(2.0 * M * n * k / us / 1e6, 1), "hbm_peak": peaks["hbm_gbs"]}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", choices=["gemv", "gemm", "quant", "pack", "batch", "group", "chain", "step"], default=None)
    ap.add_argument("--layers", type=int, default=10)
    ap.add_argument("--shape", choices=list(wl.SHAPE_NK), default="q")
    ap.add_argument("--m", type=int, default=1)
    ap.add_argument("--copies", type=int, default=1)
    ap.add_argument("--context", type=int, default=4096)
    ap.add_argument("--ydtype", choices=["f32", "bf16"], default="f32")
    args = ap.parse_args()
    if args.case:
        return run_case(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
