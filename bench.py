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
CONFIG_ID = 2  # BASELINE configs[1]: decode step over all 7 BitLinear shapes of one 2B-style layer
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
    xs = {}
    for i, (name, n, k) in enumerate(wl.LAYER_SHAPES):
        xs[name] = wl.activations_normal(M, k, wl.seed_for(CONFIG_ID, i)).to(dev)
    ys = {name: torch.empty(M, n, dtype=torch.float32, device=dev) for name, n, k in wl.LAYER_SHAPES}
    ws = torch.empty(max(bl.bitlinear_workspace_bytes(M, n, k) for _, n, k in wl.LAYER_SHAPES), dtype=torch.uint8,
                     device=dev)

    def step():
        for p in pool:
            bl.bitlinear_forward(xs[p["name"]], gains[p["K"]], p["packed"], p["s_w"], p["N"], wl.RMS_EPS, ws=ws,
                                 out=ys[p["name"]])

    launches_per_step = 2 * len(pool)  # one quantiser kernel + one contraction kernel per forward

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

    # ---- roofline of the dominant kernel: the decode contraction, timed launch by launch ----
    xq_d = {}
    for name, n, k in wl.LAYER_SHAPES:
        xq_d[name] = bl.bitlinear_quant_act(xs[name], gains[k], wl.RMS_EPS)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in pool]
    gemv_ms = []
    for rep in range(max(3, args.steps)):
        torch.cuda.synchronize()
        for (e0, e1), p in zip(ev, pool):
            xq, d, xsum = xq_d[p["name"]]
            e0.record()
            bl.bitlinear_matmul_q(xq, d, xsum, p["packed"], p["s_w"], p["N"], path=bl.PATH_GEMV)
            e1.record()
        torch.cuda.synchronize()
        if rep >= 1:
            gemv_ms.append(sum(e0.elapsed_time(e1) for e0, e1 in ev))
    gemv_launch_s = statistics.median(gemv_ms) / 1e3 / len(pool)
    bytes_per_launch = packed_bytes / len(pool)
    achieved = bytes_per_launch / gemv_launch_s / 1e9
    roofline = {"bound": "hbm", "kernel": "gemv_kernel (decode contraction, M=1)", "achieved": round(achieved, 1),
                "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4),
                "algorithmic_bytes_per_launch": bytes_per_launch, "avg_launch_us": round(gemv_launch_s * 1e6, 3),
                "traffic": None}

    # ---- end to end with host buffers through bitlinear_forward_host ----
    e2e = None
    if rank == 0 or world > 1:
        xh = {name: wl.activations_normal(M, k, wl.seed_for(CONFIG_ID, i)).pin_memory()
              for i, (name, n, k) in enumerate(wl.LAYER_SHAPES)}
        yh = {name: torch.empty(M, n, dtype=torch.float32).pin_memory() for name, n, k in wl.LAYER_SHAPES}
        ws_h = torch.empty(max(bl.bitlinear_workspace_bytes(M, n, k) + bl.bitlinear_host_staging_bytes(M, n, k)
                               for _, n, k in wl.LAYER_SHAPES), dtype=torch.uint8, device=dev)

        def step_host():
            for p in pool:
                bl.bitlinear_forward_host(xh[p["name"]], gains[p["K"]], p["packed"], p["s_w"], p["N"], yh[p["name"]],
                                          wl.RMS_EPS, ws=ws_h)

        for _ in range(2):
            step_host()
        replicas.barrier()
        n_e2e = max(1, min(args.steps, 5))
        ms_h = cuda_time_ms(lambda: [step_host() for _ in range(n_e2e)])
        replicas.barrier()
        v_h, _ = replicas.aggregate_throughput(packed_bytes * n_e2e / 1e9, ms_h / 1e3, device=str(dev))
        e2e = {"value": round(v_h, 2), "unit": UNIT,
               "h2d_bytes_per_step": sum(2 * M * p["K"] for p in pool),
               "d2h_bytes_per_step": sum(4 * M * p["N"] for p in pool),
               "api": "bitlinear_forward_host, one call per BitLinear (copy in, forward, copy out, sync)"}

    # ---- prefill: int8 tensor-core path at M = 2048 on the 7 shapes (rank 0 only) ----
    prefill = None
    if rank == 0:
        prefill = run_prefill(bl, dev, pool[:7], gains, peaks, reps=max(3, min(args.steps, 10)))

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
            "roofline": roofline, "prefill": prefill, "cpu_baseline": cpu,
        }
        print(json.dumps(out))
    replicas.finalize()


def run_prefill(bl, dev, layer, gains, peaks, reps):
    """Forward at M = 2048 on the 7 shapes: per-shape contraction TOPS and the layer aggregate."""
    M = PREFILL_M
    int8_peak = 2.0 * peaks["bf16_tflops"]  # int8 dense peak = 2 x the measured bf16 peak (nominal ratio 4.5/2.25)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    per_shape, t_gemm_total, t_fwd_total, ops_total = {}, 0.0, 0.0, 0.0
    for i, p in enumerate(layer):
        n, k = p["N"], p["K"]
        x = wl.activations_outlier(M, k, wl.seed_for(4, i)).to(dev)
        y = torch.empty(M, n, dtype=torch.float32, device=dev)
        ws = torch.empty(bl.bitlinear_workspace_bytes(M, n, k), dtype=torch.uint8, device=dev)
        ws_mm = torch.empty(bl.bitlinear_matmul_workspace_bytes(M, n, k), dtype=torch.uint8, device=dev)
        xq, d, xsum = bl.bitlinear_quant_act(x, gains[k], wl.RMS_EPS)
        t_mm, t_fwd = [], []
        for rep in range(reps + 2):
            flush.zero_()
            a = cuda_time_ms(lambda: bl.bitlinear_matmul_q(xq, d, xsum, p["packed"], p["s_w"], n, ws=ws_mm))
            flush.zero_()
            b = cuda_time_ms(lambda: bl.bitlinear_forward(x, gains[k], p["packed"], p["s_w"], n, wl.RMS_EPS, ws=ws, out=y))
            if rep >= 2:
                t_mm.append(a)
                t_fwd.append(b)
        ops = 2.0 * M * n * k
        mm, fw = statistics.median(t_mm) / 1e3, statistics.median(t_fwd) / 1e3
        per_shape[p["name"]] = {"N": n, "K": k, "matmul_us": round(mm * 1e6, 2), "matmul_tops": round(ops / mm / 1e12, 1),
                                "forward_us": round(fw * 1e6, 2), "forward_tops": round(ops / fw / 1e12, 1)}
        t_gemm_total += mm
        t_fwd_total += fw
        ops_total += ops
    tops = ops_total / t_gemm_total / 1e12
    return {"metric": "bitlinear_prefill_int8_tops_m2048", "M": M, "value": round(tops, 1), "unit": "TOP/s",
            "forward_value": round(ops_total / t_fwd_total / 1e12, 1),
            "peak": round(int8_peak, 1), "peak_source": f"2 x {peaks['source']} bf16 burst",
            "frac": round(tops / int8_peak, 4), "l2": "256 MB flush between timed calls",
            "note": "matmul = unpack-to-codes pass + tcgen05 GEMM with fused epilogue; forward adds the fused "
                    "RMSNorm+quant kernel", "per_shape": per_shape}


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
        if el > budget_s or passes >= 200:
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
