"""Parity of the GROUPED prefill call (bitlinear_forward_batch on problems of more than 16 tokens) with the CPU
oracle, in the launch configuration the benchmark times: the seven matmuls of a layer at M = 2048 in one call, q/k/v
and gate/up reading one shared input, and the same call again with the quantised activations reused.

The grouped call runs the CTA-pair tensor-core kernel (256 x 256 tiles, two CTAs per tile) beside the weight
expansion launch.  The cases below make every pair run several tiles, so that the second accumulator buffer, the
stage ring carried from tile to tile, the per-tile ready counters of the expansion and the walk across problems of
different K are all checked against the oracle - element by element where the oracle finishes in seconds, on sampled
outputs (tile edges included) and bitwise against the single-call kernel at full size.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def stable_rows(fragile, n_rows):
    """Rows the oracle does not flag (flagged: the RMSNorm scale sits on an fp32 rounding boundary of the sum of
    squares, about three rows in 1e5)."""
    ok = np.asarray(fragile) == 0
    flagged = int(n_rows - ok.sum())
    print(f"rows flagged as fragile: {flagged} of {n_rows}")
    assert flagged <= n_rows // 1000  # none at all in cases of fewer than 1000 rows
    return ok


class Layer:
    """Problems (name, M, N, K, input key): problems with the same input key share ONE x tensor and ONE gain tensor."""

    def __init__(self, spec, seed, x_kind="outlier", gains=True, y_dtype=torch.float32):
        gen = {"normal": wl.activations_normal, "outlier": wl.activations_outlier, "student_t": wl.activations_student_t}[x_kind]
        self.spec, self.x, self.g, self.w, items = spec, {}, {}, [], []
        for i, (name, M, N, K, key) in enumerate(spec):
            if key not in self.x:
                self.x[key] = gen(M, K, seed + 10 * i)
                self.g[key] = wl.gain_random(K, seed + 10 * i + 1) if gains else None
            W = wl.latent_weights(N, K, seed + 10 * i + 2)
            packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
            wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
            assert np.array_equal(packed.cpu().numpy(), wref["packed"])
            self.w.append((packed, s_w, wref))
        self.x_dev = {k: v.to(DEV) for k, v in self.x.items()}
        self.g_dev = {k: None if v is None else v.to(DEV) for k, v in self.g.items()}
        for (name, M, N, K, key), (packed, s_w, _) in zip(spec, self.w):
            items.append((self.x_dev[key], self.g_dev[key], packed, s_w,
                          torch.full((M, N), float("nan"), dtype=y_dtype, device=DEV)))
        self.batch = bl.ProblemBatch(items, wl.RMS_EPS)
        self.ws = torch.empty(self.batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
        self.q = {}

    def quant_ref(self, key):
        if key not in self.q:
            g = self.g[key]
            self.q[key] = oracle.rmsnorm_quant(wl.bf16_bits(self.x[key]), None if g is None else wl.bf16_bits(g), wl.RMS_EPS)
        return self.q[key]

    def run(self, **kw):
        bl.bitlinear_forward_batch(self.batch, self.ws, **kw)
        torch.cuda.synchronize()
        assert bl.bitlinear_poll_status() == 0

    def outputs(self):
        return [t[4] for t in self.batch.tensors]

    def poison(self):
        for y in self.outputs():
            y.fill_(float("nan"))


def check_sampled(layer, n_samples, seed):
    """Sampled outputs of every problem (tile edges at rows / columns 127, 128, 255, 256 and the corners included)
    against accumulators the oracle computes one by one."""
    rng = np.random.default_rng(seed)
    for (name, M, N, K, key), (_, _, wref), y in zip(layer.spec, layer.w, layer.outputs()):
        qref = layer.quant_ref(key)
        ok = stable_rows(qref["fragile"], M)
        y_host = y.float().cpu().numpy()
        assert not np.isnan(y_host).any(), name
        m_idx = rng.choice(np.nonzero(ok)[0], n_samples).astype(np.int32)
        n_idx = rng.integers(0, N, n_samples).astype(np.int32)
        edges_m = [m for m in (0, 127, 128, 255, 256, 257, M - 129, M - 128, M - 1) if 0 <= m < M and ok[m]]
        edges_n = [n for n in (0, 127, 128, 255, 256, 257, N - 257, N - 256, N - 1) if 0 <= n < N]
        em, en = np.meshgrid(np.array(edges_m, np.int32), np.array(edges_n, np.int32), indexing="ij")
        m_idx = np.concatenate([m_idx, em.reshape(-1)])
        n_idx = np.concatenate([n_idx, en.reshape(-1)])
        acc = oracle.matmul_i32_sampled(qref["q"], wref["wq"], m_idx, n_idx)
        want = (oracle.dequant(acc.reshape(1, -1), wref["s_w"], np.ones(1, np.float32))[0] * qref["d"][m_idx]).astype(np.float32)
        got = y_host[m_idx, n_idx]
        if y.dtype == torch.float32:
            w64, g64 = want.astype(np.float64), got.astype(np.float64)
            assert np.all(np.abs(g64 - w64) <= 1e-6 * np.abs(w64)), name
            assert np.all(g64[acc == 0] == 0.0), name
        else:
            want_bits = oracle.f32_to_bf16(want).astype(np.int32)
            got_bits = wl.bf16_bits(y.cpu())[m_idx, n_idx].astype(np.int32)
            assert np.all(np.abs(got_bits - want_bits) <= 1), name


def check_full(layer):
    """Every output element of every problem against the oracle's forward."""
    for (name, M, N, K, key), (_, _, wref), y in zip(layer.spec, layer.w, layer.outputs()):
        g = layer.g[key]
        ref = oracle.bitlinear_forward(wl.bf16_bits(layer.x[key]), None if g is None else wl.bf16_bits(g), wl.RMS_EPS,
                                       wref["wq"], wref["s_w"])
        ok = stable_rows(ref["fragile"], M)
        got = y.cpu().numpy().astype(np.float64)[ok]
        want = ref["y"].astype(np.float64)[ok]
        assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want)), name
        assert np.all(got[ref["acc"][ok] == 0] == 0.0), name


def check_against_single_calls(layer):
    """Bitwise equality with bitlinear_forward, the single-call kernel whose accumulators the full-size tests compare
    with the oracle one by one: the grouped call has no accumulator output of its own."""
    for (name, M, N, K, key), (packed, s_w, _), y in zip(layer.spec, layer.w, layer.outputs()):
        y1 = bl.bitlinear_forward(layer.x_dev[key], layer.g_dev[key], packed, s_w, N, wl.RMS_EPS, y_dtype=y.dtype)
        assert torch.equal(y, y1), name


def layer_spec(M):
    shared = {"q": "qkv", "k": "qkv", "v": "qkv", "o": "o", "gate": "gu", "up": "gu", "down": "down"}
    return [(name, M, n, k, shared[name]) for name, n, k in wl.LAYER_SHAPES]


def test_group_full_layer_as_benchmarked():
    # configs[3]: the seven matmuls of a layer at M = 2048 in ONE call, q/k/v and gate/up sharing their input tensor,
    # 1 % outlier channels; 360 pair tiles on 74 CTA pairs; then the same call with the quantiser launch skipped
    layer = Layer(layer_spec(2048), wl.seed_for(4, 0, 7))
    layer.run()
    check_sampled(layer, 1500, 11)
    check_against_single_calls(layer)
    first = [y.clone() for y in layer.outputs()]
    layer.poison()
    layer.run(reuse_act=True)
    for a, b in zip(first, layer.outputs()):
        assert torch.equal(a, b)
    layer.poison()
    layer.run()  # a full call again after a reuse call
    for a, b in zip(first, layer.outputs()):
        assert torch.equal(a, b)


def test_group_many_tiles_per_pair_mixed_k_element_by_element():
    # 186 pair tiles (more than twice the CTA pairs of a 148-SM part) over problems of K = 256 ... 6912 and ragged
    # token counts, so that every pair walks several tiles of different depth in one launch; every element checked
    spec = [("a", 1024, 5120, 256, "a"), ("b", 512, 2560, 6912, "b"), ("c", 512, 2560, 512, "c"),
            ("d", 300, 640, 2560, "d"), ("e", 1024, 2560, 256, "a"), ("f", 700, 1280, 768, "f")]
    layer = Layer(spec, 4242, x_kind="student_t")
    layer.run()
    check_full(layer)
    first = [y.clone() for y in layer.outputs()]
    layer.poison()
    layer.run(reuse_act=True)
    for a, b in zip(first, layer.outputs()):
        assert torch.equal(a, b)


def test_group_down_projection_4096_tokens_and_bf16():
    n, k = wl.SHAPE_NK["down"]
    layer = Layer([("down", 4096, n, k, "x"), ("k", 4096, 640, 2560, "y")], wl.seed_for(5, 0, 3), x_kind="student_t",
                  y_dtype=torch.bfloat16)
    layer.run()
    check_sampled(layer, 1500, 13)
    check_against_single_calls(layer)


def test_group_more_problems_than_one_launch_group():
    # 40 problems: two launch groups of at most 32 over consecutive workspace regions
    spec = []
    for j in range(20):  # pairs of problems; every other pair shares its input (same M, K, x and gain)
        M, K, share = 64 + 16 * j, 256 * (1 + j % 4), j % 2 == 0
        for t in range(2):
            i = 2 * j + t
            spec.append((f"p{i}", M if share else M + 8 * t, 128 * (1 + i % 3), K, f"s{j}" if share else f"u{i}"))
    layer = Layer(spec, 777, x_kind="normal")
    layer.run()
    check_full(layer)
