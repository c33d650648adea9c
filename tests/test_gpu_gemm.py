"""Parity of the tcgen05 tensor-core contraction (prefill path) with the CPU oracle.

Small and ragged cases are compared element by element; the full prefill shapes (M = 2048 on the
seven layer shapes, and the batch sweep on the FFN down projection) are compared on sampled
outputs the oracle computes one by one, plus row/column sums that hold at any size.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def to_np(t):
    return t.detach().cpu().numpy()


def stable_rows(fragile):
    """Rows whose RMSNorm scale does not sit on an fp32 rounding boundary of the sum of squares.

    On the (about one in 1e5) rows the oracle flags, two equally valid fp64 summation orders may
    round the scale to neighbouring fp32 values, so bit-exactness is only required elsewhere."""
    ok = np.asarray(fragile) == 0
    flagged = int(ok.size - ok.sum())
    if flagged:
        print(f"rows flagged as fragile: {flagged} of {ok.size}")
    assert flagged <= ok.size // 1000  # none at all in cases of fewer than 1000 rows
    return ok


def check_full(M, N, K, seed, x_kind="normal", y_dtype=torch.float32, path=None):
    path = bl.PATH_GEMM if path is None else path
    gen = {"normal": wl.activations_normal, "outlier": wl.activations_outlier, "student_t": wl.activations_student_t}[x_kind]
    x = gen(M, K, seed)
    W = wl.latent_weights(N, K, seed + 1)
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
    assert np.array_equal(to_np(packed), wref["packed"])
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), None, wl.RMS_EPS, wref["wq"], wref["s_w"])
    ok = stable_rows(ref["fragile"])
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    y, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, y_dtype=y_dtype, want_acc=True, path=path)
    assert bl.bitlinear_poll_status() == 0
    assert np.array_equal(to_np(acc)[ok], ref["acc"][ok])
    if y_dtype == torch.float32:
        yy = to_np(y).astype(np.float64)[ok]
        rr = ref["y"].astype(np.float64)[ok]
        assert np.all(np.abs(yy - rr) <= 1e-6 * np.abs(rr))
        assert np.all(yy[ref["acc"][ok] == 0] == 0.0)
    else:
        want = oracle.f32_to_bf16(ref["y"]).astype(np.int32)[ok]
        got = wl.bf16_bits(y.cpu()).astype(np.int32)[ok]
        assert np.all(np.abs(got - want) <= 1)


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 256),     # exactly one tile, two k-blocks
    (17, 128, 256),      # fewer tokens than a tile, half a tile of weight rows
    (64, 128, 512),
    (129, 384, 768),     # ragged in M and N
    (300, 640, 2560),    # the k/v projection shape, three token tiles with a tail
    (256, 512, 6912),    # long K: the ring wraps many times
])
def test_gemm_parity_small(M, N, K):
    check_full(M, N, K, wl.seed_for(4, 0, M % 10))


def test_gemm_parity_forced_at_decode_sizes():
    for M in (1, 5, 16):
        check_full(M, 256, 512, wl.seed_for(5, 0, M), x_kind="student_t")


def test_gemm_bf16_output():
    check_full(130, 256, 768, wl.seed_for(4, 1, 3), y_dtype=torch.bfloat16, x_kind="outlier")


def test_gemm_many_tiles_per_cta():
    # more tiles than SMs so that every CTA loops and both accumulator buffers are reused
    check_full(1024, 5120, 256, wl.seed_for(4, 2, 1))


def test_auto_path_switches_above_sixteen_tokens_and_matches_gemv():
    M, N, K = 48, 256, 512
    x = wl.activations_normal(M, K, 31)
    packed, s_w = bl.bitlinear_pack_weights(wl.latent_weights(N, K, 32).to(DEV))
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    y_auto = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N)
    y_gemv = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, path=bl.PATH_GEMV)
    y_gemm = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, path=bl.PATH_GEMM)
    assert torch.equal(y_auto, y_gemm) and torch.equal(y_gemv, y_gemm)
    y_fwd = bl.bitlinear_forward(x.to(DEV), None, packed, s_w, N)
    assert torch.equal(y_fwd, y_gemm)


def sampled_check(M, N, K, x, W, n_samples=4096, seed=0):
    """Full-size case: sampled accumulators bit-exact, sampled outputs within tolerance, and the
    all-column sum of every token's accumulators against an int64 identity."""
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
    assert np.array_equal(to_np(packed), wref["packed"])
    qref = oracle.rmsnorm_quant(wl.bf16_bits(x), None, wl.RMS_EPS)
    ok = stable_rows(qref["fragile"])
    y = bl.bitlinear_forward(x.to(DEV), None, packed, s_w, N)
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    y2, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, want_acc=True)
    assert bl.bitlinear_poll_status() == 0
    assert torch.equal(y, y2)
    assert np.array_equal(to_np(xq)[ok], qref["q"][ok])
    rng = np.random.default_rng(seed)
    m_idx = rng.choice(np.nonzero(ok)[0], n_samples).astype(np.int32)
    n_idx = rng.integers(0, N, n_samples).astype(np.int32)
    # make sure the corners and tile edges are in the sample
    edge_m = np.array([0, M - 1, min(127, M - 1), min(128, M - 1), M - 1], np.int32)
    edge_n = np.array([0, N - 1, 255 % N, 256 % N, 0], np.int32)
    keep = ok[edge_m]
    m_idx = np.concatenate([m_idx, edge_m[keep]])
    n_idx = np.concatenate([n_idx, edge_n[keep]])
    acc_ref = oracle.matmul_i32_sampled(qref["q"], wref["wq"], m_idx, n_idx)
    acc_gpu = to_np(acc)
    assert np.array_equal(acc_gpu[m_idx, n_idx], acc_ref)
    y_ref = oracle.dequant(acc_ref.reshape(1, -1), wref["s_w"], np.ones(1, np.float32))  # acc * s_w
    y_ref = (y_ref[0] * qref["d"][m_idx]).astype(np.float32)
    got = to_np(y)[m_idx, n_idx].astype(np.float64)
    assert np.all(np.abs(got - y_ref.astype(np.float64)) <= 1e-6 * np.abs(y_ref.astype(np.float64)))
    # property at full size: sum_n acc[m, n] = q[m, :] . (sum_n Wq[n, :])
    col = wref["wq"].astype(np.int64).sum(axis=0)
    want_rows = qref["q"].astype(np.int64) @ col
    assert np.array_equal(acc_gpu.astype(np.int64).sum(axis=1)[ok], want_rows[ok])


@pytest.mark.parametrize("name", [n for n, _, _ in wl.LAYER_SHAPES])
def test_prefill_layer_shapes_sampled(name):
    N, K = wl.SHAPE_NK[name]
    M = 2048
    seed = wl.seed_for(4, wl.SHAPE_INDEX[name])
    sampled_check(M, N, K, wl.activations_outlier(M, K, seed), wl.latent_weights(N, K, seed + 1), seed=seed)


@pytest.mark.parametrize("M", [32, 64, 256, 1024, 4096])
def test_batch_sweep_down_projection_sampled(M):
    N, K = wl.SHAPE_NK["down"]
    seed = wl.seed_for(5, 0, M % 10)
    sampled_check(M, N, K, wl.activations_student_t(M, K, seed), wl.latent_weights(N, K, wl.seed_for(5, 0) + 1),
                  n_samples=2048, seed=seed)
