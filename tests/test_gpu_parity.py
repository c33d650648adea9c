"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Integer stages (int8 activations, packed bytes, ternary weights, int32 accumulators) must be
bit-exact; the fp32 output within 1e-6 relative (exactly 0 where the accumulator is 0); the bf16
output within one bf16 ulp.
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


def pack_both(W: torch.Tensor, eps=wl.WEIGHT_EPS):
    """Quantise + pack on the GPU and in the oracle; returns (gpu packed, gpu s_w, oracle dict)."""
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), eps)
    Wf = W.float().numpy()
    return packed, s_w, oracle.quantize_weights(Wf, eps)


def stable_rows(fragile):
    """Rows whose RMSNorm scale does not sit on an fp32 rounding boundary of the sum of squares
    (the oracle flags about one row in 1e5 where two valid fp64 summation orders may differ)."""
    ok = np.asarray(fragile) == 0
    flagged = int(ok.size - ok.sum())
    if flagged:
        print(f"rows flagged as fragile: {flagged} of {ok.size}")
    assert flagged <= ok.size // 1000  # none at all in cases of fewer than 1000 rows
    return ok


def assert_fp32_close(y, ref, acc):
    y = y.astype(np.float64)
    ref = ref.astype(np.float64)
    assert np.all(np.abs(y - ref) <= 1e-6 * np.abs(ref)), float(np.max(np.abs(y - ref) / np.maximum(np.abs(ref), 1e-30)))
    assert np.all(y[acc == 0] == 0.0)


# ------------------------------------------------------------------------------- weights


@pytest.mark.parametrize("N,K", [(16, 256), (48, 768), (640, 2560), (2560, 6912)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_pack_weights_bit_exact(N, K, dtype):
    if dtype == torch.bfloat16 and N * K > 2_000_000:
        pytest.skip("bf16 master weights covered at the smaller shapes")
    W = wl.latent_weights(N, K, wl.seed_for(2, 1, N % 7)).to(dtype)
    packed, s_w, ref = pack_both(W)
    assert not ref["fragile"]
    assert packed.numel() == N * K // 4
    assert np.float32(to_np(s_w)[0]) == ref["s_w"]
    assert np.array_equal(to_np(packed), ref["packed"])
    wq = bl.bitlinear_unpack_weights(packed, N, K)
    assert np.array_equal(to_np(wq), ref["wq"])
    assert set(np.unique(to_np(wq)).tolist()) <= {-1, 0, 1}


def test_pack_weights_edge_cases():
    # all-zero matrix: scale = eps, all trits 0, packed bytes all 0x55
    W = torch.zeros(16, 256)
    packed, s_w, ref = pack_both(W)
    assert np.array_equal(to_np(packed), ref["packed"]) and np.all(to_np(packed) == 0x55)
    assert np.float32(to_np(s_w)[0]) == np.float32(1e-5)
    # ties and clipping: mean|W| = 1 exactly with eps 0
    W = torch.tensor([1.0, 1.0, 0.5, 1.5, -1.0, -1.0, -0.5, -1.5] * 512).reshape(16, 256)
    packed, s_w, ref = pack_both(W, eps=0.0)
    assert float(to_np(s_w)[0]) == 1.0
    assert np.array_equal(to_np(packed), ref["packed"])
    assert to_np(bl.bitlinear_unpack_weights(packed, 16, 256))[0, :8].tolist() == [1, 1, 0, 1, -1, -1, 0, -1]
    # deterministic run to run
    W = wl.latent_weights(128, 512, 99)
    p1, s1 = bl.bitlinear_pack_weights(W.to(DEV))
    p2, s2 = bl.bitlinear_pack_weights(W.to(DEV))
    assert torch.equal(p1, p2) and torch.equal(s1, s2)


# ------------------------------------------------------------------------------- activations


@pytest.mark.parametrize("M,K", [(1, 256), (3, 768), (17, 2560), (5, 6912), (2, 16384), (300, 2560)])
@pytest.mark.parametrize("kind", ["normal", "outlier", "student_t"])
def test_quant_act_bit_exact(M, K, kind):
    gen = {"normal": wl.activations_normal, "outlier": wl.activations_outlier, "student_t": wl.activations_student_t}[kind]
    x = gen(M, K, wl.seed_for(2, 0, M))
    gain = wl.gain_random(K, 5) if kind == "normal" else None
    ref = oracle.rmsnorm_quant(wl.bf16_bits(x), None if gain is None else wl.bf16_bits(gain), wl.RMS_EPS)
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None if gain is None else gain.to(DEV), wl.RMS_EPS)
    ok = stable_rows(ref["fragile"])
    assert np.array_equal(to_np(xq)[ok], ref["q"][ok])
    assert np.array_equal(to_np(d).view(np.uint32)[ok], ref["d"].view(np.uint32)[ok])
    assert np.array_equal(to_np(xsum)[ok], ref["xsum"][ok])


def test_quant_act_edge_rows():
    K = 2560
    x = torch.zeros(6, K)
    x[1] = 1.0            # constant row -> all 127
    x[2] = -3.0           # constant negative -> all -127
    x[3, 77] = -2.0       # single spike
    x[4] = torch.linspace(-1, 1, K)
    x[5, ::2] = 6.1e-5    # tiny values, stays far above denormals after the square
    xb = x.to(torch.bfloat16)
    ref = oracle.rmsnorm_quant(wl.bf16_bits(xb), None, wl.RMS_EPS)
    xq, d, xsum = bl.bitlinear_quant_act(xb.to(DEV), None, wl.RMS_EPS)
    assert np.array_equal(to_np(xq), ref["q"])
    assert np.array_equal(to_np(d), ref["d"])
    assert np.array_equal(to_np(xsum), ref["xsum"])
    q = to_np(xq)
    assert not q[0].any() and np.all(q[1] == 127) and np.all(q[2] == -127)
    assert q[3, 77] == -127 and np.count_nonzero(q[3]) == 1
    assert q.min() >= -127


def test_quant_act_guard_bands_and_determinism():
    M, K = 7, 2560
    x = wl.activations_normal(M, K, 1234).to(DEV)
    lib = bl.lib()
    pad = 256
    buf = torch.full((pad + M * K + pad,), 0x5A, dtype=torch.uint8, device=DEV)
    dbuf = torch.full((64 + M + 64,), -7.0, dtype=torch.float32, device=DEV)
    sbuf = torch.full((64 + M + 64,), -7, dtype=torch.int32, device=DEV)
    rc = lib.bitlinear_quant_act(x.data_ptr(), None, wl.RMS_EPS, M, K, buf.data_ptr() + pad, dbuf.data_ptr() + 256,
                                 sbuf.data_ptr() + 256, torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert torch.all(buf[:pad] == 0x5A) and torch.all(buf[pad + M * K:] == 0x5A)
    assert torch.all(dbuf[:64] == -7.0) and torch.all(dbuf[64 + M:] == -7.0)
    assert torch.all(sbuf[:64] == -7) and torch.all(sbuf[64 + M:] == -7)
    xq, d, xsum = bl.bitlinear_quant_act(x, None, wl.RMS_EPS)
    assert torch.equal(buf[pad:pad + M * K].view(torch.int8).view(M, K), xq)
    assert torch.equal(dbuf[64:64 + M], d) and torch.equal(sbuf[64:64 + M], xsum)


# ------------------------------------------------------------------------------- contraction


def run_matmul_case(M, N, K, seed, path, y_dtype=torch.float32, x_kind="normal"):
    gen = {"normal": wl.activations_normal, "outlier": wl.activations_outlier, "student_t": wl.activations_student_t}[x_kind]
    x = gen(M, K, seed)
    W = wl.latent_weights(N, K, seed + 1)
    packed, s_w, wref = pack_both(W)
    assert np.array_equal(to_np(packed), wref["packed"])
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), None, wl.RMS_EPS, wref["wq"], wref["s_w"])
    ok = stable_rows(ref["fragile"])
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    y, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, y_dtype=y_dtype, want_acc=True, path=path)
    assert np.array_equal(to_np(xq)[ok], ref["q"][ok])
    assert np.array_equal(to_np(acc)[ok], ref["acc"][ok])
    if y_dtype == torch.float32:
        assert_fp32_close(to_np(y)[ok], ref["y"][ok], ref["acc"][ok])
    else:
        want = oracle.f32_to_bf16(ref["y"]).astype(np.int32)[ok]
        got = wl.bf16_bits(y.cpu()).astype(np.int32)[ok]
        # same sign (or both zero) and at most one ulp apart
        assert np.all(np.abs(got - want) <= 1)
    return y


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 9, 16])
@pytest.mark.parametrize("N,K", [(16, 256), (48, 768), (128, 1024), (640, 2560), (2560, 6912)])
def test_gemv_parity(M, N, K):
    if N * K > 2_000_000 and M not in (1, 4, 16):
        pytest.skip("large shape covered at M in {1,4,16}")
    run_matmul_case(M, N, K, wl.seed_for(2, 3, M), bl.PATH_GEMV)


@pytest.mark.parametrize("M", [17, 33, 40])
def test_gemv_parity_beyond_sixteen_tokens(M):
    run_matmul_case(M, 48, 768, wl.seed_for(5, 0, M), bl.PATH_GEMV, x_kind="student_t")


@pytest.mark.parametrize("M", [1, 5, 16])
def test_gemv_bf16_output_within_one_ulp(M):
    run_matmul_case(M, 640, 2560, wl.seed_for(2, 1, M), bl.PATH_GEMV, y_dtype=torch.bfloat16)


def test_gemv_structured_weights_pin_the_packed_layout():
    # identity and one-hot patterns travel through the GPU packer AND the GPU contraction: any
    # permutation error in the packed layout or in the kernel's indexing shows up here
    M, N, K = 3, 256, 256
    x = wl.activations_normal(M, K, 77)
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    q = to_np(xq).astype(np.int32)

    def acc_for(Wt):
        packed, s_w = bl.bitlinear_pack_weights(Wt.to(DEV), 0.0)
        _, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, want_acc=True, path=bl.PATH_GEMV)
        return to_np(acc)

    assert np.array_equal(acc_for(torch.eye(N, K)), q)
    assert np.array_equal(acc_for(-torch.eye(N, K)), -q)
    assert np.array_equal(acc_for(torch.ones(N, K)), np.repeat(q.sum(axis=1, keepdims=True), N, axis=1))
    shifted = torch.roll(torch.eye(N, K), shifts=37, dims=1)  # W[n, (n+37) % K] = 1
    assert np.array_equal(acc_for(shifted), np.roll(q, -37, axis=1))
    for (n, k) in ((0, 0), (5, 200), (255, 1), (100, 101), (17, 255)):
        Wt = torch.zeros(N, K)
        Wt[n, k] = -1.0
        # mean|W| is tiny here, so the single entry saturates to -1
        expect = np.zeros((M, N), np.int32)
        expect[:, n] = -q[:, k]
        assert np.array_equal(acc_for(Wt), expect)


def test_extreme_accumulators_do_not_overflow():
    N, K = 16, 16384
    x = torch.ones(2, K, dtype=torch.bfloat16)
    x[1] = -1.0
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, 0.0)
    for sign in (1.0, -1.0):
        packed, s_w = bl.bitlinear_pack_weights((sign * torch.ones(N, K)).to(DEV), 0.0)
        _, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, want_acc=True, path=bl.PATH_GEMV)
        a = to_np(acc)
        assert np.all(a[0] == sign * 127 * K) and np.all(a[1] == -sign * 127 * K)


# ------------------------------------------------------------------------------- whole forward


@pytest.mark.parametrize("name", [n for n, _, _ in wl.LAYER_SHAPES])
@pytest.mark.parametrize("M", [1, 4, 16])
def test_forward_layer_shapes_decode(name, M):
    N, K = wl.SHAPE_NK[name]
    seed = wl.seed_for(2, wl.SHAPE_INDEX[name], M)
    x = wl.activations_normal(M, K, seed)
    gain = wl.gain_ones(K)
    W = wl.latent_weights(N, K, seed + 1)
    packed, s_w, wref = pack_both(W)
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), wl.bf16_bits(gain), wl.RMS_EPS, wref["wq"], wref["s_w"])
    y = bl.bitlinear_forward(x.to(DEV), gain.to(DEV), packed, s_w, N, wl.RMS_EPS)
    ok = stable_rows(ref["fragile"])
    assert_fp32_close(to_np(y)[ok], ref["y"][ok], ref["acc"][ok])
    # twice the same bits
    y2 = bl.bitlinear_forward(x.to(DEV), gain.to(DEV), packed, s_w, N, wl.RMS_EPS)
    assert torch.equal(y, y2)


def test_forward_host_buffers():
    M, N, K = 4, 640, 2560
    x = wl.activations_normal(M, K, 4242)
    W = wl.latent_weights(N, K, 4243)
    packed, s_w, wref = pack_both(W)
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), None, wl.RMS_EPS, wref["wq"], wref["s_w"])
    xh = x.pin_memory()
    yh = torch.empty(M, N, dtype=torch.float32).pin_memory()
    bl.bitlinear_forward_host(xh, None, packed, s_w, N, yh, wl.RMS_EPS)
    assert_fp32_close(yh.numpy(), ref["y"], ref["acc"])


def test_empty_batch_and_status():
    packed, s_w = bl.bitlinear_pack_weights(wl.latent_weights(16, 256, 1).to(DEV))
    x = torch.empty(0, 256, dtype=torch.bfloat16, device=DEV)
    y = bl.bitlinear_forward(x, None, packed, s_w, 16)
    assert y.shape == (0, 16)
    assert bl.bitlinear_poll_status() == 0
