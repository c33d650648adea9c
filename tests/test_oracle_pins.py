"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's formulas to compare it with itself:
each one is a hand-computed value, an invariant the paper states (ternary
weights, 8-bit activations, four weights per byte: Section 2 and Section 5.1),
a closed form, a special case that reduces to a textbook or library routine, or
a brute-force evaluation of the definition in fp64 / int64.
"""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2504_12285_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits_of(values):
    """Exact bf16 bit patterns of fp32 values that are representable in bf16."""
    a = np.asarray(values, np.float32)
    bits = a.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0), "test value is not exactly representable in bf16"
    return (bits >> 16).astype(np.uint16)


# --------------------------------------------------------------------------- weights


def test_weight_quant_hand_case():
    # mean|W| = (0.3+0.1+0.05+0.55)/4 = 0.25; ratios 1.2, -0.4, 0.2, -2.2 -> round 1, 0, 0, -2 -> clip 1, 0, 0, -1
    W = np.array([[0.3, -0.1, 0.05, -0.55]], np.float32)
    for eps in (0.0, 1e-5):
        s_w, _ = oracle.weight_scale(W, eps)
        assert abs(float(s_w) - (0.25 + eps)) < 1e-7
        assert oracle.weight_quant(W, s_w).tolist() == [[1, 0, 0, -1]]


def test_weight_quant_ties_round_half_to_even():
    # mean|W| = 1 exactly, eps 0: ratios 1, 1, 0.5, 1.5.  Half-to-even gives 0 and 2 (clipped to 1);
    # half-away-from-zero would give 1 for the 0.5.  -0.5 and -1.5 mirror it.
    W = np.array([[1.0, 1.0, 0.5, 1.5]], np.float32)
    s_w, _ = oracle.weight_scale(W, 0.0)
    assert float(s_w) == 1.0
    assert oracle.weight_quant(W, s_w).tolist() == [[1, 1, 0, 1]]
    Wn = np.array([[-1.0, -1.0, -0.5, -1.5]], np.float32)
    assert oracle.weight_quant(Wn, np.float32(1.0)).tolist() == [[-1, -1, 0, -1]]
    # 2.5 -> 2 -> clip 1 and -2.5 -> -2 -> clip -1: clipping works on both sides
    assert oracle.weight_quant(np.array([[2.5, -2.5, 0.49, -0.51]], np.float32), np.float32(1.0)).tolist() == [
        [1, -1, 0, -1]
    ]


def test_weight_quant_all_zero_matrix():
    W = np.zeros((16, 256), np.float32)
    s_w, _ = oracle.weight_scale(W, 1e-5)
    assert float(s_w) == float(np.float32(1e-5))
    wq = oracle.weight_quant(W, s_w)
    assert not wq.any()


def test_weight_scale_is_the_mean_absolute_value():
    # 1, -2, 3, -4 ... mean of |.| over 1..64 is 32.5 (exact in fp32)
    W = (np.arange(1, 65, dtype=np.float32) * np.where(np.arange(64) % 2, -1, 1)).reshape(4, 16)
    s_w, fragile = oracle.weight_scale(W, 0.0)
    assert float(s_w) == 32.5 and not fragile


def test_weights_are_ternary_and_match_gaussian_closed_form():
    # For W ~ N(0, sigma^2): mean|W| -> sigma*sqrt(2/pi); a weight quantises to 0 iff |W| < s_w/2,
    # so P(0) = erf( s_w / (2*sqrt(2)*sigma) ) = 0.3101 and P(+1) = P(-1) = 0.3450.
    sigma = wl.WEIGHT_STD
    W = wl.latent_weights(2560, 2560, wl.seed_for(1, 0)).numpy()
    s_w, _ = oracle.weight_scale(W, wl.WEIGHT_EPS)
    s_theory = sigma * math.sqrt(2.0 / math.pi) + wl.WEIGHT_EPS
    assert abs(float(s_w) - s_theory) / s_theory < 1e-3
    wq = oracle.weight_quant(W, s_w)
    assert set(np.unique(wq).tolist()) == {-1, 0, 1}
    p0 = math.erf(s_theory / (2.0 * math.sqrt(2.0) * sigma))
    assert abs(p0 - 0.3101) < 2e-4
    assert abs(float((wq == 0).mean()) - p0) < 1e-3
    assert abs(float((wq == 1).mean()) - (1 - p0) / 2) < 1e-3
    assert abs(float((wq == -1).mean()) - (1 - p0) / 2) < 1e-3
    # the quantiser is odd: W -> -W flips every trit
    assert np.array_equal(oracle.weight_quant(-W, s_w), -wq)


# --------------------------------------------------------------------------- activations


def test_act_quant_hand_cases():
    # a = 127 -> s = 1: values are rounded directly; ties go to even (0.5->0, 1.5->2, 2.5->2)
    y = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -2.5]], np.float32)
    q, d, xsum = oracle.absmax_quant(y)
    assert q.tolist() == [[127, 0, 2, 2, 0, -2]]
    assert float(d[0]) == 1.0 and int(xsum[0]) == 129
    # a = 2 -> s = 63.5: 63.5 -> 64 (tie to even), -127, 31.75 -> 32, 0
    y = np.array([[1.0, -2.0, 0.5, 0.0]], np.float32)
    q, d, xsum = oracle.absmax_quant(y)
    assert q.tolist() == [[64, -127, 32, 0]]
    assert float(d[0]) == float(np.float32(2.0) / np.float32(127.0))
    assert int(xsum[0]) == 64 - 127 + 32


def test_act_quant_zero_row_is_safe():
    q, d, xsum = oracle.absmax_quant(np.zeros((2, 8), np.float32))
    assert not q.any() and not xsum.any()
    assert np.all(d == np.float32(1e-5) / np.float32(127.0))


def test_act_quant_range_invariants():
    # 8-bit per-token absmax: every non-zero row reaches |q| = 127 and nothing reaches -128
    for gen, cfg in ((wl.activations_normal, 2), (wl.activations_outlier, 4), (wl.activations_student_t, 5)):
        x = gen(33, 2560, wl.seed_for(cfg, 0))
        out = oracle.rmsnorm_quant(wl.bf16_bits(x), wl.bf16_bits(wl.gain_ones(2560)), wl.RMS_EPS)
        q = out["q"].astype(np.int32)
        assert q.min() >= -127 and q.max() <= 127
        assert np.all(np.abs(q).max(axis=1) == 127)
        assert np.array_equal(out["xsum"], q.sum(axis=1))


def test_rmsnorm_constant_row_and_single_spike():
    K = 256
    # constant row c: y_i = c / sqrt(c^2 + eps), all equal -> every code is +-127
    for c in (1.0, -3.0, 0.015625):
        x = bf16_bits_of(np.full((1, K), c, np.float32))
        out = oracle.rmsnorm_quant(x, None, 1e-5, want_norm=True)
        assert np.all(out["q"] == (127 if c > 0 else -127))
        expect = c / math.sqrt(c * c + 1e-5)
        assert np.allclose(out["y_norm"], expect, rtol=3e-7, atol=0)
        assert abs(float(out["d"][0]) - abs(expect) / 127.0) <= 3e-7 * abs(expect) / 127.0
    # a single spike c at position 5: y_5 = c / sqrt(c^2/K + eps), the rest 0
    x = np.zeros((1, K), np.float32)
    x[0, 5] = -2.0
    out = oracle.rmsnorm_quant(bf16_bits_of(x), None, 1e-5, want_norm=True)
    q = out["q"][0]
    assert q[5] == -127 and not np.delete(q, 5).any()
    assert abs(float(out["y_norm"][0, 5]) - (-2.0 / math.sqrt(4.0 / K + 1e-5))) < 1e-5
    # all-zero token
    out = oracle.rmsnorm_quant(np.zeros((1, K), np.uint16), None, 1e-5)
    assert not out["q"].any() and int(out["xsum"][0]) == 0


def test_rmsnorm_matches_textbook_fp64():
    K = 2560
    x = wl.activations_normal(7, K, wl.seed_for(2, 3))
    g = wl.gain_random(K, wl.seed_for(2, 3, 1))
    out = oracle.rmsnorm_quant(wl.bf16_bits(x), wl.bf16_bits(g), wl.RMS_EPS, want_norm=True)
    xd = x.double().numpy()
    gd = g.double().numpy()
    ref = xd / np.sqrt((xd * xd).mean(axis=1, keepdims=True) + wl.RMS_EPS) * gd
    assert np.allclose(out["y_norm"], ref, rtol=3e-7, atol=1e-12)
    # and the quantised row dequantises back to the normalised row within half a step
    deq = out["q"].astype(np.float64) * out["d"][:, None].astype(np.float64)
    assert np.all(np.abs(deq - ref) <= 0.5 * out["d"][:, None] * (1 + 1e-5))
    assert not out["fragile"].any()


def test_gain_is_applied_per_channel():
    K = 256
    x = bf16_bits_of(np.ones((1, K), np.float32))
    g = np.ones(K, np.float32)
    g[3] = 2.0
    g[9] = -0.5
    out = oracle.rmsnorm_quant(x, bf16_bits_of(g), 0.0)
    q = out["q"][0]
    # y = g exactly (r = 1): a = 2 -> s = 63.5 -> 63.5 rounds to 64 (tie to even), 127, -31.75 -> -32
    assert q[3] == 127 and q[9] == -32 and q[0] == 64


def test_bf16_rounding_is_nearest_even():
    f = np.array([1.0, 1.00390625, 1.01171875, 1.0078125, -1.00390625, 3.0e38], np.float32)
    # 1 + 2^-8 is a tie between 1.0 (even) and 1 + 2^-7 -> 1.0;  1 + 3*2^-8 is a tie -> 1 + 2^-6 (even)
    bits = oracle.f32_to_bf16(f)
    back = oracle.bf16_to_f32(bits)
    assert back.tolist()[:5] == [1.0, 1.0, 1.015625, 1.0078125, -1.0]
    assert np.isfinite(back[5])
    # agrees with the library cast on random data
    import torch

    r = torch.randn(4096, generator=torch.Generator().manual_seed(7))
    assert np.array_equal(oracle.f32_to_bf16(r.numpy()), wl.bf16_bits(r.to(torch.bfloat16)))


# --------------------------------------------------------------------------- packing


def _golden_positions():
    rows = []
    with open(os.path.join(GOLDEN, "pack_layout_positions.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(tuple(int(v) for v in line.split()))
    return rows


@pytest.mark.parametrize("n,k,byte,shift", _golden_positions())
def test_pack_positions_match_hand_computed_layout(n, k, byte, shift):
    N, K = 32, 512
    for trit in (1, -1):
        wq = np.zeros((N, K), np.int8)
        wq[n, k] = trit
        packed = oracle.pack(wq)
        assert packed.size == N * K // 4  # four ternary values per byte, exactly
        expect = np.full(N * K // 4, 0x55, np.uint8)  # code 1 (= trit 0) everywhere
        expect[byte] = (0x55 & ~(3 << shift)) | ((trit + 1) << shift)
        assert np.array_equal(packed, expect)


def test_pack_roundtrip_all_byte_patterns_and_random():
    # all 3^4 combinations of four neighbouring trits, at every position of one tile
    N, K = 16, 256
    combos = np.array(np.meshgrid(*[[-1, 0, 1]] * 4, indexing="ij")).reshape(4, -1).T  # 81 x 4
    wq = np.zeros((N, K), np.int8)
    flat = wq.reshape(-1, 4)
    for r in range(flat.shape[0]):
        flat[r] = combos[r % 81]
    packed = oracle.pack(wq)
    assert np.array_equal(oracle.unpack(packed, N, K), wq)
    # the code 3 never appears in any 2-bit field
    fields = np.stack([(packed >> s) & 3 for s in (0, 2, 4, 6)])
    assert fields.max() == 2
    rng = np.random.default_rng(3)
    wq = rng.integers(-1, 2, size=(48, 768)).astype(np.int8)
    packed = oracle.pack(wq)
    assert packed.size == 48 * 768 // 4
    assert np.array_equal(oracle.unpack(packed, 48, 768), wq)
    # a 16-byte chunk is 64 consecutive columns of one row: flipping them touches only that chunk
    wq2 = wq.copy()
    wq2[17, 320:384] = -wq2[17, 320:384] + (wq2[17, 320:384] == 0)
    diff = np.nonzero(oracle.pack(wq2) != packed)[0]
    assert diff.size > 0 and diff.min() // 16 == diff.max() // 16
    with pytest.raises(ValueError):
        oracle.pack(np.zeros((8, 256), np.int8))
    with pytest.raises(ValueError):
        oracle.pack(np.full((16, 256), 2, np.int8))


# --------------------------------------------------------------------------- dense packing: five per byte


def _golden_positions5():
    rows = []
    with open(os.path.join(GOLDEN, "pack5_layout_positions.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(tuple(int(v) for v in line.split()))
    return rows


@pytest.mark.parametrize("n,k,byte,digit,plus,minus", _golden_positions5())
def test_pack5_positions_match_hand_computed_layout(n, k, byte, digit, plus, minus):
    N, K = 32, 512
    for trit, value in ((1, plus), (-1, minus)):
        wq = np.zeros((N, K), np.int8)
        wq[n, k] = trit
        packed = oracle.pack5(wq)
        assert packed.size == 4096  # 32 rows x 640 padded columns / 5
        expect = np.full(4096, 128, np.uint8)  # five zero weights: v = 121 -> byte 128
        expect[byte] = value
        assert np.array_equal(packed, expect)
        assert np.array_equal(oracle.unpack5(packed, N, K), wq)


def test_pack5_all_243_byte_patterns():
    # Every combination of five neighbouring weights.  Column c = 4*e + b of a 20-column word is digit e of byte b,
    # so the five weights of byte 0 of the first word of row 0 are columns 0, 4, 8, 12, 16.
    from fractions import Fraction
    combos = np.array(np.meshgrid(*[[-1, 0, 1]] * 5, indexing="ij")).reshape(5, -1).T  # 243 x 5, digit 0 slowest
    seen = {}
    for trits in combos:
        wq = np.zeros((16, 256), np.int8)
        wq[0, [0, 4, 8, 12, 16]] = trits
        packed = oracle.pack5(wq)
        assert packed.size == 16 * 320 // 5 and np.all(packed[1:] == 128)
        B = int(packed[0])
        # the byte is the base-3 fraction 0.c0 c1 c2 c3 c4 scaled by 256 and rounded up
        frac = sum(Fraction(int(t) + 1, 3 ** (e + 1)) for e, t in enumerate(trits))
        assert B == -((-256 * frac.numerator) // frac.denominator)
        assert B not in seen
        seen[B] = tuple(trits)
        # peeling digits by repeated multiplication by 3 (what a decoder without division does) returns the codes
        rem = B
        for t in trits:
            rem *= 3
            assert rem >> 8 == int(t) + 1
            rem &= 255
        assert np.array_equal(oracle.unpack5(packed, 16, 256), wq)
    assert len(seen) == 243 and min(seen) == 0 and max(seen) == 255
    # byte values grow with the base-3 number, and the thirteen values no five codes produce are rejected
    order = sorted(seen)
    assert [seen[b] for b in order] == [tuple(c) for c in combos]
    unused = sorted(set(range(256)) - set(seen))
    assert len(unused) == 13
    for b in unused:
        bad = np.full(16 * 64, 128, np.uint8)
        bad[5] = b
        with pytest.raises(ValueError):
            oracle.unpack5(bad, 16, 256)


def test_pack5_size_roundtrip_and_locality():
    # Table 1's budget: 5 weights per byte where K is a multiple of 320, at most one extra tile of padding otherwise
    assert oracle.packed5_bytes(2560, 2560) == 2560 * 2560 // 5
    assert oracle.packed5_bytes(640, 2560) == 640 * 2560 // 5
    assert oracle.packed5_bytes(2560, 6912) == 2560 * 7040 // 5
    layer = sum(oracle.packed5_bytes(n, k) for n, k in ((2560, 2560), (640, 2560), (640, 2560), (2560, 2560),
                                                         (6912, 2560), (6912, 2560), (2560, 6912)))
    assert layer == 13_959_168 and 30 * layer == 418_775_040  # against 521,011,200 at four per byte
    assert oracle.packed5_bytes(8, 256) == 0 and oracle.packed5_bytes(16, 100) == 0
    rng = np.random.default_rng(5)
    for N, K in ((48, 768), (16, 256), (32, 6912), (640, 2560)):
        wq = rng.integers(-1, 2, size=(N, K)).astype(np.int8)
        packed = oracle.pack5(wq)
        assert packed.size == oracle.packed5_bytes(N, K)
        assert np.array_equal(oracle.unpack5(packed, N, K), wq)
    # padding columns hold zero weights: the last tile of a 256-column matrix has 64 of them per row, i.e. whole
    # words of value 128 wherever all 20 columns of the word are padding (columns 260..319 of the tile)
    wq = rng.integers(-1, 2, size=(16, 256)).astype(np.int8)
    tile = oracle.pack5(wq).reshape(2, 8, 4, 4, 4)  # h, g, t, i, b
    assert np.all(tile[:, :, 3, 1:, :] == 128)  # t = 3 covers columns 240..319: words i = 1..3 are columns 260..319
    # a 16-byte chunk is 80 consecutive columns of one row: flipping them touches only that chunk
    wq = rng.integers(-1, 2, size=(48, 768)).astype(np.int8)
    packed = oracle.pack5(wq)
    wq2 = wq.copy()
    wq2[17, 400:480] = -wq2[17, 400:480] + (wq2[17, 400:480] == 0)
    diff = np.nonzero(oracle.pack5(wq2) != packed)[0]
    assert diff.size > 0 and diff.min() // 16 == diff.max() // 16
    with pytest.raises(ValueError):
        oracle.pack5(np.full((16, 256), 2, np.int8))


def test_pack5_identity_and_one_hot_weights_through_the_contraction():
    # unpack5(pack5(W)) feeds the same contraction: the identity pattern returns the activations themselves, so any
    # permutation of rows or columns inside the dense layout would show
    rng = np.random.default_rng(6)
    K = N = 512
    q = rng.integers(-127, 128, size=(3, K)).astype(np.int8)
    eye = np.eye(N, K, dtype=np.int8)
    w = oracle.unpack5(oracle.pack5(eye), N, K)
    assert np.array_equal(oracle.matmul_i32(q, w), q.astype(np.int32))
    w = oracle.unpack5(oracle.pack5(-eye[::-1].copy()), N, K)
    assert np.array_equal(oracle.matmul_i32(q, w), -q[:, ::-1].astype(np.int32))


# --------------------------------------------------------------------------- contraction and epilogue


def _rand_case(M, N, K, seed):
    rng = np.random.default_rng(seed)
    q = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
    wq = rng.integers(-1, 2, size=(N, K)).astype(np.int8)
    return q, wq


def test_matmul_matches_int64_library_matmul():
    for (M, N, K) in ((1, 16, 256), (3, 48, 512), (4, 128, 256)):
        q, wq = _rand_case(M, N, K, M * 1000 + N)
        ref = q.astype(np.int64) @ wq.astype(np.int64).T
        assert np.array_equal(oracle.matmul_i32(q, wq).astype(np.int64), ref)
        # W -> -W negates every accumulator
        assert np.array_equal(oracle.matmul_i32(q, -wq), -oracle.matmul_i32(q, wq))


def test_matmul_structured_weights():
    M, N, K = 3, 256, 256
    q, _ = _rand_case(M, N, K, 5)
    ones = np.ones((N, K), np.int8)
    acc = oracle.matmul_i32(q, ones)
    assert np.array_equal(acc, np.repeat(q.astype(np.int32).sum(axis=1, keepdims=True), N, axis=1))
    eye = np.eye(N, K, dtype=np.int8)
    assert np.array_equal(oracle.matmul_i32(q, eye), q.astype(np.int32))
    # a transposed operand or a swapped index would break this asymmetric one-hot sweep
    for (n, k) in ((0, 0), (5, 200), (255, 1), (100, 101)):
        w = np.zeros((N, K), np.int8)
        w[n, k] = -1
        acc = oracle.matmul_i32(q, w)
        expect = np.zeros((M, N), np.int32)
        expect[:, n] = -q[:, k].astype(np.int32)
        assert np.array_equal(acc, expect)
    # extreme magnitudes do not overflow: 127 * K
    big = oracle.matmul_i32(np.full((1, 6912), 127, np.int8), np.ones((16, 6912), np.int8))
    assert np.all(big == 127 * 6912)


def test_sampled_matmul_agrees_with_full():
    q, wq = _rand_case(5, 64, 512, 11)
    full = oracle.matmul_i32(q, wq)
    m_idx = np.array([0, 4, 2, 3], np.int32)
    n_idx = np.array([63, 0, 17, 40], np.int32)
    assert np.array_equal(oracle.matmul_i32_sampled(q, wq, m_idx, n_idx), full[m_idx, n_idx])


def test_forward_equals_fp64_product_of_dequantised_operands():
    # "Lossless" reading (Section 5.2): the integer path times the two scales equals the product of
    # the fake-quantised operands, here evaluated in fp64 by brute force.
    for (M, N, K, seed) in ((1, 16, 256, 1), (4, 64, 512, 2), (3, 128, 256, 3)):
        x = wl.activations_normal(M, K, seed)
        W = wl.latent_weights(N, K, seed + 50).numpy()
        wts = oracle.quantize_weights(W, wl.WEIGHT_EPS)
        out = oracle.bitlinear_forward(wl.bf16_bits(x), None, wl.RMS_EPS, wts["wq"], wts["s_w"])
        w_deq = wts["wq"].astype(np.float64) * float(wts["s_w"])
        x_deq = out["q"].astype(np.float64) * out["d"].astype(np.float64)[:, None]
        ref = x_deq @ w_deq.T
        y = out["y"].astype(np.float64)
        assert np.all(np.abs(y - ref) <= 1e-6 * np.abs(ref))
        assert np.all(y[out["acc"] == 0] == 0.0)
        # and the output tracks the unquantised layer as closely as ternary weights allow: for Gaussian W
        # corr(W, W_q) = 2*phi(z0)/sqrt(1-p0) with z0 = sqrt(2/pi)/2, p0 = P(W_q = 0)  ->  0.887
        xd = x.double().numpy()
        yn = xd / np.sqrt((xd * xd).mean(axis=1, keepdims=True) + wl.RMS_EPS)
        full = yn @ W.astype(np.float64).T
        corr = np.corrcoef(full.ravel(), y.ravel())[0, 1]
        z0 = 0.5 * math.sqrt(2.0 / math.pi)
        p0 = math.erf(z0 / math.sqrt(2.0))
        expect = 2.0 * math.exp(-0.5 * z0 * z0) / math.sqrt(2.0 * math.pi) / math.sqrt(1.0 - p0)
        assert abs(expect - 0.887) < 2e-3
        assert abs(corr - expect) < 0.06


def test_dequant_hand_case():
    acc = np.array([[3, -5, 0]], np.int32)
    y = oracle.dequant(acc, np.float32(0.5), np.array([0.25], np.float32))
    assert y.tolist() == [[0.375, -0.625, 0.0]]


def test_packed_artifact_roundtrip_at_layer_shape():
    W = wl.latent_weights(640, 2560, wl.seed_for(2, 1)).numpy()
    wts = oracle.quantize_weights(W, wl.WEIGHT_EPS)
    assert wts["packed"].size == 640 * 2560 // 4
    assert np.array_equal(oracle.unpack(wts["packed"], 640, 2560), wts["wq"])
    assert not wts["fragile"]


# ---- chained decode: the glue between BitLinears (squared ReLU, residual, attention stand-in) ----


def test_chain_glue_closed_forms():
    """With every weight matrix all zeros each BitLinear returns 0, so the chain must leave h unchanged (residual
    adds of zero); with gate weights that make g negative the squared-ReLU branch must contribute exactly nothing."""
    from oracle import chain as oc

    H, F, nq, nkv, hd = 256, 256, 2, 1, 128
    zero = lambda n, k: dict(wq=np.zeros((n, k), np.int8), s_w=np.float32(1e-5))
    layer = {"q": zero(H, H), "k": zero(nkv * hd, H), "v": zero(nkv * hd, H), "o": zero(H, H), "gate": zero(F, H),
             "up": zero(F, H), "down": zero(H, F)}
    h0 = wl.bf16_bits(wl.activations_normal(3, H, 321))
    out = oc.decode_chain(h0, [layer, layer], nq, nkv, hd, 1e-5)
    assert np.array_equal(out["h"], h0)
    assert np.all(out["k"] == 0)


def test_chain_attention_standin_and_relu2_by_hand():
    """One layer with identity-like ternary weights, checked against the formulas written out in numpy fp64 on the
    oracle's own integer stages: a = q + v[head // group], f = relu(g)^2 * u, both residuals."""
    from oracle import chain as oc

    H, F, nq, nkv, hd = 256, 256, 2, 1, 128
    rng = np.random.default_rng(7)
    mats = {}
    for name, (n, k) in {"q": (H, H), "k": (nkv * hd, H), "v": (nkv * hd, H), "o": (H, H), "gate": (F, H), "up": (F, H),
                         "down": (H, F)}.items():
        mats[name] = dict(wq=rng.integers(-1, 2, size=(n, k)).astype(np.int8), s_w=np.float32(0.02))
    h0 = wl.bf16_bits(wl.activations_normal(2, H, 654))
    out = oc.decode_chain(h0, [mats], nq, nkv, hd, 1e-5)

    def lin(bits, m):
        return oracle.bitlinear_forward(bits, None, 1e-5, m["wq"], m["s_w"])["y"].astype(np.float64)

    def bf(x64):  # fp64 values that are exactly representable in fp32 after one fp32 op are passed as float32
        return oracle.f32_to_bf16(x64.astype(np.float32))

    q, v = lin(h0, mats["q"]), lin(h0, mats["v"])
    a = np.concatenate([q[:, :hd] + v[:, :hd], q[:, hd:] + v[:, :hd]], axis=1)
    a_bits = bf(np.float32(q.astype(np.float32)[:, :]) * 0 + a.astype(np.float32))  # one fp32 rounding of the sum
    h1 = bf((oracle.bf16_to_f32(h0).astype(np.float64) + lin(a_bits, mats["o"])).astype(np.float32))
    g, u = lin(h1, mats["gate"]).astype(np.float32), lin(h1, mats["up"]).astype(np.float32)
    r = np.maximum(g, 0)
    f_bits = bf(((r * r).astype(np.float32) * u).astype(np.float32))
    h2 = bf((oracle.bf16_to_f32(h1).astype(np.float64) + lin(f_bits, mats["down"])).astype(np.float32))
    assert np.array_equal(out["h"], h2)


# --------------------------------------------------------------------------- glue fused into the quantiser


def test_glue_functions_by_hand():
    bf = lambda a: oracle.bf16_to_f32(a)  # noqa: E731
    # squared ReLU gate: negative gates give 0 whatever `up` is; bf16 keeps 8 significant bits
    f = bf(oracle.glue_relu2(np.array([[-1.0, 2.0, 0.5, 3.0, 1.5]], np.float32), np.array([[5.0, 0.25, -4.0, 1.0, 1.0078125]], np.float32)))
    #  r*r = 0, 4, 0.25, 9, 2.25 ; times up = 0, 1, -1, 9, 2.267578125 -> bf16: 2.265625 (2.2676 lies between 2.265625 and 2.28125)
    assert f.tolist() == [[0.0, 1.0, -1.0, 9.0, 2.265625]]
    # residual: exact tie 1 + 2^-8 rounds to even (1.0); 1 + 3 * 2^-8 rounds up to 1 + 2^-6
    h = oracle.f32_to_bf16(np.array([[1.0, 1.0, -2.0]], np.float32))
    out = bf(oracle.glue_residual(h, np.array([[2.0 ** -8, 3 * 2.0 ** -8, 0.5]], np.float32)))
    assert out.tolist() == [[1.0, 1.015625, -1.5]]
    # stand-in: 4 query heads on 2 KV heads of width 2: heads 0,1 read KV head 0, heads 2,3 read KV head 1
    q = np.arange(8, dtype=np.float32).reshape(1, 8)
    v = np.array([[100.0, 200.0, 300.0, 400.0]], np.float32)
    a = bf(oracle.glue_attn_standin(q, v, 4, 2, 2))
    # 405 and 407 need nine significant bits: both are ties and round to the even neighbour (404, 408)
    assert a.tolist() == [[100.0, 201.0, 102.0, 203.0, 304.0, 404.0, 306.0, 408.0]]


def test_fused_glue_quantisers_are_glue_then_quantiser():
    rng = np.random.default_rng(12)
    M, F = 3, 512
    gate = rng.standard_normal((M, F)).astype(np.float32)
    up = rng.standard_normal((M, F)).astype(np.float32)
    gain = oracle.f32_to_bf16((1 + 0.25 * rng.standard_normal(F)).astype(np.float32))
    out = oracle.relu2_rmsnorm_quant(gate, up, gain, 1e-5)
    # closed form of the quantiser on a row whose gates are all negative: x = 0, codes 0, scale floor 1e-5 / 127
    z = oracle.relu2_rmsnorm_quant(-np.abs(gate), up, gain, 1e-5)
    assert not z["q"].any() and np.all(z["d"] == np.float32(1e-5) / np.float32(127.0)) and not oracle.bf16_to_f32(z["x"]).any()  # +0 or -0 (0 * negative)
    # about half of the gates are negative, so about half of the inputs of the quantiser are exactly zero
    assert 0.4 < (oracle.bf16_to_f32(out["x"]) == 0).mean() < 0.6
    # every non-zero row reaches +-127 and the norm is applied to the bf16-rounded product (textbook fp64 check)
    assert np.all(np.abs(out["q"]).max(axis=1) == 127)
    x = oracle.bf16_to_f32(out["x"]).astype(np.float64)
    g64 = oracle.bf16_to_f32(gain).astype(np.float64)
    yn = x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-5) * g64
    a = np.abs(yn).max(axis=1, keepdims=True)
    assert np.abs(out["q"] - yn * 127.0 / a).max() <= 0.5 + 1e-3
    # residual and stand-in variants: x is the glue result, the rest the plain quantiser of that x
    h = oracle.f32_to_bf16(rng.standard_normal((M, F)).astype(np.float32))
    res = oracle.residual_rmsnorm_quant(h, up, None, 1e-5)
    ref = oracle.rmsnorm_quant(oracle.glue_residual(h, up), None, 1e-5)
    assert np.array_equal(res["q"], ref["q"]) and np.array_equal(res["d"], ref["d"])
    assert np.array_equal(oracle.bf16_to_f32(res["x"]), oracle.bf16_to_f32(oracle.f32_to_bf16((oracle.bf16_to_f32(h) + up).astype(np.float32))))


# --------------------------------------------------------------------------- the rest of a decode step


def test_rope_pins():
    from oracle import decode_step as ds
    rng = np.random.default_rng(21)
    hd, nh = 8, 3
    x = rng.standard_normal((4, nh * hd))
    pos = np.array([0, 1, 7, 1000])
    y = ds.rope(x, pos, nh, hd, base=10000.0)
    assert np.array_equal(y[0], x[0])  # position 0 is the identity
    # a rotation: the norm of every pair (i, i + hd/2), hence of every head, is kept
    assert np.allclose((y.reshape(4, nh, hd) ** 2).sum(-1), (x.reshape(4, nh, hd) ** 2).sum(-1), rtol=1e-12)
    # hand case: head_dim 2 has one pair and angle = pos (frequency base^0 = 1): (1, 0) at pos = pi/2 -> (0, 1)
    y2 = ds.rope(np.array([[1.0, 0.0]]), np.array([np.pi / 2]), 1, 2, base=10000.0)
    assert np.allclose(y2, [[0.0, 1.0]], atol=1e-15)
    # head_dim 4, base 100: frequencies 1 and 100^(-1/2) = 0.1; pairs (0,2) and (1,3)
    y4 = ds.rope(np.array([[1.0, 1.0, 0.0, 0.0]]), np.array([2.0]), 1, 4, base=100.0)
    assert np.allclose(y4, [[np.cos(2.0), np.cos(0.2), np.sin(2.0), np.sin(0.2)]], atol=1e-15)
    # the reason for the scheme: the product of a rotated query and a rotated key depends on the distance only
    q, k = rng.standard_normal((1, hd)), rng.standard_normal((1, hd))
    d1 = ds.rope(q, [5], 1, hd) @ ds.rope(k, [3], 1, hd).T
    d2 = ds.rope(q, [105], 1, hd) @ ds.rope(k, [103], 1, hd).T
    assert np.allclose(d1, d2, rtol=1e-9)


def test_attention_decode_pins():
    from oracle import decode_step as ds
    rng = np.random.default_rng(22)
    n_q, n_kv, hd, T = 4, 2, 8, 6
    f = lambda a: oracle.f32_to_bf16(np.asarray(a, np.float32))  # noqa: E731
    k = rng.standard_normal((T, n_kv * hd)).astype(np.float32)
    v = rng.standard_normal((T, n_kv * hd)).astype(np.float32)
    vb = oracle.bf16_to_f32(f(v)).astype(np.float64).reshape(T, n_kv, hd)
    # a zero query scores every position alike: the output is the mean of the first `length` values of the KV head
    out = ds.attention_decode(f(np.zeros(n_q * hd)), f(k), f(v), 5, n_q, n_kv, hd).reshape(n_q, hd)
    for h in range(n_q):
        assert np.allclose(out[h], vb[:5, h // 2].mean(axis=0), rtol=1e-12)
    # length 1: the output is the first value row, whatever the query
    out = ds.attention_decode(f(rng.standard_normal(n_q * hd)), f(k), f(v), 1, n_q, n_kv, hd).reshape(n_q, hd)
    assert np.allclose(out[3], vb[0, 1]) and np.allclose(out[0], vb[0, 0])
    # a query 64 times a key direction makes that position win: keys are unit vectors e_t, query = 64 e_2 for head 0
    kk = np.zeros((T, n_kv * hd), np.float32)
    for t in range(T):
        kk[t, t] = 1.0       # KV head 0
        kk[t, hd + t] = 1.0  # KV head 1
    q = np.zeros(n_q * hd, np.float32)
    q[2] = 64.0              # query head 0 -> KV head 0, position 2
    q[3 * hd + 4] = 64.0     # query head 3 -> KV head 1, position 4
    out = ds.attention_decode(f(q), f(kk), f(v), T, n_q, n_kv, hd).reshape(n_q, hd)
    w = np.exp(64.0 / np.sqrt(hd))  # weight of the winner against weight 1 of the five others
    assert np.allclose(out[0], (w * vb[2, 0] + (vb[:, 0].sum(0) - vb[2, 0])) / (w + 5), rtol=1e-12)
    assert np.allclose(out[3], (w * vb[4, 1] + (vb[:, 1].sum(0) - vb[4, 1])) / (w + 5), rtol=1e-12)
    # heads 1 and 2 have a zero query: plain means
    assert np.allclose(out[1], vb[:, 0].mean(0)) and np.allclose(out[2], vb[:, 1].mean(0))


def test_lm_head_and_embedding_pins():
    from oracle import decode_step as ds
    rng = np.random.default_rng(23)
    V, K = 40, 16
    table = oracle.f32_to_bf16(rng.standard_normal((V, K)).astype(np.float32))
    ids = np.array([3, 39, 0, 3])
    rows = ds.embed(ids, table)
    assert np.array_equal(rows, table[[3, 39, 0, 3]])
    # logits of a one-hot input are a column of the table; of an embedding row, its products with every row
    onehot = np.zeros((1, K), np.float32)
    onehot[0, 5] = 2.0
    logits = ds.lm_head(oracle.f32_to_bf16(onehot), table)
    assert np.array_equal(logits[0], 2.0 * oracle.bf16_to_f32(table)[:, 5].astype(np.float64))
    e = oracle.bf16_to_f32(table).astype(np.float64)
    assert np.allclose(ds.lm_head(rows, table), e[[3, 39, 0, 3]] @ e.T, rtol=1e-14)
