/*
 * CPU oracle for the W1.58A8 BitLinear forward of BitNet b1.58 (Section 2 of the
 * paper: absmean ternary weights, per-token absmax int8 activations, subln
 * normalisation, no bias; Section 5.1: four ternary values per stored byte).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step definition of
 * what the path computes, used only by the tests, the smoke check and the
 * benchmark's CPU-baseline leg.  The product (the CUDA library) never calls it
 * and shares no code, header, table or helper with it.
 *
 * Every fp32 operation below is a single IEEE-754 round-to-nearest-even
 * operation (build with -ffp-contract=off, no fast-math); "Round" is
 * round-half-to-even (rintf under the default rounding mode).
 *
 * The steps, in the order the layer applies them:
 *   1. x (bf16) and gain g (bf16) are widened to fp32 exactly.
 *   2. RMSNorm (the subln normalisation in front of every BitLinear):
 *        r = fl32( 1 / sqrt( mean(x^2) + eps ) ),   y_i = fl32( fl32(x_i * r) * g_i )
 *      mean(x^2) is taken from an extended-precision sum of the exact squares.
 *   3. a = max_i |y_i|, clamped below by 1e-5 so that an all-zero token is safe.
 *   4. Activation quantiser: s = fl32(127 / a);
 *        q_i = clip( Round( fl32(y_i * s) ), -128, 127 );   d = fl32(a / 127).
 *   5. Weight scale: beta = fl32( mean |W| ) over the whole matrix; s_w = fl32(beta + eps_w).
 *   6. Weight quantiser: W_q = clip( Round( fl32(W / s_w) ), -1, 1 ).
 *   7. Packing: four ternary codes per byte in the tiled order documented at
 *      oracle_pack_index() below; or (7b) five per byte, see oracle_pack5_index().
 *   8. Contraction: acc[m][n] = sum_k q[m][k] * W_q[n][k] in int32.
 *   9. Dequantising epilogue: y[m][n] = fl32( fl32( (float)acc * s_w ) * d[m] ).
 *
 * Parity pins (see tests/test_oracle_pins.py): hand-computed rounding, tie and
 * clip cases; range invariants; the Gaussian closed form for the share of zero
 * weights; textbook RMSNorm in fp64; int64 library matmul; identity / one-hot /
 * all-ones weight patterns; fp64 brute force of the dequantised operands; for the
 * five-per-byte layout all 243 byte patterns against exact rational arithmetic,
 * hand-derived positions and byte values, sizes, round trips, identity weights.
 * Parity on the released model weights is unpinned: they are not available here.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- bf16 <-> fp32 ------------------------------------------------------- */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* Round-to-nearest-even narrowing of a finite fp32 value to bf16. */
static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
    uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
    return (uint16_t)upper;
}

void oracle_f32_to_bf16(const float *in, long n, uint16_t *out) {
    for (long i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(in[i]);
}

void oracle_bf16_to_f32(const uint16_t *in, long n, float *out) {
    for (long i = 0; i < n; ++i) out[i] = bf16_to_f32(in[i]);
}

/* ---- steps 3-4: absmax int8 quantiser of one already-normalised row ------- */

static void absmax_quant_row(const float *y, int K, int8_t *q, float *d, int32_t *xsum) {
    float a = 0.0f;
    for (int i = 0; i < K; ++i) {
        float v = fabsf(y[i]);
        if (v > a) a = v;
    }
    if (a < 1e-5f) a = 1e-5f;
    float s = 127.0f / a;
    int32_t sum = 0;
    for (int i = 0; i < K; ++i) {
        float v = y[i] * s;
        float r = rintf(v);
        if (r > 127.0f) r = 127.0f;
        if (r < -128.0f) r = -128.0f;
        q[i] = (int8_t)r;
        sum += (int32_t)q[i];
    }
    *d = a / 127.0f;
    if (xsum) *xsum = sum;
}

/* Steps 3-4 on M rows of fp32 values (no normalisation): used to pin the quantiser alone. */
void oracle_absmax_quant(const float *y, int M, int K, int8_t *q, float *d, int32_t *xsum) {
    for (int m = 0; m < M; ++m)
        absmax_quant_row(y + (long)m * K, K, q + (long)m * K, d + m, xsum ? xsum + m : 0);
}

/* ---- steps 1-4: fused RMSNorm + absmax int8 quantiser --------------------- */

static float rms_scale(long double S, int K, float eps) {
    double mean = (double)(S / (long double)K);
    return (float)(1.0 / sqrt(mean + (double)eps));
}

/*
 * x: [M][K] bf16 bit patterns; g: [K] bf16 bit patterns or NULL (all ones).
 * Outputs: q [M][K], d [M], xsum [M] (nullable), y_norm [M][K] fp32 (nullable: the
 * normalised row before quantisation), fragile [M] (nullable): 1 where the fp32
 * rounding of r would change if the sum of squares moved by max(K*2^-52, 2^-40)
 * relative, i.e. where another (equally valid) way of summing the exact squares -
 * another fp64 order, or partial sums carried as error-free pairs of fp32 - could
 * legitimately give another r.
 */
void oracle_rmsnorm_quant(const uint16_t *x, const uint16_t *g, float eps, int M, int K,
                          int8_t *q, float *d, int32_t *xsum, float *y_norm, int *fragile) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t *xr = x + (long)m * K;
        long double S = 0.0L;
        for (int i = 0; i < K; ++i) {
            double v = (double)bf16_to_f32(xr[i]);
            S += (long double)(v * v); /* the square of an 8-bit significand is exact in fp64 */
        }
        float r = rms_scale(S, K, eps);
        if (fragile) {
            long double rel = (long double)K * 2.220446049250313e-16L;
            if (rel < 9.094947017729282e-13L) rel = 9.094947017729282e-13L; /* 2^-40 */
            float r_lo = rms_scale(S * (1.0L - rel), K, eps);
            float r_hi = rms_scale(S * (1.0L + rel), K, eps);
            fragile[m] = (r_lo != r || r_hi != r) ? 1 : 0;
        }
        float *yrow = y_norm ? y_norm + (long)m * K : 0;
        /* two passes over the row: normalise (finding the max), then quantise */
        float a = 0.0f;
        for (int i = 0; i < K; ++i) {
            float xf = bf16_to_f32(xr[i]);
            float gf = g ? bf16_to_f32(g[i]) : 1.0f;
            float t = xf * r;
            float y = t * gf;
            if (yrow) yrow[i] = y;
            float v = fabsf(y);
            if (v > a) a = v;
        }
        if (a < 1e-5f) a = 1e-5f;
        float s = 127.0f / a;
        int32_t sum = 0;
        int8_t *qr = q + (long)m * K;
        for (int i = 0; i < K; ++i) {
            float xf = bf16_to_f32(xr[i]);
            float gf = g ? bf16_to_f32(g[i]) : 1.0f;
            float t = xf * r;
            float y = t * gf;
            float v = y * s;
            float rv = rintf(v);
            if (rv > 127.0f) rv = 127.0f;
            if (rv < -128.0f) rv = -128.0f;
            qr[i] = (int8_t)rv;
            sum += (int32_t)qr[i];
        }
        d[m] = a / 127.0f;
        if (xsum) xsum[m] = sum;
    }
}

/* ---- step 5: absmean weight scale ---------------------------------------- */

/*
 * W: count fp32 values (the whole [N][K] matrix).  s_w = fl32( fl32(mean|W|) + eps_w ).
 * fragile (nullable): 1 if beta's fp32 rounding changes when the sum moves by 1e-11 relative.
 */
void oracle_weight_scale(const float *W, long count, float eps_w, float *s_w, int *fragile) {
    long double B = 0.0L;
    for (long i = 0; i < count; ++i) B += (long double)fabs((double)W[i]);
    float beta = (float)(double)(B / (long double)count);
    if (fragile) {
        float lo = (float)(double)(B * (1.0L - 1e-11L) / (long double)count);
        float hi = (float)(double)(B * (1.0L + 1e-11L) / (long double)count);
        *fragile = (lo != beta || hi != beta) ? 1 : 0;
    }
    *s_w = beta + eps_w;
}

/* ---- step 6: ternary weight quantiser ------------------------------------ */

void oracle_weight_quant(const float *W, long count, float s_w, int8_t *wq) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < count; ++i) {
        float t = W[i] / s_w;
        float r = rintf(t);
        if (r > 1.0f) r = 1.0f;
        if (r < -1.0f) r = -1.0f;
        wq[i] = (int8_t)r;
    }
}

/* ---- step 7: the packed layout ------------------------------------------- */

/*
 * Four ternary values per byte (Section 5.1), stored as the 2-bit code c = W_q + 1
 * (0, 1 or 2; the value 3 never occurs).  N must be a multiple of 16 and K of 256.
 *
 * The matrix is cut into tiles of 16 rows x 256 columns; tiles are stored one after
 * another, row-block major (all column tiles of rows 0..15, then rows 16..31, ...),
 * 1024 bytes each.  Inside a tile, for row r = 8*h + g (h in 0..1, g in 0..7) and
 * column c = 64*t + 16*i + 4*j + b (t, i, j, b each in 0..3):
 *     byte offset in the tile = 512*h + 64*g + 16*t + 4*i + b
 *     bit position in the byte = 2*j   (bits 2j and 2j+1 hold the code)
 * So a 16-byte chunk is 64 consecutive columns of one row, a little-endian 32-bit
 * word is 16 consecutive columns, and (word >> 2j) & 0x03030303 is four consecutive
 * columns' codes, one per byte.
 */
static void oracle_pack_index(int n, int k, int K, long *byte_index, int *shift) {
    long tile = (long)(n / 16) * (K / 256) + (k / 256);
    int r = n % 16, h = r / 8, g = r % 8;
    int c = k % 256, t = c / 64, i = (c % 64) / 16, j = (c % 16) / 4, b = c % 4;
    *byte_index = tile * 1024 + 512 * h + 64 * g + 16 * t + 4 * i + b;
    *shift = 2 * j;
}

/* Returns 0 on success, -1 on an unsupported shape, -2 if a value is not in {-1,0,1}. */
int oracle_pack(const int8_t *wq, int N, int K, uint8_t *packed) {
    if (N <= 0 || K <= 0 || N % 16 || K % 256) return -1;
    memset(packed, 0, (size_t)N * (size_t)K / 4);
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            int w = wq[(long)n * K + k];
            if (w < -1 || w > 1) return -2;
            long bi;
            int sh;
            oracle_pack_index(n, k, K, &bi, &sh);
            packed[bi] |= (uint8_t)((w + 1) << sh);
        }
    return 0;
}

/* Returns 0 on success, -1 on an unsupported shape, -2 if the unused code 3 is met. */
int oracle_unpack(const uint8_t *packed, int N, int K, int8_t *wq) {
    if (N <= 0 || K <= 0 || N % 16 || K % 256) return -1;
    int bad = 0;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            long bi;
            int sh;
            oracle_pack_index(n, k, K, &bi, &sh);
            int c = (packed[bi] >> sh) & 3;
            if (c == 3) bad = 1;
            wq[(long)n * K + k] = (int8_t)(c - 1);
        }
    return bad ? -2 : 0;
}

/* ---- step 7b: the dense packed layout, five ternary values per byte -------- */

/*
 * 1.6 bits per weight: Table 1 of the paper counts the non-embedding memory of the 2B
 * model at about 1.58 bits per weight, and Section 5.1 packs weights to cut the bytes
 * that cross HBM; 3^5 = 243 <= 256, so five ternary values fit one byte.  The paper
 * gives no layout for this; the one below is this library's.
 *
 * Byte value.  With the codes c_e = W_q + 1 (0, 1 or 2) of five weights, digit 0 the
 * most significant, v = c_0*81 + c_1*27 + c_2*9 + c_3*3 + c_4 lies in [0, 242] and the
 * stored byte is B = ceil(256 * v / 243): the base-3 fraction 0.c_0 c_1 c_2 c_3 c_4
 * scaled to 8 bits and rounded up.  v is recovered as floor(243 * B / 256).  Thirteen
 * of the 256 byte values are never produced.
 *
 * Position.  K is padded with zero weights to Kp = 320 * ceil(K / 320).  The matrix is
 * cut into tiles of 16 rows x 320 columns, 1024 bytes each, stored row-block major:
 * tile = (n / 16) * (Kp / 320) + (k / 320).  Inside a tile, for row r = 8*h + g and
 * column c = 80*t + 20*i + 4*e + b  (t, i, b in 0..3, e in 0..4):
 *     byte offset in the tile = 512*h + 64*g + 16*t + 4*i + b,   base-3 digit e.
 * So a 16-byte chunk is 80 consecutive columns of one row, a 4-byte word is 20
 * consecutive columns, and digit e of the four bytes of a word is four consecutive
 * columns.  N must be a multiple of 16 and K of 256.
 */
long oracle_packed5_bytes(int N, int K) {
    if (N <= 0 || K <= 0 || N % 16 || K % 256) return 0;
    long kp = ((long)K + 319) / 320 * 320;
    return (long)N * kp / 5;
}

static void oracle_pack5_index(int n, int k, int K, long *byte_index, int *digit) {
    long tiles_per_block = ((long)K + 319) / 320;
    long tile = (long)(n / 16) * tiles_per_block + (k / 320);
    int r = n % 16, h = r / 8, g = r % 8;
    int c = k % 320, t = c / 80, i = (c % 80) / 20, e = (c % 20) / 4, b = c % 4;
    *byte_index = tile * 1024 + 512 * h + 64 * g + 16 * t + 4 * i + b;
    *digit = e;
}

static const int kPow3[5] = {81, 27, 9, 3, 1}; /* weight of digit e */

/* Returns 0 on success, -1 on an unsupported shape, -2 if a value is not in {-1,0,1}. */
int oracle_pack5(const int8_t *wq, int N, int K, uint8_t *packed) {
    long bytes = oracle_packed5_bytes(N, K);
    if (bytes == 0) return -1;
    /* v of every byte, starting from five zero weights (code 1 in every digit: 121) */
    int16_t *v = (int16_t *)malloc((size_t)bytes * sizeof(int16_t));
    if (!v) return -1;
    for (long i = 0; i < bytes; ++i) v[i] = 121;
    int rc = 0;
    for (int n = 0; n < N && rc == 0; ++n)
        for (int k = 0; k < K; ++k) {
            int w = wq[(long)n * K + k];
            if (w < -1 || w > 1) { rc = -2; break; }
            long bi;
            int e;
            oracle_pack5_index(n, k, K, &bi, &e);
            v[bi] = (int16_t)(v[bi] + w * kPow3[e]);
        }
    if (rc == 0)
        for (long i = 0; i < bytes; ++i) packed[i] = (uint8_t)((256 * (int)v[i] + 242) / 243);
    free(v);
    return rc;
}

/* Returns 0 on success, -1 on an unsupported shape, -2 if a byte value that no five codes produce is met.
 * Padding columns (k >= K) are not returned. */
int oracle_unpack5(const uint8_t *packed, int N, int K, int8_t *wq) {
    long bytes = oracle_packed5_bytes(N, K);
    if (bytes == 0) return -1;
    for (long i = 0; i < bytes; ++i) {
        int v = (243 * (int)packed[i]) / 256;
        if ((256 * v + 242) / 243 != (int)packed[i]) return -2;
    }
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            long bi;
            int e;
            oracle_pack5_index(n, k, K, &bi, &e);
            int v = (243 * (int)packed[bi]) / 256;
            wq[(long)n * K + k] = (int8_t)((v / kPow3[e]) % 3 - 1);
        }
    return 0;
}

/* ---- step 8: the contraction --------------------------------------------- */

void oracle_matmul_i32(const int8_t *q, const int8_t *wq, int M, int N, int K, int32_t *acc) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const int8_t *wr = wq + (long)n * K;
        for (int m = 0; m < M; ++m) {
            const int8_t *qr = q + (long)m * K;
            int32_t s = 0;
            for (int k = 0; k < K; ++k) s += (int32_t)qr[k] * (int32_t)wr[k];
            acc[(long)m * N + n] = s;
        }
    }
}

/* Selected outputs only: acc[i] for (m_idx[i], n_idx[i]); lets full-size cases be sampled. */
void oracle_matmul_i32_sampled(const int8_t *q, const int8_t *wq, int K, const int32_t *m_idx,
                               const int32_t *n_idx, long count, int32_t *acc) {
    for (long i = 0; i < count; ++i) {
        const int8_t *qr = q + (long)m_idx[i] * K;
        const int8_t *wr = wq + (long)n_idx[i] * K;
        int32_t s = 0;
        for (int k = 0; k < K; ++k) s += (int32_t)qr[k] * (int32_t)wr[k];
        acc[i] = s;
    }
}

/* ---- step 9: the dequantising epilogue ----------------------------------- */

void oracle_dequant(const int32_t *acc, float s_w, const float *d, int M, int N, float *y) {
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            float t = (float)acc[(long)m * N + n] * s_w;
            y[(long)m * N + n] = t * d[m];
        }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
