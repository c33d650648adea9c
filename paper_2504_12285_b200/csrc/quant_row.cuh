// Fused RMSNorm + per-token absmax int8 activation quantiser for one row, shared by the stand-alone
// kernel and the batched decode pre-pass.
// (Paper Section 2: subln normalisation in front of BitLinear; 8-bit absmax quantisation per token.)
//
// The bf16 row is read once with 128-bit loads and kept in registers; the sum of squares is reduced
// in fp64 (warp shuffles, then a fixed-order sum over warps), the maximum of the normalised row in
// fp32; the second pass quantises from registers and writes 8 codes per store.
#pragma once

#include "common.cuh"

namespace bitlinear {

constexpr int kQuantThreads = 256;
constexpr int kQuantWarps = kQuantThreads / 32;

template <int WARPS>
struct RowReduceSmemT {
    double sq[WARPS];
    float r;
    float mx[WARPS];
    int sum[WARPS];
};
using RowReduceSmem = RowReduceSmemT<kQuantWarps>;

__device__ __forceinline__ void unpack_bf16x8(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        f[2 * e] = __uint_as_float(w[e] << 16);
        f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
}

// Round-half-even of a float with |v| < 2^22 to an integer whose low byte is the int8 code: adding 1.5 * 2^23 leaves
// the rounded integer in the low mantissa bits (one full-rate add instead of a conversion).  |v| <= 127 * (1 + 2^-24)
// by construction of the absmax scale, so the clip to [-128, 127] of the definition is the identity and is not coded.
__device__ __forceinline__ uint32_t round_code(float v) { return __float_as_uint(__fadd_rn(v, 12582912.0f)); }

// Packs the low bytes of four round_code results into one word and adds their (signed) sum to csum.
__device__ __forceinline__ uint32_t pack_codes4(uint32_t a, uint32_t b, uint32_t c, uint32_t d, int& csum) {
    const uint32_t w = __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
    asm("dp4a.s32.s32 %0, %1, %2, %0;" : "+r"(csum) : "r"(w), "r"(0x01010101));
    return w;
}

// Sum of the squares of up to eight bf16 values (given widened to fp32) as an fp64 number.  fp64 arithmetic is slow
// on this GPU (measured: sixteen fp64 multiply-adds per thread cost a 512-thread CTA about 3 us), so the exact squares
// (8-bit significands: each is exact in fp32) are added with an error-free fp32 two-sum chain whose residue is kept,
// and only two conversions and one fp64 add are spent per eight elements.  The result differs from the correctly
// rounded sum by less than 2^-42 relative - far inside the band in which the oracle flags a row as fragile.
__device__ __forceinline__ double sum_squares8(const float (&f)[8]) {
    float hi = __fmul_rn(f[0], f[0]), lo = 0.0f;
#pragma unroll
    for (int e = 1; e < 8; ++e) {
        const float p = __fmul_rn(f[e], f[e]);
        const float s = __fadd_rn(hi, p);
        const float bb = __fsub_rn(s, hi);
        lo = __fadd_rn(lo, __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(p, bb)));
        hi = s;
    }
    return (double)hi + (double)lo;
}

// ---- where a row comes from -------------------------------------------------------------------------------------
// The quantisers read their input through a source object: load(v) returns 16-byte vector v of the row as eight bf16
// bit patterns, store(v, bits) is called once per vector for sources that also have to write the row they produce.
// Besides a plain bf16 row, a source can apply the element-wise step that sits in front of a BitLinear in a decoder
// layer (paper Section 2: squared-ReLU feed-forward block, residual connections), so that the step costs no launch of
// its own: one fp32 operation per arithmetic step, then one round-to-nearest-even cast to bf16, exactly as the
// stand-alone glue kernels do.
__device__ __forceinline__ uint32_t bf16x2_rn(float lo, float hi) {
    const __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&pk);
}

struct RowBf16 {
    const uint4* x;
    __device__ __forceinline__ uint4 load(int v) const { return x[v]; }
    __device__ __forceinline__ void store(int, const uint4&) const {}
};

// x = bf16( fl32( fl32(r * r) * up ) ), r = max(gate, 0)
struct RowRelu2 {
    const float4* gate;
    const float4* up;
    uint4* out;  // nullable
    __device__ __forceinline__ uint4 load(int v) const {
        const float4 g0 = gate[2 * v], g1 = gate[2 * v + 1], u0 = up[2 * v], u1 = up[2 * v + 1];
        const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const float u[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float r = fmaxf(g[e], 0.0f);
            f[e] = __fmul_rn(__fmul_rn(r, r), u[e]);
        }
        return make_uint4(bf16x2_rn(f[0], f[1]), bf16x2_rn(f[2], f[3]), bf16x2_rn(f[4], f[5]), bf16x2_rn(f[6], f[7]));
    }
    __device__ __forceinline__ void store(int v, const uint4& b) const {
        if (out != nullptr) out[v] = b;
    }
};

// x = bf16( fl32( float(h) + y ) ); the new hidden state goes to `out` (which must not be `h`: some quantisers read a
// row three times)
struct RowResidual {
    const uint4* h;
    const float4* y;
    uint4* out;
    __device__ __forceinline__ uint4 load(int v) const {
        const uint4 hb = h[v];
        const float4 y0 = y[2 * v], y1 = y[2 * v + 1];
        const uint32_t w[4] = {hb.x, hb.y, hb.z, hb.w};
        const float yy[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
        uint32_t r[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            r[e] = bf16x2_rn(__fadd_rn(__uint_as_float(w[e] << 16), yy[2 * e]),
                             __fadd_rn(__uint_as_float(w[e] & 0xffff0000u), yy[2 * e + 1]));
        return make_uint4(r[0], r[1], r[2], r[3]);
    }
    __device__ __forceinline__ void store(int v, const uint4& b) const {
        if (out != nullptr) out[v] = b;
    }
};

// Stand-in for attention (not a BitLinear): x[h * D + j] = bf16( fl32( q[h * D + j] + v[(h / group) * D + j] ) );
// D a multiple of 8, so the eight elements of a vector lie inside one head.
struct RowStandin {
    const float* q;
    const float* v;
    uint4* out;  // nullable
    int head_dim, group;
    __device__ __forceinline__ uint4 load(int vec) const {
        const int c = 8 * vec, head = c / head_dim, j = c - head * head_dim;
        const float4* qp = reinterpret_cast<const float4*>(q + c);
        const float4* vp = reinterpret_cast<const float4*>(v + (head / group) * head_dim + j);
        const float4 q0 = qp[0], q1 = qp[1], v0 = vp[0], v1 = vp[1];
        return make_uint4(bf16x2_rn(__fadd_rn(q0.x, v0.x), __fadd_rn(q0.y, v0.y)), bf16x2_rn(__fadd_rn(q0.z, v0.z), __fadd_rn(q0.w, v0.w)),
                          bf16x2_rn(__fadd_rn(q1.x, v1.x), __fadd_rn(q1.y, v1.y)), bf16x2_rn(__fadd_rn(q1.z, v1.z), __fadd_rn(q1.w, v1.w)));
    }
    __device__ __forceinline__ void store(int vec, const uint4& b) const {
        if (out != nullptr) out[vec] = b;
    }
};

// The element-wise step in front of a problem's quantiser, as the batch descriptors carry it.
struct RowOp {
    const void* x2;  // second operand (up / y / v), fp32
    void* x_out;     // bf16 [M][K] result of the step, nullable except for the residual step
    int op;          // BITLINEAR_X_*
    int arg0, arg1;  // attention stand-in: head_dim, query heads per KV head
    int pad;
};

// Calls f(source) with the source of row m of a problem whose first operand is x ([M][K]; bf16 or fp32 as the step says).
template <class F>
__device__ __forceinline__ void with_row_source(const RowOp& o, const void* x, int m, int K, F&& f) {
    const size_t off = (size_t)m * K;
    if (o.op == BITLINEAR_X_RELU2) {
        f(RowRelu2{reinterpret_cast<const float4*>(static_cast<const float*>(x) + off),
                   reinterpret_cast<const float4*>(static_cast<const float*>(o.x2) + off),
                   o.x_out ? reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.x_out) + off) : nullptr});
    } else if (o.op == BITLINEAR_X_RESIDUAL) {
        f(RowResidual{reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(x) + off),
                      reinterpret_cast<const float4*>(static_cast<const float*>(o.x2) + off),
                      o.x_out ? reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.x_out) + off) : nullptr});
    } else if (o.op == BITLINEAR_X_ATTN_STANDIN) {
        f(RowStandin{static_cast<const float*>(x) + off, static_cast<const float*>(o.x2) + (size_t)m * (K / o.arg1),
                     o.x_out ? reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.x_out) + off) : nullptr, o.arg0, o.arg1});
    } else {
        f(RowBf16{reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(x) + off)});
    }
}

// Quantises one row with the kQuantThreads threads of the calling CTA (all must call it).
// LAYOUT 0: codes are stored in column order.
// LAYOUT 1: inside every block of 256 columns the sixteen 16-byte pieces are stored transposed (piece 4t+q,
//           columns 64t+16q .. +15, at byte 64q+16t), the order in which the four column lanes of the batched
//           decode kernel read them.
// LAYOUT 2: tensor-core tile images: xq_row points at this row inside the first 128-row x 128-column tile of its
//           row tile (tiles of 16 KiB follow each other along K); 16-byte piece p of a row sits at (p ^ swz) * 16,
//           swz = row & 7 - the 128-byte shared-memory swizzle.
// LAYOUT 3: the same with tiles of 16 rows x 128 columns (2 KiB): the token-side operand of the decode kernel that
//           runs on the tensor cores with the tokens as the narrow dimension.
// THREADS = threads of the CTA (all of them take part; the block-wide barriers are __syncthreads).
template <int VPT, int LAYOUT = 0, class Src = RowBf16, int THREADS = kQuantThreads>  // VPT = 16-byte vectors (8 bf16) per thread
__device__ __forceinline__ void quant_row_src(const Src src, const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                              int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                              int32_t* __restrict__ xsum_out, RowReduceSmemT<THREADS / 32>& sm, int swz = 0) {
    const int n_vec = K >> 3;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint4* grow = reinterpret_cast<const uint4*>(gain);

    uint4 xv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * THREADS;
        xv[i] = make_uint4(0, 0, 0, 0);
        if (v < n_vec) {
            xv[i] = src.load(v);
            src.store(v, xv[i]);
        }
    }

    // ---- sum of squares in fp64 (each square of a bf16 value is exact) ----
    double sq = 0.0;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        float f[8];
        unpack_bf16x8(xv[i], f);
        sq += sum_squares8(f);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) sm.sq[warp] = sq;
    __syncthreads();
    if (tid == 0) {  // one thread does the fp64 divide and square root
        double S = 0.0;
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) S += sm.sq[w];
        sm.r = (float)(1.0 / sqrt(S / (double)K + (double)eps));
    }
    __syncthreads();
    const float r = sm.r;

    // ---- normalise (kept in registers) and find the absolute maximum ----
    float y[VPT][8];
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * THREADS;
        float f[8], g[8];
        unpack_bf16x8(xv[i], f);
        if (gain != nullptr && v < n_vec) {
            unpack_bf16x8(grow[v], g);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 1.0f;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            y[i][e] = __fmul_rn(__fmul_rn(f[e], r), g[e]);
            amax = fmaxf(amax, fabsf(y[i][e]));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) sm.mx[warp] = amax;
    __syncthreads();
    float a = 0.0f;
#pragma unroll
    for (int w = 0; w < THREADS / 32; ++w) a = fmaxf(a, sm.mx[w]);
    a = fmaxf(a, 1e-5f);
    const float s = __fdiv_rn(127.0f, a);

    // ---- quantise from registers ----
    int csum = 0;
    uint2* qrow = reinterpret_cast<uint2*>(xq_row);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * THREADS;
        uint32_t c[8], packed[2];
#pragma unroll
        for (int e = 0; e < 8; ++e) c[e] = round_code(__fmul_rn(y[i][e], s));
        packed[0] = pack_codes4(c[0], c[1], c[2], c[3], csum);
        packed[1] = pack_codes4(c[4], c[5], c[6], c[7], csum);
        int dst = v;  // in units of 8 codes
        if (LAYOUT == 1) {
            const int piece = (v >> 1) & 15;  // 16-byte piece inside the 256-column block: 4t + q
            dst = (v & ~31) | ((((piece & 3) << 2) | (piece >> 2)) << 1) | (v & 1);
        } else if (LAYOUT == 2 || LAYOUT == 3) {
            const int kb = v >> 4, piece = (v >> 1) & 7;  // 128-column tile along K, 16-byte piece in the row
            dst = kb * ((LAYOUT == 2 ? 128 : 16) * 128 / 8) + (((piece ^ swz) << 1) | (v & 1));
        }
        if (v < n_vec) qrow[dst] = make_uint2(packed[0], packed[1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
    if (lane == 0) sm.sum[warp] = csum;
    __syncthreads();
    if (tid == 0) {
        int total = 0;
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) total += sm.sum[w];
        *d_out = __fdiv_rn(a, 127.0f);
        if (xsum_out != nullptr) *xsum_out = total;
    }
}


template <int VPT, int LAYOUT = 0>
__device__ __forceinline__ void quant_row(const __nv_bfloat16* __restrict__ x_row,
                                          const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                          int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                          int32_t* __restrict__ xsum_out, RowReduceSmem& sm, int swz = 0) {
    quant_row_src<VPT, LAYOUT>(RowBf16{reinterpret_cast<const uint4*>(x_row)}, gain, eps, K, xq_row, d_out, xsum_out, sm, swz);
}

// Warp-per-row variant for many-token calls: the same arithmetic with one warp owning a whole row (16-byte
// vector v of the row belongs to lane v % 32), so a CTA of kQuantThreads threads quantises eight rows with no
// block-wide barrier.  The row is read from HBM once; the second and third pass read it again (it is still in
// L1 / L2), which keeps the register count low and no shared memory is needed, so many rows are in flight per SM.
template <int LAYOUT = 0, class Src = RowBf16>
__device__ __forceinline__ void quant_row_warp_src(const Src src, const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                                   int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                                   int32_t* __restrict__ xsum_out, int swz = 0) {
    const int n_vec = K >> 3;
    const int lane = threadIdx.x & 31;
    const uint4* grow = reinterpret_cast<const uint4*>(gain);
    double sq = 0.0;
#pragma unroll 4
    for (int v = lane; v < n_vec; v += 32) {
        const uint4 u = src.load(v);
        src.store(v, u);
        float f[8];
        unpack_bf16x8(u, f);
        sq += sum_squares8(f);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    float r = 0.0f;
    if (lane == 0) r = (float)(1.0 / sqrt(sq / (double)K + (double)eps));  // one lane does the fp64 divide and root
    r = __shfl_sync(0xffffffffu, r, 0);

    float amax = 0.0f;
#pragma unroll 2
    for (int v = lane; v < n_vec; v += 32) {
        float f[8], g[8];
        unpack_bf16x8(src.load(v), f);
        if (gain != nullptr) {
            unpack_bf16x8(grow[v], g);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 1.0f;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(__fmul_rn(__fmul_rn(f[e], r), g[e])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float a = fmaxf(amax, 1e-5f);
    const float s = __fdiv_rn(127.0f, a);

    int csum = 0;
    uint2* qrow = reinterpret_cast<uint2*>(xq_row);
#pragma unroll 2
    for (int v = lane; v < n_vec; v += 32) {
        float f[8], g[8];
        unpack_bf16x8(src.load(v), f);
        if (gain != nullptr) {
            unpack_bf16x8(grow[v], g);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 1.0f;
        }
        uint32_t c[8], packed[2];
#pragma unroll
        for (int e = 0; e < 8; ++e) c[e] = round_code(__fmul_rn(__fmul_rn(__fmul_rn(f[e], r), g[e]), s));
        packed[0] = pack_codes4(c[0], c[1], c[2], c[3], csum);
        packed[1] = pack_codes4(c[4], c[5], c[6], c[7], csum);
        int dst = v;  // in units of 8 codes
        if (LAYOUT == 1) {
            const int piece = (v >> 1) & 15;
            dst = (v & ~31) | ((((piece & 3) << 2) | (piece >> 2)) << 1) | (v & 1);
        } else if (LAYOUT == 2 || LAYOUT == 3) {
            const int kb = v >> 4, piece = (v >> 1) & 7;
            dst = kb * ((LAYOUT == 2 ? 128 : 16) * 128 / 8) + (((piece ^ swz) << 1) | (v & 1));
        }
        qrow[dst] = make_uint2(packed[0], packed[1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
    if (lane == 0) {
        *d_out = __fdiv_rn(a, 127.0f);
        if (xsum_out != nullptr) *xsum_out = csum;
    }
}

template <int LAYOUT = 0>
__device__ __forceinline__ void quant_row_warp(const __nv_bfloat16* __restrict__ x_row,
                                               const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                               int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                               int32_t* __restrict__ xsum_out, int swz = 0) {
    quant_row_warp_src<LAYOUT>(RowBf16{reinterpret_cast<const uint4*>(x_row)}, gain, eps, K, xq_row, d_out, xsum_out, swz);
}

// WARPS warps per row (WARPS = 2 or 4; the group's threads are 32 * WARPS consecutive threads of the CTA): for calls
// with few rows, where one warp per row leaves the GPU mostly idle and a long row is a long serial chain for its warp.
// Same arithmetic and the same three passes as quant_row_warp; the partial results of the warps meet in shared memory
// behind a named barrier of the group (bar_id, 1 .. 15, one per group of the CTA).
struct GroupReduceSmem {
    double sq[4];
    float mx[4];
    int sum[4];
    float r;
};

template <int LAYOUT, int WARPS, class Src = RowBf16>
__device__ __forceinline__ void quant_row_group_src(const Src src, const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                                    int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                                    int32_t* __restrict__ xsum_out, GroupReduceSmem& sm, int bar_id, int swz = 0) {
    constexpr int T = 32 * WARPS;
    const int n_vec = K >> 3;
    const int gt = threadIdx.x % T, w = gt >> 5, lane = gt & 31;
    const uint4* grow = reinterpret_cast<const uint4*>(gain);
    auto group_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(T) : "memory"); };
    double sq = 0.0;
#pragma unroll 4
    for (int v = gt; v < n_vec; v += T) {
        float f[8];
        const uint4 u = src.load(v);
        src.store(v, u);
        unpack_bf16x8(u, f);
        sq += sum_squares8(f);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) sm.sq[w] = sq;
    group_sync();
    if (gt == 0) {
        double S = 0.0;
#pragma unroll
        for (int i = 0; i < WARPS; ++i) S += sm.sq[i];
        sm.r = (float)(1.0 / sqrt(S / (double)K + (double)eps));  // one thread does the fp64 divide and root
    }
    group_sync();
    const float r = sm.r;

    float amax = 0.0f;
#pragma unroll 2
    for (int v = gt; v < n_vec; v += T) {
        float f[8], g[8];
        unpack_bf16x8(src.load(v), f);
        if (gain != nullptr) {
            unpack_bf16x8(grow[v], g);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 1.0f;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(__fmul_rn(__fmul_rn(f[e], r), g[e])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) sm.mx[w] = amax;
    group_sync();
    float a = 1e-5f;
#pragma unroll
    for (int i = 0; i < WARPS; ++i) a = fmaxf(a, sm.mx[i]);
    const float s = __fdiv_rn(127.0f, a);

    int csum = 0;
    uint2* qrow = reinterpret_cast<uint2*>(xq_row);
#pragma unroll 2
    for (int v = gt; v < n_vec; v += T) {
        float f[8], g[8];
        unpack_bf16x8(src.load(v), f);
        if (gain != nullptr) {
            unpack_bf16x8(grow[v], g);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 1.0f;
        }
        uint32_t c[8], packed[2];
#pragma unroll
        for (int e = 0; e < 8; ++e) c[e] = round_code(__fmul_rn(__fmul_rn(__fmul_rn(f[e], r), g[e]), s));
        packed[0] = pack_codes4(c[0], c[1], c[2], c[3], csum);
        packed[1] = pack_codes4(c[4], c[5], c[6], c[7], csum);
        int dst = v;  // in units of 8 codes
        if (LAYOUT == 1) {
            const int piece = (v >> 1) & 15;
            dst = (v & ~31) | ((((piece & 3) << 2) | (piece >> 2)) << 1) | (v & 1);
        } else if (LAYOUT == 2 || LAYOUT == 3) {
            const int kb = v >> 4, piece = (v >> 1) & 7;
            dst = kb * ((LAYOUT == 2 ? 128 : 16) * 128 / 8) + (((piece ^ swz) << 1) | (v & 1));
        }
        qrow[dst] = make_uint2(packed[0], packed[1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
    if (lane == 0) sm.sum[w] = csum;
    group_sync();
    if (gt == 0) {
        int total = 0;
#pragma unroll
        for (int i = 0; i < WARPS; ++i) total += sm.sum[i];
        *d_out = __fdiv_rn(a, 127.0f);
        if (xsum_out != nullptr) *xsum_out = total;
    }
}

template <int LAYOUT, int WARPS>
__device__ __forceinline__ void quant_row_group(const __nv_bfloat16* __restrict__ x_row,
                                                const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                                int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                                int32_t* __restrict__ xsum_out, GroupReduceSmem& sm, int bar_id, int swz = 0) {
    quant_row_group_src<LAYOUT, WARPS>(RowBf16{reinterpret_cast<const uint4*>(x_row)}, gain, eps, K, xq_row, d_out, xsum_out, sm,
                                       bar_id, swz);
}

}  // namespace bitlinear
