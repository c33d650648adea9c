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

struct RowReduceSmem {
    double sq[kQuantWarps];
    float mx[kQuantWarps];
    int sum[kQuantWarps];
};

__device__ __forceinline__ void unpack_bf16x8(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        f[2 * e] = __uint_as_float(w[e] << 16);
        f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
}

// Quantises one row with the kQuantThreads threads of the calling CTA (all must call it).
// PERM = false: codes are stored in column order.  PERM = true: inside every block of 256 columns the
// sixteen 16-byte pieces are stored transposed (piece 4t+q, columns 64t+16q .. +15, at byte 64q+16t), the
// order in which the four column lanes of the batched decode kernel read them.
template <int VPT, bool PERM = false>  // VPT = 16-byte vectors (8 bf16) per thread
__device__ __forceinline__ void quant_row(const __nv_bfloat16* __restrict__ x_row,
                                          const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                          int8_t* __restrict__ xq_row, float* __restrict__ d_out,
                                          int32_t* __restrict__ xsum_out, RowReduceSmem& sm) {
    const int n_vec = K >> 3;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint4* xrow = reinterpret_cast<const uint4*>(x_row);
    const uint4* grow = reinterpret_cast<const uint4*>(gain);

    uint4 xv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kQuantThreads;
        xv[i] = (v < n_vec) ? xrow[v] : make_uint4(0, 0, 0, 0);
    }

    // ---- sum of squares in fp64 (each square of a bf16 value is exact) ----
    double sq = 0.0;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        float f[8];
        unpack_bf16x8(xv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const double v = (double)f[e];
            sq += v * v;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) sm.sq[warp] = sq;
    __syncthreads();
    double S = 0.0;
#pragma unroll
    for (int w = 0; w < kQuantWarps; ++w) S += sm.sq[w];
    const float r = (float)(1.0 / sqrt(S / (double)K + (double)eps));

    // ---- normalise (kept in registers) and find the absolute maximum ----
    float y[VPT][8];
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kQuantThreads;
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
    for (int w = 0; w < kQuantWarps; ++w) a = fmaxf(a, sm.mx[w]);
    a = fmaxf(a, 1e-5f);
    const float s = __fdiv_rn(127.0f, a);

    // ---- quantise from registers ----
    int csum = 0;
    uint2* qrow = reinterpret_cast<uint2*>(xq_row);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kQuantThreads;
        uint32_t packed[2] = {0u, 0u};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int q = __float2int_rn(__fmul_rn(y[i][e], s));
            q = max(-128, min(127, q));
            csum += q;
            packed[e >> 2] |= (uint32_t)(q & 0xff) << (8 * (e & 3));
        }
        int dst = v;  // in units of 8 codes
        if (PERM) {
            const int piece = (v >> 1) & 15;  // 16-byte piece inside the 256-column block: 4t + q
            dst = (v & ~31) | ((((piece & 3) << 2) | (piece >> 2)) << 1) | (v & 1);
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
        for (int w = 0; w < kQuantWarps; ++w) total += sm.sum[w];
        *d_out = __fdiv_rn(a, 127.0f);
        if (xsum_out != nullptr) *xsum_out = total;
    }
}


}  // namespace bitlinear
