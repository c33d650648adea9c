// Fused RMSNorm + per-token absmax int8 activation quantiser.
// (Paper Section 2: subln normalisation in front of BitLinear; 8-bit absmax quantisation per token.)
//
// One CTA per token.  The bf16 row is read once with 128-bit loads and kept in registers; the sum
// of squares is reduced in fp64 (warp shuffles, then a fixed-order sum over warps), the maximum of
// the normalised row in fp32; the second pass quantises from registers and writes 8 codes per store.
#include "common.cuh"

namespace bitlinear {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct RowReduceSmem {
    double sq[kWarps];
    float mx[kWarps];
    int sum[kWarps];
};

__device__ __forceinline__ void unpack_bf16x8(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        f[2 * e] = __uint_as_float(w[e] << 16);
        f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
}

template <int VPT>  // 16-byte vectors (8 bf16) per thread
__global__ void __launch_bounds__(kThreads) quant_act_kernel(const __nv_bfloat16* __restrict__ x,
                                                             const __nv_bfloat16* __restrict__ gain, float eps,
                                                             int K, int8_t* __restrict__ xq, float* __restrict__ d_out,
                                                             int32_t* __restrict__ xsum_out) {
    __shared__ RowReduceSmem sm;
    const int row = blockIdx.x;
    const int n_vec = K >> 3;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint4* xrow = reinterpret_cast<const uint4*>(x + (size_t)row * K);
    const uint4* grow = reinterpret_cast<const uint4*>(gain);

    uint4 xv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kThreads;
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
    for (int w = 0; w < kWarps; ++w) S += sm.sq[w];
    const float r = (float)(1.0 / sqrt(S / (double)K + (double)eps));

    // ---- normalise (kept in registers) and find the absolute maximum ----
    float y[VPT][8];
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kThreads;
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
    for (int w = 0; w < kWarps; ++w) a = fmaxf(a, sm.mx[w]);
    a = fmaxf(a, 1e-5f);
    const float s = __fdiv_rn(127.0f, a);

    // ---- quantise from registers ----
    int csum = 0;
    uint2* qrow = reinterpret_cast<uint2*>(xq + (size_t)row * K);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kThreads;
        uint32_t packed[2] = {0u, 0u};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int q = __float2int_rn(__fmul_rn(y[i][e], s));
            q = max(-128, min(127, q));
            csum += q;
            packed[e >> 2] |= (uint32_t)(q & 0xff) << (8 * (e & 3));
        }
        if (v < n_vec) qrow[v] = make_uint2(packed[0], packed[1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
    if (lane == 0) sm.sum[warp] = csum;
    __syncthreads();
    if (tid == 0) {
        int total = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) total += sm.sum[w];
        d_out[row] = __fdiv_rn(a, 127.0f);
        if (xsum_out != nullptr) xsum_out[row] = total;
    }
}

}  // namespace

cudaError_t launch_quant_act(const __nv_bfloat16* x, const __nv_bfloat16* gain, float eps, int M, int K,
                             int8_t* xq, float* d, int32_t* xsum, cudaStream_t st) {
    const int n_vec = K / 8;
    const int vpt = (n_vec + kThreads - 1) / kThreads;
    const dim3 grid((unsigned)M), block(kThreads);
    if (vpt <= 1) quant_act_kernel<1><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 2) quant_act_kernel<2><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 4) quant_act_kernel<4><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else quant_act_kernel<8><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);  // K <= 16384
    return cudaGetLastError();
}

}  // namespace bitlinear
