// Decode contraction (M <= 16 tokens): streams the 2-bit packed weights once, unpacks in registers
// into dot-product-of-four operands, and applies the dequantising epilogue.
// (Paper Section 5.1: packed weights come from HBM and are expanded on chip right before the
// product with the 8-bit activations; the cost that matters is the packed bytes moved.)
//
// One CTA per block of 16 weight rows.  The warps of the CTA split that row block's 16x256 tiles;
// inside a tile lane (g, t) = (lane/4, lane%4) owns the 16-byte chunks of rows g and g+8 that hold
// columns 64t..64t+63, so one warp-wide 128-bit load covers 512 contiguous bytes.  Partial sums are
// folded over the four t lanes with shuffles and over the warps through shared memory.
#include "common.cuh"

namespace bitlinear {

namespace {

__device__ __forceinline__ int dp4a_u8_s8(uint32_t a_u8x4, uint32_t b_s8x4, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_u8x4), "r"(b_s8x4), "r"(c));
    return d;
}

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    // weights are read exactly once: bypass L1 allocation
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <int MT, int TPW>  // tokens per CTA pass, tiles per warp
__global__ void __launch_bounds__(512) gemv_kernel(const int8_t* __restrict__ xq, const float* __restrict__ d,
                                                   const int32_t* __restrict__ xsum,
                                                   const uint32_t* __restrict__ packed,
                                                   const float* __restrict__ s_w_ptr, int m0, int M, int N, int K,
                                                   void* __restrict__ y, int y_dtype, int32_t* __restrict__ acc_out) {
    extern __shared__ int red[];  // [warps][16 rows][MT]
    const int warps = blockDim.x >> 5;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int k_tiles = K / kTileCols;
    const int rb = blockIdx.x;
    const uint4* tiles = reinterpret_cast<const uint4*>(packed) + (size_t)rb * k_tiles * (kTileBytes / 16);

    // issue every weight load of this warp first
    uint4 wv[TPW][2];
#pragma unroll
    for (int it = 0; it < TPW; ++it) {
        const int kt = warp + it * warps;
        if (kt < k_tiles) {
            wv[it][0] = ldg_stream(tiles + (size_t)kt * 64 + lane);
            wv[it][1] = ldg_stream(tiles + (size_t)kt * 64 + 32 + lane);
        } else {
            wv[it][0] = make_uint4(0, 0, 0, 0);
            wv[it][1] = make_uint4(0, 0, 0, 0);
        }
    }

    int acc[2][MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[0][m] = acc[1][m] = 0;

#pragma unroll
    for (int it = 0; it < TPW; ++it) {
        const int kt = warp + it * warps;
        if (kt >= k_tiles) break;
        // the 16 code words (4 per 32-bit word) of both rows, shared by all tokens
        uint32_t c0[4][4], c1[4][4];
        const uint32_t w0[4] = {wv[it][0].x, wv[it][0].y, wv[it][0].z, wv[it][0].w};
        const uint32_t w1[4] = {wv[it][1].x, wv[it][1].y, wv[it][1].z, wv[it][1].w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                c0[i][j] = (w0[i] >> (2 * j)) & 0x03030303u;
                c1[i][j] = (w1[i] >> (2 * j)) & 0x03030303u;
            }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m0 + m < M) {
                const uint4* xr =
                    reinterpret_cast<const uint4*>(xq + (size_t)(m0 + m) * K + (size_t)kt * kTileCols + 64 * t);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 xv = __ldg(xr + i);
                    const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc[0][m] = dp4a_u8_s8(c0[i][j], xw[j], acc[0][m]);
                        acc[1][m] = dp4a_u8_s8(c1[i][j], xw[j], acc[1][m]);
                    }
                }
            }
        }
    }

    // fold the four column lanes of each row
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int v = acc[h][m];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            acc[h][m] = v;
        }
    }
    if (t == 0) {
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            red[(warp * 16 + g) * MT + m] = acc[0][m];
            red[(warp * 16 + 8 + g) * MT + m] = acc[1][m];
        }
    }
    __syncthreads();

    // fold the warps, remove the code offset (sum of c*x minus sum of x), dequantise, store
    const float s_w = *s_w_ptr;
    for (int o = threadIdx.x; o < 16 * MT; o += blockDim.x) {
        const int m = o >> 4, r = o & 15;
        if (m0 + m >= M) continue;
        int total = 0;
        for (int w = 0; w < warps; ++w) total += red[(w * 16 + r) * MT + m];
        total -= xsum[m0 + m];
        const size_t idx = (size_t)(m0 + m) * N + (size_t)rb * kTileRows + r;
        const float val = __fmul_rn(__fmul_rn((float)total, s_w), d[m0 + m]);
        if (y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(val);
        else reinterpret_cast<float*>(y)[idx] = val;
        if (acc_out != nullptr) acc_out[idx] = total;
    }
}

template <int MT>
cudaError_t launch_mt(int tpw, dim3 grid, dim3 block, size_t smem, cudaStream_t st, const int8_t* xq, const float* d,
                      const int32_t* xsum, const uint32_t* packed, const float* s_w, int m0, int M, int N, int K,
                      void* y, int y_dtype, int32_t* acc_out) {
    switch (tpw) {
        case 1: gemv_kernel<MT, 1><<<grid, block, smem, st>>>(xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out); break;
        case 2: gemv_kernel<MT, 2><<<grid, block, smem, st>>>(xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out); break;
        case 3: gemv_kernel<MT, 3><<<grid, block, smem, st>>>(xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out); break;
        default: gemv_kernel<MT, 4><<<grid, block, smem, st>>>(xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out); break;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemv(const int8_t* xq, const float* d, const int32_t* xsum, const uint32_t* packed,
                        const float* s_w, int M, int N, int K, void* y, int y_dtype, int32_t* acc_out,
                        cudaStream_t st) {
    const int k_tiles = K / kTileCols;          // <= 64
    const int tpw = (k_tiles + 15) / 16;        // 1..4
    const int warps = (k_tiles + tpw - 1) / tpw;  // <= 16
    const dim3 grid((unsigned)(N / kTileRows)), block((unsigned)(warps * 32));
    for (int m0 = 0; m0 < M; m0 += kGemvMaxTokens) {
        const int rem = M - m0;
        cudaError_t e;
        if (rem <= 1) e = launch_mt<1>(tpw, grid, block, warps * 16 * 1 * sizeof(int), st, xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out);
        else if (rem <= 2) e = launch_mt<2>(tpw, grid, block, warps * 16 * 2 * sizeof(int), st, xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out);
        else if (rem <= 4) e = launch_mt<4>(tpw, grid, block, warps * 16 * 4 * sizeof(int), st, xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out);
        else if (rem <= 8) e = launch_mt<8>(tpw, grid, block, warps * 16 * 8 * sizeof(int), st, xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out);
        else e = launch_mt<16>(tpw, grid, block, warps * 16 * 16 * sizeof(int), st, xq, d, xsum, packed, s_w, m0, M, N, K, y, y_dtype, acc_out);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace bitlinear
