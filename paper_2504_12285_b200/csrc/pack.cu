// Offline weight path: absmean scale, ternary quantiser, 2-bit tiled packing, and the unpackers.
// (Paper Section 2, "Weight Quantization"; Section 5.1, four ternary values per stored byte.)
#include "common.cuh"

namespace bitlinear {

namespace {

constexpr int kRedThreads = 256;
constexpr int kMaxPartials = 1024;

__device__ __forceinline__ double block_sum_fixed_tree(double v, double* smem) {
    // warp butterfly, then a fixed-order sum of the per-warp values: the same tree every run
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double total = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += smem[w];
    __syncthreads();
    return total;
}

// Pass 1: each block sums |W| over a fixed, contiguous slice in fp64.
template <typename T>
__global__ void __launch_bounds__(kRedThreads) absmean_partial_kernel(const T* __restrict__ W, size_t count,
                                                                      double* __restrict__ partials) {
    __shared__ double smem[kRedThreads / 32];
    const size_t per_block = (count + gridDim.x - 1) / gridDim.x;
    const size_t begin = (size_t)blockIdx.x * per_block;
    size_t end = begin + per_block;
    if (end > count) end = count;
    double s = 0.0;
    for (size_t i = begin + threadIdx.x; i < end; i += kRedThreads) {
        float f;
        if constexpr (sizeof(T) == 2) f = __bfloat162float(W[i]);
        else f = W[i];
        s += (double)fabsf(f);
    }
    const double total = block_sum_fixed_tree(s, smem);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

// Pass 2: one block folds the partial sums in a fixed order and writes s_w = fl32(mean) + eps_w.
__global__ void __launch_bounds__(kRedThreads) absmean_final_kernel(const double* __restrict__ partials,
                                                                    int n_partials, size_t count, float eps_w,
                                                                    float* __restrict__ s_w_out) {
    __shared__ double smem[kRedThreads / 32];
    double s = 0.0;
    for (int i = threadIdx.x; i < n_partials; i += kRedThreads) s += partials[i];
    const double total = block_sum_fixed_tree(s, smem);
    if (threadIdx.x == 0) {
        const float beta = (float)(total / (double)count);
        *s_w_out = __fadd_rn(beta, eps_w);
    }
}

// Decode a packed 32-bit word index into its row and first column.
__device__ __forceinline__ void word_to_row_col(size_t word, int k_tiles, int& n, int& k0) {
    const size_t tile = word >> 8;  // 256 words per 1024-byte tile
    const int wo = (int)(word & 255);
    const int h = wo >> 7, g = (wo >> 4) & 7, t = (wo >> 2) & 3, i = wo & 3;
    n = (int)(tile / k_tiles) * kTileRows + 8 * h + g;
    k0 = (int)(tile % k_tiles) * kTileCols + 64 * t + 16 * i;
}

__device__ __forceinline__ uint32_t ternary_code(float w, float s_w) {
    float r = rintf(__fdiv_rn(w, s_w));
    r = fminf(fmaxf(r, -1.0f), 1.0f);
    return (uint32_t)((int)r + 1);
}

// Pass 3: one thread quantises 16 consecutive weights of a row into one packed 32-bit word.
template <typename T>
__global__ void __launch_bounds__(256) quant_pack_kernel(const T* __restrict__ W, int N, int K,
                                                         const float* __restrict__ s_w_ptr,
                                                         uint32_t* __restrict__ packed) {
    const size_t n_words = (size_t)N * K / 16;
    const size_t word = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= n_words) return;
    const float s_w = *s_w_ptr;
    int n, k0;
    word_to_row_col(word, K / kTileCols, n, k0);
    const T* src = W + (size_t)n * K + k0;
    float f[16];
    if constexpr (sizeof(T) == 2) {
        const uint4* v = reinterpret_cast<const uint4*>(src);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const uint4 u = v[q];
            const uint32_t w4[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                f[q * 8 + 2 * e] = __uint_as_float(w4[e] << 16);
                f[q * 8 + 2 * e + 1] = __uint_as_float(w4[e] & 0xffff0000u);
            }
        }
    } else {
        const float4* v = reinterpret_cast<const float4*>(src);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 u = v[q];
            f[4 * q] = u.x; f[4 * q + 1] = u.y; f[4 * q + 2] = u.z; f[4 * q + 3] = u.w;
        }
    }
    uint32_t out = 0;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const int j = e >> 2, b = e & 3;
        out |= ternary_code(f[e], s_w) << (8 * b + 2 * j);
    }
    packed[word] = out;
}

// Tensor-core staging order of the unpacked codes (see launch_unpack_codes_u8): one thread expands one
// packed word into the 16-byte piece of its 256-row x 128-column tile.
__global__ void __launch_bounds__(256) unpack_codes_tiled_kernel(const uint32_t* __restrict__ packed, int N, int K,
                                                                 uint8_t* __restrict__ out) {
    const size_t n_words = (size_t)N * K / 16;
    const size_t word = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= n_words) return;
    int n, k0;
    word_to_row_col(word, K / kTileCols, n, k0);
    const uint32_t p = packed[word];
    uint32_t v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = (p >> (2 * j)) & 0x03030303u;
    const int r = n & 255, piece = (k0 & 127) >> 4;
    const size_t tile = (size_t)(n >> 8) * (K / 128) + (k0 >> 7);
    *reinterpret_cast<uint4*>(out + tile * 32768 + (size_t)r * 128 + ((piece ^ (r & 7)) << 4)) =
        make_uint4(v[0], v[1], v[2], v[3]);
}

// One thread expands one packed word into 16 bytes.  SIGNED: values -1/0/1, else codes 0/1/2.
template <bool SIGNED>
__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t* __restrict__ packed, int N, int K,
                                                     uint8_t* __restrict__ out) {
    const size_t n_words = (size_t)N * K / 16;
    const size_t word = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= n_words) return;
    int n, k0;
    word_to_row_col(word, K / kTileCols, n, k0);
    const uint32_t p = packed[word];
    uint32_t v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t c = (p >> (2 * j)) & 0x03030303u;
        if (SIGNED) c = __vsub4(c, 0x01010101u);  // per-byte c - 1 (wraps 0 -> 0xff = -1)
        v[j] = c;
    }
    *reinterpret_cast<uint4*>(out + (size_t)n * K + k0) = make_uint4(v[0], v[1], v[2], v[3]);
}

// ---- dense layout: five ternary values per byte (see "Dense packed weight layout" in bitlinear.h) ----

// One thread quantises the 20 consecutive weights of one packed 32-bit word: column k0 + 4*e + b is base-3 digit e
// (digit 0 most significant) of byte b; columns past K are padding and count as zero weights.
template <typename T>
__global__ void __launch_bounds__(256) quant_pack5_kernel(const T* __restrict__ W, int N, int K,
                                                          const float* __restrict__ s_w_ptr,
                                                          uint32_t* __restrict__ packed) {
    const int k_tiles = dense_k_tiles(K);
    const size_t n_words = (size_t)(N / kTileRows) * k_tiles * (kTileBytes / 4);
    const size_t word = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= n_words) return;
    const float s_w = *s_w_ptr;
    const size_t tile = word >> 8;
    const int wo = (int)(word & 255);
    const int h = wo >> 7, g = (wo >> 4) & 7, t = (wo >> 2) & 3, i = wo & 3;
    const int n = (int)(tile / k_tiles) * kTileRows + 8 * h + g;
    const int k0 = (int)(tile % k_tiles) * kDenseTileCols + 80 * t + 20 * i;
    const T* src = W + (size_t)n * K;
    uint32_t v[4] = {0u, 0u, 0u, 0u};  // the base-3 number of each byte, built digit by digit
#pragma unroll
    for (int e = 0; e < 5; ++e)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int k = k0 + 4 * e + b;
            uint32_t c = 1u;
            if (k < K) {
                float w;
                if constexpr (sizeof(T) == 2) w = __bfloat162float(src[k]);
                else w = src[k];
                c = ternary_code(w, s_w);
            }
            v[b] = v[b] * 3u + c;
        }
    uint32_t out = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b) out |= ((256u * v[b] + 242u) / 243u) << (8 * b);  // ceil(256 v / 243)
    packed[word] = out;
}

// Test hook: one thread per weight; the byte's base-3 number is recovered as floor(243 B / 256) and the digit by division.
__global__ void __launch_bounds__(256) unpack5_kernel(const uint8_t* __restrict__ packed, int N, int K, int8_t* __restrict__ out) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx - (size_t)n * K);
    const int k_tiles = dense_k_tiles(K);
    const size_t tile = (size_t)(n / kTileRows) * k_tiles + k / kDenseTileCols;
    const int r = n % kTileRows, c = k % kDenseTileCols;
    const int t = c / 80, i = (c % 80) / 20, e = (c % 20) / 4, b = c % 4;
    const uint32_t B = packed[tile * kTileBytes + 512 * (r / 8) + 64 * (r % 8) + 16 * t + 4 * i + b];
    uint32_t v = (243u * B) >> 8;
    for (int s = e; s < 4; ++s) v /= 3u;
    out[idx] = (int8_t)((int)(v % 3u) - 1);
}

}  // namespace

cudaError_t launch_quant_pack5(const void* W, int w_dtype, int N, int K, const float* s_w, uint32_t* packed, cudaStream_t st) {
    const size_t n_words = (size_t)(N / kTileRows) * dense_k_tiles(K) * (kTileBytes / 4);
    const unsigned blocks = (unsigned)((n_words + 255) / 256);
    if (w_dtype == BITLINEAR_BF16)
        quant_pack5_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W), N, K, s_w, packed);
    else
        quant_pack5_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(W), N, K, s_w, packed);
    return cudaGetLastError();
}

cudaError_t launch_unpack5_i8(const uint8_t* packed, int N, int K, int8_t* wq, cudaStream_t st) {
    const size_t n = (size_t)N * K;
    unpack5_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(packed, N, K, wq);
    return cudaGetLastError();
}

int absmean_num_partials(size_t count) {
    size_t want = (count + (size_t)kRedThreads * 64 - 1) / ((size_t)kRedThreads * 64);
    if (want < 1) want = 1;
    if (want > kMaxPartials) want = kMaxPartials;
    return (int)want;
}

cudaError_t launch_absmean(const void* W, int w_dtype, size_t count, float eps_w, double* partials,
                           int n_partials, float* s_w_out, cudaStream_t st) {
    if (w_dtype == BITLINEAR_BF16)
        absmean_partial_kernel<__nv_bfloat16><<<n_partials, kRedThreads, 0, st>>>(
            static_cast<const __nv_bfloat16*>(W), count, partials);
    else
        absmean_partial_kernel<float><<<n_partials, kRedThreads, 0, st>>>(static_cast<const float*>(W), count,
                                                                          partials);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    absmean_final_kernel<<<1, kRedThreads, 0, st>>>(partials, n_partials, count, eps_w, s_w_out);
    return cudaGetLastError();
}

cudaError_t launch_quant_pack(const void* W, int w_dtype, int N, int K, const float* s_w, uint32_t* packed,
                              cudaStream_t st) {
    const size_t n_words = (size_t)N * K / 16;
    const unsigned blocks = (unsigned)((n_words + 255) / 256);
    if (w_dtype == BITLINEAR_BF16)
        quant_pack_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W), N, K, s_w,
                                                                 packed);
    else
        quant_pack_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(W), N, K, s_w, packed);
    return cudaGetLastError();
}

cudaError_t launch_unpack_i8(const uint32_t* packed, int N, int K, int8_t* wq, cudaStream_t st) {
    const size_t n_words = (size_t)N * K / 16;
    unpack_kernel<true><<<(unsigned)((n_words + 255) / 256), 256, 0, st>>>(packed, N, K,
                                                                           reinterpret_cast<uint8_t*>(wq));
    return cudaGetLastError();
}

// Codes 0/1/2 as bytes, in the order the tensor-core kernel stages them: the [N][K] matrix is cut into tiles of
// 256 rows x 128 columns, 32 KiB each, stored row-tile major; inside a tile row r keeps its eight 16-byte pieces at
// r*128 + ((piece ^ (r & 7)) * 16), which is the 128-byte shared-memory swizzle.  A tile is therefore the exact
// shared-memory image of one pipeline stage of the weight operand and is fetched with one linear bulk copy.
cudaError_t launch_unpack_codes_u8(const uint32_t* packed, int N, int K, uint8_t* codes, cudaStream_t st) {
    const size_t n_words = (size_t)N * K / 16;
    unpack_codes_tiled_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, st>>>(packed, N, K, codes);
    return cudaGetLastError();
}

}  // namespace bitlinear
