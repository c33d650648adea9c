// One level of a decoder layer at ONE token: up to four BitLinear forwards that read the same input row through the same
// step and norm (q/k/v, o, gate/up, down), in ONE launch with no tables in global memory.
// (Paper Section 5.1: decode is bound by loading the packed weights; at one token a level of the 2B model is 1.6 - 8.8 MB,
// so what a level costs is latency, not bytes: launch, dependent global reads, block barriers.)
//
// Everything the kernel needs is in its parameters.  A CTA takes a contiguous run of 16-row weight blocks and
//   1. before anything else starts bulk copies of its whole share of the packed weights (11 - 60 KB) into shared memory,
//      and lets the next launch of the stream begin (programmatic dependent launch): with level kernels back to back the
//      next level's CTAs sit beside this level's and fetch their weights while this level computes.  (Only a caller that
//      vouches that the launch in front does not write weights, scales or gain gets this launch as a dependent; for
//      everybody else the launch is ordinary and step 2 returns at once.)
//   2. waits for the launch before it (griddepcontrol.wait) - nothing but weights, their scales and the norm's gain
//      (all static) is read earlier;
//   3. quantises the input row itself (fused RMSNorm + absmax int8, the element-wise step in front of it included):
//      every CTA repeats this, which costs less than a quantiser launch and its round trip through memory;
//   4. multiplies: a warp takes a slice of the 256-column tiles of one row block (dot-products-of-four on
//      word & (0x03030303 << 2j), as in the streaming kernel), partial sums meet in shared memory (integers: exact);
//   5. dequantises and stores.
// CTA 0 also writes the codes, the scale and the code sum where a quantiser launch would have put them (when the caller
// names such a place), so that a later call on the same workspace may reuse them.
#include "decode_level.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

constexpr int kLevelThreads = 512;
// CTAs per SM the row blocks are dealt to: with two, a CTA's weight copy and products halve while the quantiser, which every
// CTA repeats anyway, runs in parallel.  Measured per decoded token of the 2B configuration (CUDA graph): 1.05 ms with
// one CTA per SM, 1.00 ms with two, 1.11 ms when the largest level is dealt to three (a second wave of CTAs).
constexpr int kLevelCtasPerSm = 2;
constexpr int kLevelWarps = kLevelThreads / 32;

__device__ __forceinline__ int dp4a_u8_s8(uint32_t a_u8x4, uint32_t b_s8x4, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_u8x4), "r"(b_s8x4), "r"(c));
    return d;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// shared memory: [weights: rb_per_cta x k_tiles KiB][codes of the row: K bytes][gain: 2K bytes][partial sums][barrier, abort flag]
__host__ __device__ inline size_t level_smem_bytes(int rb_per_cta, int K) {
    return (size_t)rb_per_cta * (K / kTileCols) * kTileBytes + (size_t)3 * K + (size_t)rb_per_cta * kLevelWarps * 16 * sizeof(int) + 32;
}

template <int VPT>
__global__ void __launch_bounds__(kLevelThreads) decode_level_kernel(const __grid_constant__ LevelParams P) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ RowReduceSmemT<kLevelWarps> qsm;
    __shared__ float d_s;
    __shared__ int xsum_s;
    const int k_tiles = P.K / kTileCols;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb_lo = blockIdx.x * P.rb_per_cta, rb_hi = min(P.total_rb, rb_lo + P.rb_per_cta);
    const int R = rb_hi - rb_lo;  // >= 1 by the grid size
    const uint32_t rb_bytes = (uint32_t)k_tiles * kTileBytes;
    uint8_t* arena = smem + (size_t)P.rb_per_cta * rb_bytes;
    uint4* gain_s = reinterpret_cast<uint4*>(arena + P.K);  // the norm's gain, copied before the wait (it is static)
    int* part = reinterpret_cast<int*>(arena + 3 * (size_t)P.K);  // [rb][warp slot][16 rows]
    uint64_t* bar = reinterpret_cast<uint64_t*>(part + P.rb_per_cta * kLevelWarps * 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar + 1);
    const uint32_t bar_s = smem_u32(bar), w_s = smem_u32(smem);

    // which problem a global row block belongs to, and its index inside that problem
    auto locate = [&](int rb, int& i, int& local) {
        i = 0;
        local = rb;
        while (i + 1 < P.count && local >= P.prob[i].N / kTileRows) {
            local -= P.prob[i].N / kTileRows;
            ++i;
        }
    };

    // ---- 1. the weights of this CTA's row blocks: one bulk copy per row block, issued by one thread per warp ----
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar_s, 1);
        mbar_init_fence();
        mbar_expect_tx(bar_s, (uint32_t)R * rb_bytes);
    }
    __syncthreads();
    if (lane == 0)
        for (int j = warp; j < R; j += kLevelWarps) {
            int i, local;
            locate(rb_lo + j, i, local);
            bulk_load_once(w_s + (uint32_t)j * rb_bytes, P.prob[i].packed + (size_t)local * rb_bytes, rb_bytes, bar_s,
                           l2_evict_first_policy());  // a decode loop's weights pass through L2 once per token
        }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // what else does not depend on the launch before this one: the gain vector and the weight scales
    if (P.gain != nullptr)
        for (int v = threadIdx.x; v < (P.K >> 3); v += kLevelThreads) gain_s[v] = reinterpret_cast<const uint4*>(P.gain)[v];
    float s_w[kLevelMaxProblems];
#pragma unroll
    for (int i = 0; i < kLevelMaxProblems; ++i) s_w[i] = i < P.count ? *P.prob[i].s_w : 0.0f;

    // ---- 2. everything else depends on the launch before this one ----
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();  // the gain copy is complete

    // ---- 3. the input row -> int8 codes in shared memory ----
    {
        RowOp op = P.op;
        if (blockIdx.x != 0) op.x_out = nullptr;  // the step's own output (a new hidden state) is written once
        with_row_source(op, P.x, P.x_row0, P.K, [&](auto src) {
            quant_row_src<VPT, 1, decltype(src), kLevelThreads>(src, P.gain ? reinterpret_cast<const __nv_bfloat16*>(gain_s) : nullptr, P.eps,
                                                                P.K, reinterpret_cast<int8_t*>(arena), &d_s, &xsum_s, qsm);
        });
        __syncthreads();
        if (blockIdx.x == 0 && P.xq_out != nullptr) {
            for (int o = threadIdx.x * 16; o < P.K; o += kLevelThreads * 16)
                *reinterpret_cast<uint4*>(P.xq_out + o) = *reinterpret_cast<const uint4*>(arena + o);
            if (threadIdx.x == 0) {
                *P.d_out = d_s;
                *P.xsum_out = xsum_s;
            }
        }
    }

    // ---- 4. the products: S warps share the tiles of a row block ----
    const int S = R >= kLevelWarps ? 1 : kLevelWarps / R;  // warps per row block
    const bool ok = mbar_wait(bar_s, 0, abort_flag);
    if (ok) {
        const int g = lane >> 2, t = lane & 3;
        const uint32_t x_s = smem_u32(arena) + (uint32_t)t * 16u;
        for (int item = warp; item < R * S; item += kLevelWarps) {
            const int j = item / S, s = item - j * S;
            const int t0 = (k_tiles * s) / S, t1 = (k_tiles * (s + 1)) / S;
            int acc[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[h][q] = 0;
            uint32_t wa = w_s + (uint32_t)j * rb_bytes + (uint32_t)t0 * kTileBytes + (uint32_t)lane * 16u;
            uint32_t xo = (uint32_t)t0 * kTileCols;
#pragma unroll 2
            for (int tile = t0; tile < t1; ++tile, wa += kTileBytes, xo += kTileCols) {
                const uint4 w0v = lds128(wa), w1v = lds128(wa + 512);
                const uint32_t w0[4] = {w0v.x, w0v.y, w0v.z, w0v.w};
                const uint32_t w1[4] = {w1v.x, w1v.y, w1v.z, w1v.w};
                // the codes are stored with the four 16-byte pieces of each lane's 64 columns interleaved (piece q of lane t
                // at 64q + 16t inside the tile), so the four t lanes read 64 contiguous bytes
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 v = lds128(x_s + xo + 64u * q);
                    const uint32_t xw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t mask = 0x03030303u << (2 * c);
                        acc[0][c] = dp4a_u8_s8(w0[q] & mask, xw[c], acc[0][c]);
                        acc[1][c] = dp4a_u8_s8(w1[q] & mask, xw[c], acc[1][c]);
                    }
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                // accumulator c holds 4^c x its share: 64 x the sum is ((a0*4 + a1)*4 + a2)*4 + a3 (no overflow for K <= 8192)
                int sum = ((acc[h][0] * 4 + acc[h][1]) * 4 + acc[h][2]) * 4 + acc[h][3];
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                if (t == 0) part[(j * kLevelWarps + s) * 16 + g + 8 * h] = sum >> 6;  // exact: a multiple of 64
            }
        }
    }
    __syncthreads();  // partial sums complete - or the CTA gives up together
    if (*abort_flag) {
        if (threadIdx.x == 0 && P.status_word != nullptr) atomicExch(P.status_word, BITLINEAR_ERR_TIMEOUT);
        abort_drain();
        return;
    }

    // ---- 5. one thread per weight row: add the slices, remove the code offset, dequantise, store ----
    for (int idx = threadIdx.x; idx < R * 16; idx += kLevelThreads) {
        const int j = idx >> 4, r = idx & 15;
        int v = 0;
        for (int s = 0; s < S; ++s) v += part[(j * kLevelWarps + s) * 16 + r];
        v -= xsum_s;
        int i, local;
        locate(rb_lo + j, i, local);
        const LevelProblem& p = P.prob[i];
        float sw = s_w[0];
#pragma unroll
        for (int c = 1; c < kLevelMaxProblems; ++c) sw = i == c ? s_w[c] : sw;
        const float val = __fmul_rn(__fmul_rn((float)v, sw), d_s);
        const size_t n = (size_t)local * kTileRows + r;
        if (p.acc_out != nullptr) p.acc_out[n] = v;
        if (p.y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(p.y)[n] = __float2bfloat16_rn(val);
        else reinterpret_cast<float*>(p.y)[n] = val;
    }
}

// dependent: launch as a programmatic dependent of the launch before it (the kernel then reads weights, scales and gain
// while that launch may still be running: only for callers who vouch that it does not write them)
template <int VPT>
cudaError_t launch_level(const LevelParams& P, int grid, size_t smem, cudaStream_t st, bool dependent) {
    // the opt-in is per device and cheap: repeated so that every device a process uses gets it
    if (smem > 40 * 1024) {  // the 48 KiB default covers static and dynamic shared memory together
        const cudaError_t e = cudaFuncSetAttribute(decode_level_kernel<VPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kLevelThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, decode_level_kernel<VPT>, P);
}

}  // namespace

bool decode_level_fits(int count, int total_rb, int K, int sm_count) {
    if (count < 1 || count > kLevelMaxProblems || K > 8192 || sm_count <= 0) return false;
    const int rb_per_cta = (total_rb + kLevelCtasPerSm * sm_count - 1) / (kLevelCtasPerSm * sm_count);
    return level_smem_bytes(rb_per_cta, K) <= 100 * 1024 / kLevelCtasPerSm;  // two launches of this kind fit an SM side by side
}

int decode_level_forward(LevelParams& P, int sm_count, cudaStream_t st, bool dependent) {
    P.rb_per_cta = (P.total_rb + kLevelCtasPerSm * sm_count - 1) / (kLevelCtasPerSm * sm_count);
    const int grid = (P.total_rb + P.rb_per_cta - 1) / P.rb_per_cta;
    const size_t smem = level_smem_bytes(P.rb_per_cta, P.K);
    const cudaError_t e = P.K <= 8 * kLevelThreads ? launch_level<1>(P, grid, smem, st, dependent) : launch_level<2>(P, grid, smem, st, dependent);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

}  // namespace bitlinear
