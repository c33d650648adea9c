// Batched decode: many independent BitLinear forwards (M <= 16 tokens each) in two launches.
// (Paper Section 5.1: the decode cost is the packed weight bytes that must cross HBM; a single
// decode matmul is smaller than the memory system's bandwidth-delay product, so the weights of a
// whole batch of matmuls are streamed back to back by one persistent kernel.)
//
//   launch 1  batch_quant_kernel : one CTA per token of every problem - fused RMSNorm + absmax
//             int8 quantiser into the workspace.
//   launch 2  decode_stream_kernel : one persistent CTA per SM.  The work list is every block of
//             16 weight rows of every problem ("item": 16 x K/4 contiguous packed bytes); each CTA
//             owns a contiguous, byte-balanced range of it.
//               warp 0      producer : one thread issues a linear bulk copy per item into a ring of
//                                      shared-memory stages (mbarrier completion)
//               warps 1-10  consumers: warp w owns the 16x256 tiles w, w+10, ... of every item; its
//                                      slice of the quantised activations stays in registers for
//                                      the whole problem.  M = 1: dot-product-of-four accumulation;
//                                      M > 1: legacy mma.sync m16n8k32 (u8 codes x s8 activations),
//                                      weights are the 16-row operand, tokens the 8-wide one.
//               warp 11     epilogue : folds the consumers' partial sums, subtracts the code offset,
//                                      applies the two scales and stores y.
//             Stages, partial-sum buffers and activations hand over through mbarriers only, so the
//             copy engine keeps streaming while consumers and epilogue work on earlier items.
#include <vector>

#include "quant_row.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

struct DevProblem {
    const uint32_t* packed;
    const float* s_w;
    void* y;
    const __nv_bfloat16* x;
    const __nv_bfloat16* gain;
    int8_t* xq;
    float* d;
    int32_t* xsum;
    int M, N, K, y_dtype;
    float eps;
    int k_tiles;
    int rb_per_item;  // 16-row blocks per work item (the last item of a problem may hold fewer)
    int item_begin;  // index of this problem's first item in the global work list
    int row_begin;   // index of this problem's first token in the global token list
};

// First bytes of the uploaded plan.  The kernels compare it with the values the host passes at
// launch, so a workspace that was overwritten between calls (with BITLINEAR_BATCH_REUSE_PLAN) is
// detected and reported instead of being followed into stale pointers.
struct PlanHeader {
    unsigned magic;
    int count, total_items, grid, rows;
    int pad[3];
};
constexpr unsigned kPlanMagic = 0xB171A9E5u;

namespace {

__device__ __forceinline__ bool plan_matches(const PlanHeader* h, int count, int total_items, int grid, int rows) {
    return h->magic == kPlanMagic && h->count == count && h->total_items == total_items && h->grid == grid &&
           h->rows == rows;
}

constexpr int kConsumers = 10;
constexpr int kStreamThreads = (kConsumers + 2) * 32;
constexpr int kMaxStages = 16;            // ring slots; a slot holds one item (16 rows x K/4 bytes, K <= 8192)
constexpr int kRedBufs = 2;
constexpr int kItemBytesCap = 32 * 1024;  // an item is as many 16-row blocks as fit in this many packed bytes
constexpr int kBatchMaxK = 8192;

// ------------------------------------------------------------------------------------ launch 1

template <int VPT>
__global__ void __launch_bounds__(kQuantThreads) batch_quant_kernel(const PlanHeader* __restrict__ hdr,
                                                                    const DevProblem* __restrict__ probs, int count,
                                                                    int total_items, int grid, int* status_word) {
    __shared__ RowReduceSmem sm;
    if (!plan_matches(hdr, count, total_items, grid, (int)gridDim.x)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int row = blockIdx.x;
    int lo = 0, hi = count - 1;  // last problem whose row_begin <= row
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (probs[mid].row_begin <= row) lo = mid;
        else hi = mid - 1;
    }
    const DevProblem& p = probs[lo];
    const int m = row - p.row_begin;
    quant_row<VPT>(p.x + (size_t)m * p.K, p.gain, p.eps, p.K, p.xq + (size_t)m * p.K, p.d + m, p.xsum + m, sm);
}

// ------------------------------------------------------------------------------------ launch 2

__device__ __forceinline__ int dp4a_u8_s8(uint32_t a_u8x4, uint32_t b_s8x4, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_u8x4), "r"(b_s8x4), "r"(c));
    return d;
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

struct StreamParams {
    const DevProblem* probs;
    const int* item_begin;  // [count + 1]
    const int* cta_begin;   // [gridDim.x + 1]
    const PlanHeader* hdr;
    int count, total_items, rows;
    int stages;
    int rb_max;       // largest rb_per_item of the batch
    int stage_bytes;  // size of a ring slot: the largest item of the batch, a multiple of 1024
    int* status_word;
};

// Compute the partial sums of one 16-row block for this warp's tiles and write them to `rbuf`
// ([16 rows][MP tokens]).  NT = 0: one token, dp4a.  NT = 1 / 2: up to 8 / 16 tokens, mma.sync.
template <int NT, int TPW>
__device__ __forceinline__ void row_block_partials(const uint4 (&wv)[TPW][2],
                                                   const uint32_t (&xr)[TPW][NT == 0 ? 1 : NT][16], int n_act,
                                                   int* rbuf, int g, int t) {
    constexpr int MP = NT == 0 ? 1 : 8 * NT;
    constexpr int XT = NT == 0 ? 1 : NT;
    if constexpr (NT == 0) {
        // accumulators per row and per bit position j hold 4^j x the true partial sum
        int acc[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
#pragma unroll
        for (int i = 0; i < TPW; ++i) {
            if (i >= n_act) break;  // warp-uniform: this warp owns n_act tiles of the row block
            const uint32_t w0[4] = {wv[i][0].x, wv[i][0].y, wv[i][0].z, wv[i][0].w};
            const uint32_t w1[4] = {wv[i][1].x, wv[i][1].y, wv[i][1].z, wv[i][1].w};
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t mask = 0x03030303u << (2 * j);
                    acc[0][j] = dp4a_u8_s8(w0[q] & mask, xr[i][0][4 * q + j], acc[0][j]);
                    acc[1][j] = dp4a_u8_s8(w1[q] & mask, xr[i][0][4 * q + j], acc[1][j]);
                }
        }
        int v0 = acc[0][0] + (acc[0][1] >> 2) + (acc[0][2] >> 4) + (acc[0][3] >> 6);
        int v1 = acc[1][0] + (acc[1][1] >> 2) + (acc[1][2] >> 4) + (acc[1][3] >> 6);
        v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
        v0 += __shfl_xor_sync(0xffffffffu, v0, 2);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 2);
        if (t == 0) {
            rbuf[g] = v0;
            rbuf[8 + g] = v1;
        }
    } else {
        int acc[4][XT][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int nt = 0; nt < XT; ++nt)
#pragma unroll
                for (int r = 0; r < 4; ++r) acc[j][nt][r] = 0;
#pragma unroll
        for (int i = 0; i < TPW; ++i) {
            if (i >= n_act) break;  // warp-uniform
            const uint32_t w0[4] = {wv[i][0].x, wv[i][0].y, wv[i][0].z, wv[i][0].w};
            const uint32_t w1[4] = {wv[i][1].x, wv[i][1].y, wv[i][1].z, wv[i][1].w};
#pragma unroll
            for (int q2 = 0; q2 < 2; ++q2)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t mask = 0x03030303u << (2 * j);
                    const int qa = 2 * q2, qb = 2 * q2 + 1;
                    const uint32_t a0 = w0[qa] & mask, a1 = w1[qa] & mask, a2 = w0[qb] & mask, a3 = w1[qb] & mask;
#pragma unroll
                    for (int nt = 0; nt < XT; ++nt)
                        mma_u8s8(acc[j][nt], a0, a1, a2, a3, xr[i][nt][4 * qa + j], xr[i][nt][4 * qb + j]);
                }
        }
#pragma unroll
        for (int nt = 0; nt < XT; ++nt) {
            int v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
                v[r] = acc[0][nt][r] + (acc[1][nt][r] >> 2) + (acc[2][nt][r] >> 4) + (acc[3][nt][r] >> 6);
            // fragment layout: r0 (row g, token 2t), r1 (g, 2t+1), r2 (g+8, 2t), r3 (g+8, 2t+1)
            const int tok = 8 * nt + 2 * t;
            *reinterpret_cast<int2*>(rbuf + g * MP + tok) = make_int2(v[0], v[1]);
            *reinterpret_cast<int2*>(rbuf + (g + 8) * MP + tok) = make_int2(v[2], v[3]);
        }
    }
}

// NT = 0: one token, dp4a.  NT = 1 / 2: up to 8 / 16 tokens, mma.sync with NT token tiles.
template <int NT, int TPW>
__global__ void __launch_bounds__(kStreamThreads, 1) decode_stream_kernel(const StreamParams prm) {
    constexpr int MP = NT == 0 ? 1 : 8 * NT;  // padded token count of the partial-sum buffers
    constexpr int XT = NT == 0 ? 1 : NT;
    constexpr int RB_INTS = kConsumers * 16 * MP;  // partial sums of one row block
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int stages = prm.stages;
    const int stage_bytes = prm.stage_bytes;
    int* red = reinterpret_cast<int*>(smem + (size_t)stages * stage_bytes);  // [kRedBufs][rb_max][kConsumers][16][MP]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red + kRedBufs * prm.rb_max * RB_INTS);
    uint64_t* full_bar = bars;                       // [stages]  bytes of the item landed
    uint64_t* empty_bar = bars + kMaxStages;         // [stages]  all consumers are done reading the item
    uint64_t* redfull_bar = bars + 2 * kMaxStages;   // [kRedBufs] all consumers wrote their partial sums
    uint64_t* redfree_bar = redfull_bar + kRedBufs;  // [kRedBufs] the epilogue is done with the buffer
    volatile int* abort_flag = reinterpret_cast<volatile int*>(redfree_bar + kRedBufs);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!plan_matches(prm.hdr, prm.count, prm.total_items, (int)gridDim.x, prm.rows)) {  // uniform over the grid
        if (blockIdx.x == 0 && threadIdx.x == 0 && prm.status_word != nullptr)
            atomicExch(prm.status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), kConsumers);
        }
        for (int b = 0; b < kRedBufs; ++b) {
            mbar_init(smem_u32(redfull_bar + b), kConsumers);
            mbar_init(smem_u32(redfree_bar + b), 1);
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const int item_lo = prm.cta_begin[blockIdx.x], item_hi = prm.cta_begin[blockIdx.x + 1];
    // problem that holds item_lo
    int p = 0;
    {
        int lo = 0, hi = prm.count - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prm.item_begin[mid] <= item_lo) lo = mid;
            else hi = mid - 1;
        }
        p = lo;
    }

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        if (lane == 0) {
            int next_begin = prm.item_begin[p];  // forces the first refresh
            const uint8_t* base = nullptr;
            int first = 0, rbpi = 1, n_rb = 0;
            uint32_t rb_bytes = 0;
            --p;
            uint32_t stage = 0, phase = 0;
            for (int it = item_lo; it < item_hi; ++it) {
                while (it >= next_begin) {
                    ++p;
                    next_begin = prm.item_begin[p + 1];
                    const DevProblem& pr = prm.probs[p];
                    base = reinterpret_cast<const uint8_t*>(pr.packed);
                    rb_bytes = (uint32_t)pr.k_tiles * kTileBytes;
                    first = pr.item_begin;
                    rbpi = pr.rb_per_item;
                    n_rb = pr.N / kTileRows;
                }
                const int rb0 = (it - first) * rbpi;
                const int nrb = (n_rb - rb0) < rbpi ? (n_rb - rb0) : rbpi;
                const uint32_t bytes = (uint32_t)nrb * rb_bytes;
                if (!mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag)) break;
                const uint32_t fb = smem_u32(full_bar + stage);
                mbar_expect_tx(fb, bytes);
                bulk_load(smem_u32(smem + (size_t)stage * stage_bytes), base + (size_t)rb0 * rb_bytes, bytes, fb);
                if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp <= kConsumers) {
        // ---------------------------------------------------------------- consumers
        const int w = warp - 1;
        const int g = lane >> 2, t = lane & 3;
        int next_begin = prm.item_begin[p], k_tiles = 0, first = 0, rbpi = 1, n_rb = 0, n_act = 0;
        --p;
        uint32_t xr[TPW][XT][16];  // this lane's activation bytes: tile, token tile, 16 words = 64 columns
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int it = item_lo; ok && it < item_hi; ++it) {
            if (it >= next_begin) {
                while (it >= next_begin) {
                    ++p;
                    next_begin = prm.item_begin[p + 1];
                }
                const DevProblem& pr = prm.probs[p];
                k_tiles = pr.k_tiles;
                first = pr.item_begin;
                rbpi = pr.rb_per_item;
                n_rb = pr.N / kTileRows;
                n_act = w < k_tiles ? (k_tiles - w + kConsumers - 1) / kConsumers : 0;  // tiles w, w+10, ... < k_tiles
#pragma unroll
                for (int i = 0; i < TPW; ++i) {
                    const int kt = w + i * kConsumers;
#pragma unroll
                    for (int nt = 0; nt < XT; ++nt) {
                        const int tok = NT == 0 ? 0 : g + 8 * nt;
                        if (kt < k_tiles && tok < pr.M) {
                            const uint4* src =
                                reinterpret_cast<const uint4*>(pr.xq + (size_t)tok * pr.K + (size_t)kt * kTileCols + 64 * t);
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint4 v = src[q];
                                xr[i][nt][4 * q] = v.x; xr[i][nt][4 * q + 1] = v.y;
                                xr[i][nt][4 * q + 2] = v.z; xr[i][nt][4 * q + 3] = v.w;
                            }
                        } else {
#pragma unroll
                            for (int q = 0; q < 16; ++q) xr[i][nt][q] = 0u;
                        }
                    }
                }
            }
            const int c = it - item_lo;
            const int rb0 = (it - first) * rbpi;
            const int nrb = (n_rb - rb0) < rbpi ? (n_rb - rb0) : rbpi;
            if (!mbar_wait(smem_u32(full_bar + stage), phase, abort_flag)) { ok = false; break; }
            const uint32_t rphase = (uint32_t)(c / kRedBufs) & 1u;
            if (!mbar_wait(smem_u32(redfree_bar + c % kRedBufs), rphase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t sbase = smem_u32(smem + (size_t)stage * stage_bytes) + lane * 16;
            int* rbase = red + (c % kRedBufs) * prm.rb_max * RB_INTS + w * 16 * MP;
            for (int r = 0; r < nrb; ++r) {
                uint4 wv[TPW][2];
#pragma unroll
                for (int i = 0; i < TPW; ++i) {
                    const int kt = w + i * kConsumers;
                    if (i < n_act) {
                        wv[i][0] = lds128(sbase + (r * k_tiles + kt) * kTileBytes);
                        wv[i][1] = lds128(sbase + (r * k_tiles + kt) * kTileBytes + 512);
                    }
                }
                row_block_partials<NT, TPW>(wv, xr, n_act, rbase + r * RB_INTS, g, t);
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(empty_bar + stage));
                mbar_arrive(smem_u32(redfull_bar + c % kRedBufs));
            }
            if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        int next_begin = prm.item_begin[p], first = 0, active = 0, M = 0, N = 0, y_dtype = 0, rbpi = 1, n_rb = 0;
        --p;
        float s_w = 0.0f;
        void* y = nullptr;
        int xs_lane = 0;       // lane m holds the code sum and the scale of token m of the current problem
        float d_lane = 0.0f;
        for (int it = item_lo; it < item_hi; ++it) {
            if (it >= next_begin) {
                while (it >= next_begin) {
                    ++p;
                    next_begin = prm.item_begin[p + 1];
                }
                const DevProblem& pr = prm.probs[p];
                first = pr.item_begin;
                active = pr.k_tiles < kConsumers ? pr.k_tiles : kConsumers;
                M = pr.M; N = pr.N; y_dtype = pr.y_dtype;
                rbpi = pr.rb_per_item;
                n_rb = pr.N / kTileRows;
                s_w = *pr.s_w;
                y = pr.y;
                xs_lane = lane < M ? pr.xsum[lane] : 0;
                d_lane = lane < M ? pr.d[lane] : 0.0f;
            }
            const int c = it - item_lo;
            const int rb0 = (it - first) * rbpi;
            const int nrb = (n_rb - rb0) < rbpi ? (n_rb - rb0) : rbpi;
            const uint32_t rphase = (uint32_t)(c / kRedBufs) & 1u;
            if (!mbar_wait(smem_u32(redfull_bar + c % kRedBufs), rphase, abort_flag)) break;
            const int* rb = red + (c % kRedBufs) * prm.rb_max * RB_INTS;
            const int rows = nrb * 16;
            for (int m = 0; m < M; ++m) {
                const int xs = __shfl_sync(0xffffffffu, xs_lane, m);
                const float dm = __shfl_sync(0xffffffffu, d_lane, m);
                for (int rr = lane; rr < rows; rr += 32) {  // consecutive lanes -> consecutive output rows
                    const int r = rr >> 4, row = rr & 15;
                    int total = 0;
                    for (int w = 0; w < active; ++w) total += rb[r * RB_INTS + (w * 16 + row) * MP + m];
                    total -= xs;
                    const float val = __fmul_rn(__fmul_rn((float)total, s_w), dm);
                    const size_t idx = (size_t)m * N + (size_t)rb0 * kTileRows + rr;
                    if (y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(val);
                    else reinterpret_cast<float*>(y)[idx] = val;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(redfree_bar + c % kRedBufs));
        }
    }

    __syncthreads();
    if (*abort_flag) {
        abort_drain();
        if (threadIdx.x == 0 && prm.status_word != nullptr) atomicExch(prm.status_word, BITLINEAR_ERR_TIMEOUT);
    }
}

template <int NT, int TPW>
cudaError_t launch_stream(const StreamParams& prm, int grid, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(decode_stream_kernel<NT, TPW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    decode_stream_kernel<NT, TPW><<<grid, kStreamThreads, smem, st>>>(prm);
    return cudaGetLastError();
}

template <int NT>
cudaError_t launch_stream_nt(int tpw, const StreamParams& prm, int grid, size_t smem, cudaStream_t st) {
    switch (tpw) {
        case 1: return launch_stream<NT, 1>(prm, grid, smem, st);
        case 2: return launch_stream<NT, 2>(prm, grid, smem, st);
        case 3: return launch_stream<NT, 3>(prm, grid, smem, st);
        default: return launch_stream<NT, 4>(prm, grid, smem, st);
    }
}

struct PlanLayout {
    size_t probs_off, item_off, cta_off, xq_off, total;
};

PlanLayout plan_layout(int count, int grid, size_t xq_bytes, size_t rows) {
    PlanLayout L;
    size_t off = 256;  // the PlanHeader sits at offset 0
    L.probs_off = off;
    off = align_up(off + (size_t)count * sizeof(DevProblem), 256);
    L.item_off = off;
    off = align_up(off + (size_t)(count + 1) * sizeof(int), 256);
    L.cta_off = off;
    off = align_up(off + (size_t)(grid + 1) * sizeof(int), 256);
    L.xq_off = off;
    off = align_up(off + xq_bytes, 256);                   // int8 activations of every problem
    off = align_up(off + rows * sizeof(float), 256);       // d
    off = align_up(off + rows * sizeof(int32_t), 256);     // xsum
    L.total = off;
    return L;
}

constexpr int kPlanGrid = 148 * 2;  // upper bound on the persistent grid used for sizing

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

size_t bitlinear_batch_workspace_bytes(const bitlinear_problem* problems, int count) {
    if (!problems || count <= 0) return 0;
    size_t xq = 0, rows = 0;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.M < 0 || q.M > kGemvMaxTokens || !shape_ok(q.N, q.K) || q.K > kBatchMaxK) return 0;
        xq += align_up((size_t)q.M * q.K, 16);
        rows += (size_t)q.M;
    }
    return plan_layout(count, kPlanGrid, xq, rows).total;
}

int bitlinear_forward_batch(const bitlinear_problem* problems, int count, int flags, void* ws, size_t ws_bytes,
                            void* stream) {
    if (count < 0) return BITLINEAR_ERR_SHAPE;
    if (count == 0) return BITLINEAR_OK;
    if (!problems) return BITLINEAR_ERR_NULL;
    if (flags & ~(BITLINEAR_BATCH_REUSE_PLAN | BITLINEAR_BATCH_REUSE_ACT)) return BITLINEAR_ERR_DTYPE;
    size_t xq_bytes = 0, rows = 0;
    int max_m = 0, max_ktiles = 0, max_k = 0;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.y_dtype != BITLINEAR_F32 && q.y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
        if (q.M < 0 || q.M > kGemvMaxTokens || !shape_ok(q.N, q.K) || q.K > kBatchMaxK) return BITLINEAR_ERR_SHAPE;
        if (q.M == 0) continue;
        if (!q.x || !q.packed || !q.s_w || !q.y) return BITLINEAR_ERR_NULL;
        if (!aligned16(q.x) || !aligned16(q.packed) || !aligned16(q.y) || (q.gain && !aligned16(q.gain)) ||
            (reinterpret_cast<uintptr_t>(q.s_w) & 3u))
            return BITLINEAR_ERR_ALIGN;
        xq_bytes += align_up((size_t)q.M * q.K, 16);
        rows += (size_t)q.M;
        if (q.M > max_m) max_m = q.M;
        if (q.K / kTileCols > max_ktiles) max_ktiles = q.K / kTileCols;
        if (q.K > max_k) max_k = q.K;
    }
    const PlanLayout L = plan_layout(count, kPlanGrid, xq_bytes, rows);
    if (!ws || !aligned16(ws) || ws_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    if (rows == 0) return BITLINEAR_OK;

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        int major = 0;
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (major != 10) return BITLINEAR_ERR_ARCH;
        sm_count = n;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);

    // ---- host plan: device descriptors, item prefix, byte-balanced CTA ranges ----
    int rb_max = 1, stage_bytes = 0;
    std::vector<DevProblem> dp;
    std::vector<int> item_begin;
    dp.reserve(count);
    item_begin.reserve(count + 1);
    {
        char* xq_ptr = base + L.xq_off;
        float* d_ptr = reinterpret_cast<float*>(base + align_up(L.xq_off + xq_bytes, 256));
        int32_t* xs_ptr = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(d_ptr) + align_up(rows * sizeof(float), 256));
        int items = 0, row = 0;
        for (int i = 0; i < count; ++i) {
            const bitlinear_problem& q = problems[i];
            if (q.M == 0) continue;
            DevProblem v;
            v.packed = static_cast<const uint32_t*>(q.packed);
            v.s_w = q.s_w;
            v.y = q.y;
            v.x = static_cast<const __nv_bfloat16*>(q.x);
            v.gain = static_cast<const __nv_bfloat16*>(q.gain);
            v.xq = reinterpret_cast<int8_t*>(xq_ptr);
            v.d = d_ptr + row;
            v.xsum = xs_ptr + row;
            v.M = q.M; v.N = q.N; v.K = q.K; v.y_dtype = q.y_dtype;
            v.eps = q.rms_eps;
            v.k_tiles = q.K / kTileCols;
            {
                int rb = kItemBytesCap / (v.k_tiles * kTileBytes);
                const int rb_cap = max_m <= 8 ? 4 : 2;  // bounds the partial-sum buffers
                if (rb > rb_cap) rb = rb_cap;
                if (rb < 1) rb = 1;
                v.rb_per_item = rb;
                if (rb > rb_max) rb_max = rb;
                if (rb * v.k_tiles * kTileBytes > stage_bytes) stage_bytes = rb * v.k_tiles * kTileBytes;
            }
            v.item_begin = items;
            v.row_begin = row;
            dp.push_back(v);
            item_begin.push_back(items);
            items += (q.N / kTileRows + v.rb_per_item - 1) / v.rb_per_item;
            row += q.M;
            xq_ptr += align_up((size_t)q.M * q.K, 16);
        }
        item_begin.push_back(items);
    }
    const int n_prob = (int)dp.size();
    const int total_items = item_begin.back();
    int grid = sm_count < total_items ? sm_count : total_items;
    std::vector<int> cta_begin(grid + 1);
    {
        double total_bytes = 0.0;
        for (int i = 0; i < n_prob; ++i) total_bytes += (double)(item_begin[i + 1] - item_begin[i]) * dp[i].k_tiles * dp[i].rb_per_item;
        int pi = 0;
        double before = 0.0;  // tile-KB before problem pi
        cta_begin[0] = 0;
        for (int c = 1; c < grid; ++c) {
            const double target = total_bytes * c / grid;
            while (pi < n_prob - 1 &&
                   before + (double)(item_begin[pi + 1] - item_begin[pi]) * dp[pi].k_tiles * dp[pi].rb_per_item <= target) {
                before += (double)(item_begin[pi + 1] - item_begin[pi]) * dp[pi].k_tiles * dp[pi].rb_per_item;
                ++pi;
            }
            int it = item_begin[pi] + (int)((target - before) / ((double)dp[pi].k_tiles * dp[pi].rb_per_item) + 0.5);
            if (it > item_begin[pi + 1]) it = item_begin[pi + 1];
            if (it < cta_begin[c - 1]) it = cta_begin[c - 1];
            cta_begin[c] = it;
        }
        cta_begin[grid] = total_items;
    }

    PlanHeader hdr_host;
    hdr_host.magic = kPlanMagic;
    hdr_host.count = n_prob;
    hdr_host.total_items = total_items;
    hdr_host.grid = grid;
    hdr_host.rows = (int)rows;
    hdr_host.pad[0] = hdr_host.pad[1] = hdr_host.pad[2] = 0;
    if (!(flags & BITLINEAR_BATCH_REUSE_PLAN)) {
        if (cudaMemcpyAsync(base, &hdr_host, sizeof(hdr_host), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.probs_off, dp.data(), dp.size() * sizeof(DevProblem), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.item_off, item_begin.data(), item_begin.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.cta_off, cta_begin.data(), cta_begin.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
    }
    const DevProblem* probs_dev = reinterpret_cast<const DevProblem*>(base + L.probs_off);

    // ---- launch 1: quantise every token of every problem ----
    if (!(flags & BITLINEAR_BATCH_REUSE_ACT)) {
        const int vpt = (max_k / 8 + kQuantThreads - 1) / kQuantThreads;
        const dim3 g((unsigned)rows), b(kQuantThreads);
        const PlanHeader* h = reinterpret_cast<const PlanHeader*>(base);
        int* sw = device_status_word();
        if (vpt <= 1) batch_quant_kernel<1><<<g, b, 0, st>>>(h, probs_dev, n_prob, total_items, grid, sw);
        else if (vpt <= 2) batch_quant_kernel<2><<<g, b, 0, st>>>(h, probs_dev, n_prob, total_items, grid, sw);
        else batch_quant_kernel<4><<<g, b, 0, st>>>(h, probs_dev, n_prob, total_items, grid, sw);
        if (cudaGetLastError() != cudaSuccess) return BITLINEAR_ERR_CUDA;
    }

    // ---- launch 2: stream the weights ----
    StreamParams prm;
    prm.probs = probs_dev;
    prm.item_begin = reinterpret_cast<const int*>(base + L.item_off);
    prm.cta_begin = reinterpret_cast<const int*>(base + L.cta_off);
    prm.hdr = reinterpret_cast<const PlanHeader*>(base);
    prm.count = n_prob;
    prm.total_items = total_items;
    prm.rows = (int)rows;
    prm.status_word = device_status_word();
    const int nt = max_m <= 1 ? 0 : (max_m <= 8 ? 1 : 2);
    const int mp = nt == 0 ? 1 : 8 * nt;
    const int tpw = (max_ktiles + kConsumers - 1) / kConsumers;  // <= 4 since K <= 8192
    const size_t fixed = 1024 + (size_t)kRedBufs * rb_max * kConsumers * 16 * mp * sizeof(int) +
                         (2 * kMaxStages + 2 * kRedBufs) * 8 + 64;
    int stages = (int)((227 * 1024 - fixed) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    prm.stages = stages;
    prm.stage_bytes = stage_bytes;
    prm.rb_max = rb_max;
    const size_t smem = fixed + (size_t)stages * stage_bytes;
    cudaError_t e;
    if (nt == 0) e = launch_stream_nt<0>(tpw, prm, grid, smem, st);
    else if (nt == 1) e = launch_stream_nt<1>(tpw, prm, grid, smem, st);
    else e = launch_stream_nt<2>(tpw, prm, grid, smem, st);
    return e == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

int bitlinear_forward_batch_host(const bitlinear_problem* problems, int count, int flags, const void* x_host,
                                 void* x_dev, size_t x_bytes, const void* y_dev, void* y_host, size_t y_bytes, void* ws,
                                 size_t ws_bytes, void* stream) {
    if (count > 0 && (!x_host || !x_dev || !y_dev || !y_host)) return BITLINEAR_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (count > 0 && x_bytes > 0 && cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    const int rc = bitlinear_forward_batch(problems, count, flags, ws, ws_bytes, stream);
    if (rc != BITLINEAR_OK) return rc;
    if ((count > 0 && y_bytes > 0 && cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

}  // extern "C"
