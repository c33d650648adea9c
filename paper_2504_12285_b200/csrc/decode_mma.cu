// Batched decode for 5 to 16 tokens per matmul on the tensor cores.
// (Paper Section 5.1: packed weights are loaded from HBM into shared memory and unpacked there right before the
// product with the 8-bit activations.  With more than a few tokens the dot-product-of-four kernel is bound by its
// arithmetic - one instruction per token per four weights - so here the product runs on tcgen05.  The time of one
// tcgen05.mma grows with the rows of its A operand and hardly with its N, so the weights are the wide, stationary
// B operand: D[tokens (16 of M = 64 rows) x 256 weight rows] += A[tokens x 32 activations (s8)] x B[256 x 32 codes (u8)].)
//
// One persistent CTA per SM owns a contiguous, byte-balanced range of work items (256 weight rows of one matmul).
//   warp 0      epilogue : tcgen05.ld of the finished accumulator (token m in lane m; double buffered), minus the
//                          code sum, two fp32 multiplies, 16-byte stores
//   warp 1      producer : bulk copies of packed weights (sixteen 16-row blocks x up to two 16x256 tiles) and of the
//                          matching slice of the quantised tokens (16-row tile images) into a 2-slot ring
//   warp 2      MMA      : one thread issues 8 tcgen05.mma (64 x 256 x 32) per 256-column step and commits
//   warps 3-10  unpack   : warp w expands row blocks 2w and 2w+1 of the current 256-column step: 2-bit codes -> bytes,
//                          written as two 128-byte-swizzled K-major operand images of 256 rows (2 stages of 64 KiB)
// Every wait is bounded; on a timeout the CTA raises the sticky status word and leaves.
#include <algorithm>
#include <vector>

#include "quant_row.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

constexpr int kItemRb = 16;       // 16-row blocks per work item
constexpr int kItemRows = kItemRb * kTileRows;  // 256 weight rows = UMMA N
constexpr int kTok = 16;          // tokens per matmul, padded; the MMA computes 64 rows of which 16 are read
constexpr int kMmaM = 64;
constexpr int kStepTiles = 2;     // 16x256 tiles per row block per ring slot (512 columns)
constexpr int kUnpackWarps = 8;   // two row blocks each
constexpr int kEpiWarp = 0, kProdWarp = 1, kMmaWarp = 2, kFirstUnpackWarp = 3;
constexpr int kMmaThreads = (kFirstUnpackWarp + kUnpackWarps) * 32;
constexpr uint32_t kXSlot = kStepTiles * 2 * kTok * 128;              // 8 KiB: 4 k-blocks of 16 x 128 token images
constexpr uint32_t kPackedSlot = kItemRb * kStepTiles * kTileBytes;   // 32 KiB of packed weights
constexpr uint32_t kKbImage = kItemRows * 128;                        // 32 KiB: 256 rows x 128 codes
constexpr uint32_t kStage = 2 * kKbImage;                             // one 256-column step
constexpr int kStages = 2;
constexpr uint32_t kTmemCols = 2 * kItemRows;                         // two accumulators of 256 columns
constexpr size_t kMmaSmem = 1024 + 2 * (size_t)(kXSlot + kPackedSlot) + kStages * (size_t)kStage + 256;

struct MmaProblem {
    const uint8_t* packed;
    const uint8_t* x_img;  // quantised tokens as 16-row tile images, K / 128 images of 2 KiB
    const float* s_w;
    const float* d;
    const int32_t* xsum;
    void* y;
    const __nv_bfloat16* x;
    const __nv_bfloat16* gain;
    int8_t* xq_out;  // = x_img, for the quantiser launch
    float* d_out;
    int32_t* xsum_out;
    int M, N, K, y_dtype;
    float eps;
    int row_begin;  // first token in the global token list
    int pad[2];
};

struct MmaHeader {
    unsigned magic;
    int count, total_items, grid, rows;
    int pad[3];
};
constexpr unsigned kMmaMagic = 0xB171A9E7u;

struct MmaParams {
    const MmaHeader* hdr;
    const MmaProblem* probs;
    const int2* items;      // {problem, first row block of the item (a multiple of 16)}
    const int* cta_begin;   // [grid + 1]
    int count, total_items, rows;
    int* status_word;
};

__device__ __forceinline__ bool mma_plan_matches(const MmaHeader* h, int count, int total_items, int grid, int rows) {
    return h->magic == kMmaMagic && h->count == count && h->total_items == total_items && h->grid == grid && h->rows == rows;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Lane l of the warp receives 16 consecutive columns of tensor-memory lane (taddr lane + l).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// K-major operand tile with 128-byte rows and the 128-byte swizzle: 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    uint64_t desc = 0;
    desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    desc |= (uint64_t)1 << 16;
    desc |= (uint64_t)(1024 >> 4) << 32;
    desc |= (uint64_t)1 << 46;
    desc |= (uint64_t)2 << 61;
    return desc;
}
// D = s32, A = s8 (activations), B = u8 (weight codes), both K-major, M = 64, N = 256.
constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (0u << 10) | ((uint32_t)(kItemRows >> 3) << 17) | ((uint32_t)(kMmaM >> 4) << 24);

template <int VPT>
__global__ void __launch_bounds__(kQuantThreads) mma_quant_kernel(const MmaHeader* __restrict__ hdr,
                                                                  const MmaProblem* __restrict__ probs,
                                                                  const int* __restrict__ row_prob, int count, int total_items,
                                                                  int grid, int* status_word) {
    __shared__ RowReduceSmem sm;
    if (!mma_plan_matches(hdr, count, total_items, grid, (int)gridDim.x)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int row = blockIdx.x;
    const MmaProblem& p = probs[row_prob[row]];
    const int m = row - p.row_begin;
    quant_row<VPT, 3>(p.x + (size_t)m * p.K, p.gain, p.eps, p.K, p.xq_out + (size_t)m * 128, p.d_out + m, p.xsum_out + m, sm,
                      m & 7);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__global__ void __launch_bounds__(kMmaThreads, 1) decode_mma_kernel(const MmaParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // The token images come first: the MMA reads 64 operand rows where 16 are stored, and what it reads past them
    // (rows whose results nobody looks at) must still be this CTA's shared memory.
    const uint32_t x_s = smem_u32(smem);          // [2] token images
    const uint32_t p_s = x_s + 2 * kXSlot;        // [2] packed weights
    const uint32_t b_s = p_s + 2 * kPackedSlot;   // [kStages] operand images of the weights
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * (size_t)(kXSlot + kPackedSlot) + kStages * (size_t)kStage);
    const uint32_t pfull = smem_u32(bars + 0), pempty = smem_u32(bars + 2), xempty = smem_u32(bars + 4);
    const uint32_t tfull = smem_u32(bars + 6), tempty = smem_u32(bars + 8);
    const uint32_t bfull = smem_u32(bars + 10), bempty = smem_u32(bars + 10 + kStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10 + 2 * kStages);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!mma_plan_matches(prm.hdr, prm.count, prm.total_items, (int)gridDim.x, prm.rows)) {  // uniform over the grid
        if (blockIdx.x == 0 && threadIdx.x == 0 && prm.status_word != nullptr)
            atomicExch(prm.status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    if (threadIdx.x == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(pfull + 8 * b, 1);
            mbar_init(pempty + 8 * b, kUnpackWarps);
            mbar_init(xempty + 8 * b, 1);
            mbar_init(tfull + 8 * b, 1);
            mbar_init(tempty + 8 * b, 1);
        }
        for (int b = 0; b < kStages; ++b) {
            mbar_init(bfull + 8 * b, kUnpackWarps);
            mbar_init(bempty + 8 * b, 1);
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int item_lo = prm.cta_begin[blockIdx.x], item_hi = prm.cta_begin[blockIdx.x + 1];

    if (warp == kProdWarp) {
        // ------------------------------------------------------------------ producer
        uint32_t sc_idx = 0;
        bool ok = true;
        for (int it = item_lo; ok && it < item_hi; ++it) {
            const int2 item = prm.items[it];
            const MmaProblem& p = prm.probs[item.x];
            const int k_tiles = p.K / kTileCols, n_rb = min(kItemRb, p.N / kTileRows - item.y);
            const uint8_t* packed = p.packed;
            const uint8_t* x_img = p.x_img;
            for (int t0 = 0; t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                const int tiles = min(kStepTiles, k_tiles - t0);
                const uint32_t slot = sc_idx & 1u, phase = (sc_idx >> 1) & 1u;
                if (!mbar_wait(pempty + 8 * slot, phase ^ 1u, abort_flag) || !mbar_wait(xempty + 8 * slot, phase ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                if (lane == 0) mbar_expect_tx(pfull + 8 * slot, (uint32_t)(n_rb * tiles * kTileBytes + tiles * 2 * kTok * 128));
                __syncwarp();
                if (lane < n_rb)
                    bulk_load(p_s + slot * kPackedSlot + lane * (kStepTiles * kTileBytes),
                              packed + ((size_t)(item.y + lane) * k_tiles + t0) * kTileBytes, (uint32_t)tiles * kTileBytes,
                              pfull + 8 * slot);
                else if (lane == kItemRb)
                    bulk_load(x_s + slot * kXSlot, x_img + (size_t)t0 * 2 * kTok * 128, (uint32_t)tiles * 2 * kTok * 128,
                              pfull + 8 * slot);
            }
        }
    } else if (warp >= kFirstUnpackWarp) {
        // ------------------------------------------------------------------ unpack: warp w expands row blocks 2w, 2w+1
        const int w = warp - kFirstUnpackWarp;
        const int g = lane >> 2, t = lane & 3;
        // lanes of the upper k-block take their words in the order 2, 3, 0, 1: the eight lanes that store together
        // then hit eight different 16-byte bank groups
        const bool up = (t & 2) != 0;
        uint32_t sc_idx = 0, st_idx = 0;
        bool ok = true;
        for (int it = item_lo; ok && it < item_hi; ++it) {
            const int2 item = prm.items[it];
            const MmaProblem& p = prm.probs[item.x];
            const int k_tiles = p.K / kTileCols, n_rb = min(kItemRb, p.N / kTileRows - item.y);
            for (int t0 = 0; ok && t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                const int tiles = min(kStepTiles, k_tiles - t0);
                const uint32_t slot = sc_idx & 1u, phase = (sc_idx >> 1) & 1u;
                if (!mbar_wait(pfull + 8 * slot, phase, abort_flag)) { ok = false; break; }
                for (int kt = 0; kt < tiles; ++kt, ++st_idx) {
                    const uint32_t stage = st_idx % kStages, sphase = (st_idx / kStages) & 1u;
                    uint4 pv[2][2] = {};
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        if (2 * w + r < n_rb) {
                            const uint32_t src = p_s + slot * kPackedSlot + (uint32_t)(2 * w + r) * (kStepTiles * kTileBytes) +
                                                 (uint32_t)kt * kTileBytes + (uint32_t)lane * 16u;
                            pv[r][0] = lds128(src);
                            pv[r][1] = lds128(src + 512u);
                        }
                    }
                    if (!mbar_wait(bempty + 8 * stage, sphase ^ 1u, abort_flag)) { ok = false; break; }
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        if (2 * w + r < n_rb) {
                            // lane (g, t) holds rows g and 8+g of the 16-row block, columns 64t .. 64t+63 of the 256:
                            // k-block t >> 1, 16-byte pieces 4*(t & 1) + q of the 128-byte operand row
                            const uint32_t dst = b_s + stage * kStage + (uint32_t)(t >> 1) * kKbImage +
                                                 (uint32_t)((2 * w + r) * kTileRows + g) * 128u;
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint4 v4 = pv[r][h];
                                const uint32_t pw[4] = {up ? v4.z : v4.x, up ? v4.w : v4.y, up ? v4.x : v4.z, up ? v4.y : v4.w};
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const uint32_t v = pw[q];
                                    const uint32_t piece = (uint32_t)(4 * (t & 1) + (q ^ (t & 2))) ^ (uint32_t)g;  // row & 7 == g
                                    sts128(dst + 1024u * h + (piece << 4), v & 0x03030303u, (v >> 2) & 0x03030303u,
                                           (v >> 4) & 0x03030303u, (v >> 6) & 0x03030303u);
                                }
                            }
                        }
                    }
                    fence_async_smem();  // the tensor core reads these bytes through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bfull + 8 * stage);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(pempty + 8 * slot);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t sc_idx = 0, st_idx = 0, it_idx = 0;
            bool ok = true;
            for (int it = item_lo; ok && it < item_hi; ++it, ++it_idx) {
                const int2 item = prm.items[it];
                const int k_tiles = prm.probs[item.x].K / kTileCols;
                const uint32_t buf = it_idx & 1u, bphase = (it_idx >> 1) & 1u;
                if (!mbar_wait(tempty + 8 * buf, bphase ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kItemRows;
                for (int t0 = 0; ok && t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                    const int tiles = min(kStepTiles, k_tiles - t0);
                    const uint32_t slot = sc_idx & 1u, phase = (sc_idx >> 1) & 1u;
                    if (!mbar_wait(pfull + 8 * slot, phase, abort_flag)) { ok = false; break; }  // the token images landed
                    for (int kt = 0; kt < tiles; ++kt, ++st_idx) {
                        const uint32_t stage = st_idx % kStages, sphase = (st_idx / kStages) & 1u;
                        if (!mbar_wait(bfull + 8 * stage, sphase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int kb = 0; kb < 2; ++kb) {
                            const uint64_t a_desc = smem_desc_sw128(x_s + slot * kXSlot + (uint32_t)(kt * 2 + kb) * (kTok * 128));
                            const uint64_t b_desc = smem_desc_sw128(b_s + stage * kStage + (uint32_t)kb * kKbImage);
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_i8(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), kIdesc,
                                        (uint32_t)((t0 | kt | kb | k) != 0));
                        }
                        umma_commit(bempty + 8 * stage);  // the stage may be rewritten once these MMAs retire
                    }
                    if (ok) umma_commit(xempty + 8 * slot);
                }
                if (ok) umma_commit(tfull + 8 * buf);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (warp 0: tensor-memory lanes 0 .. 31)
        uint32_t it_idx = 0;
        for (int it = item_lo; it < item_hi; ++it, ++it_idx) {
            const int2 item = prm.items[it];
            const MmaProblem& p = prm.probs[item.x];
            const int M = p.M, N = p.N, y_dtype = p.y_dtype;
            const float s_w = *p.s_w;
            const bool live = lane < M;  // accumulator row m of the 64 sits in tensor-memory lane m for m < 16
            const int xs = live ? p.xsum[lane] : 0;
            const float dm = live ? p.d[lane] : 0.0f;
            float* y32 = reinterpret_cast<float*>(p.y) + (size_t)lane * N;
            __nv_bfloat16* y16 = reinterpret_cast<__nv_bfloat16*>(p.y) + (size_t)lane * N;
            const uint32_t buf = it_idx & 1u, bphase = (it_idx >> 1) & 1u;
            if (!mbar_wait(tfull + 8 * buf, bphase, abort_flag)) break;
            tc_fence_after();
            for (int c = 0; c < kItemRb; ++c) {
                const int n0 = (item.y + c) * kTileRows;  // first weight row of these 16 columns
                if (n0 >= N) break;
                uint32_t r[16];
                tmem_ld_32x16(tmem_base + buf * kItemRows + (uint32_t)c * kTileRows, r);
                if (live) {
                    float v[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(__fmul_rn((float)((int)r[j] - xs), s_w), dm);
                    if (y_dtype == BITLINEAR_BF16) {
                        uint32_t h[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                            h[j] = *reinterpret_cast<const uint32_t*>(&b2);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(y16 + n0);
                        dst[0] = make_uint4(h[0], h[1], h[2], h[3]);
                        dst[1] = make_uint4(h[4], h[5], h[6], h[7]);
                    } else {
                        float4* dst = reinterpret_cast<float4*>(y32 + n0);
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty + 8 * buf);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        abort_drain();
        if (threadIdx.x == 0 && prm.status_word != nullptr) atomicExch(prm.status_word, BITLINEAR_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

namespace {

struct MmaLayout {
    size_t probs_off, items_off, cta_off, row_prob_off, x_off, d_off, xsum_off, total;
};

constexpr int kMmaPlanGrid = 148 * 2;  // upper bound on the persistent grid used for sizing

MmaLayout mma_layout(const bitlinear_problem* problems, int count) {
    MmaLayout L;
    size_t items = 0, rows = 0, x_bytes = 0;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.M <= 0) continue;
        items += (size_t)(q.N / kTileRows + kItemRb - 1) / kItemRb;
        rows += (size_t)q.M;
        x_bytes += (size_t)kTok * q.K;  // K / 128 images of 16 rows x 128 codes
    }
    size_t off = 256;  // the MmaHeader sits at offset 0
    L.probs_off = off;
    off = align_up(off + (size_t)count * sizeof(MmaProblem), 256);
    L.items_off = off;
    off = align_up(off + (items + 1) * sizeof(int2), 256);
    L.cta_off = off;
    off = align_up(off + (size_t)(kMmaPlanGrid + 1) * sizeof(int), 256);
    L.row_prob_off = off;
    off = align_up(off + (rows + 1) * sizeof(int), 1024);
    L.x_off = off;
    off = align_up(off + x_bytes, 256);
    L.d_off = off;
    off = align_up(off + rows * sizeof(float), 256);
    L.xsum_off = off;
    off = align_up(off + rows * sizeof(int32_t), 256);
    L.total = off;
    return L;
}

}  // namespace

size_t decode_mma_workspace_bytes(const bitlinear_problem* problems, int count) { return mma_layout(problems, count).total; }

// Problems are validated by the caller (1 <= M <= 16 or M == 0, shapes, pointers, alignment).
int decode_mma_forward(const bitlinear_problem* problems, int count, int flags, void* ws, size_t ws_bytes, void* stream) {
    const MmaLayout L = mma_layout(problems, count);
    if (!ws || !aligned16(ws) || ws_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, n = 0, major = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        if (major != 10) return BITLINEAR_ERR_ARCH;
        if (cudaFuncSetAttribute(decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        sm_count = n;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);

    // ---- host plan: descriptors, work items of 256 weight rows, token -> problem table, balanced CTA ranges ----
    std::vector<MmaProblem> mp;
    std::vector<int2> items;
    std::vector<double> weight;  // packed tiles of each item
    std::vector<int> row_prob;
    int max_k = 0;
    {
        uint8_t* x_ptr = reinterpret_cast<uint8_t*>(base + L.x_off);
        float* d_ptr = reinterpret_cast<float*>(base + L.d_off);
        int32_t* xs_ptr = reinterpret_cast<int32_t*>(base + L.xsum_off);
        int row = 0;
        for (int i = 0; i < count; ++i) {
            const bitlinear_problem& q = problems[i];
            if (q.M <= 0) continue;
            MmaProblem v = {};
            v.packed = static_cast<const uint8_t*>(q.packed);
            v.x_img = x_ptr;
            v.s_w = q.s_w;
            v.d = d_ptr + row;
            v.xsum = xs_ptr + row;
            v.y = q.y;
            v.x = static_cast<const __nv_bfloat16*>(q.x);
            v.gain = static_cast<const __nv_bfloat16*>(q.gain);
            v.xq_out = reinterpret_cast<int8_t*>(x_ptr);
            v.d_out = d_ptr + row;
            v.xsum_out = xs_ptr + row;
            v.M = q.M; v.N = q.N; v.K = q.K; v.y_dtype = q.y_dtype;
            v.eps = q.rms_eps;
            v.row_begin = row;
            const int n_rb = q.N / kTileRows;
            for (int rb = 0; rb < n_rb; rb += kItemRb) {
                items.push_back(make_int2((int)mp.size(), rb));
                weight.push_back((double)std::min(kItemRb, n_rb - rb) * (q.K / kTileCols));
            }
            for (int m = 0; m < q.M; ++m) row_prob.push_back((int)mp.size());
            mp.push_back(v);
            row += q.M;
            x_ptr += (size_t)kTok * q.K;
            if (q.K > max_k) max_k = q.K;
        }
        row_prob.push_back(0);
    }
    const int rows = (int)row_prob.size() - 1;
    if (rows == 0) return BITLINEAR_OK;
    const int n_prob = (int)mp.size(), total_items = (int)items.size();
    const int grid = std::min(std::min(sm_count, kMmaPlanGrid), total_items);
    std::vector<int> cta_begin(grid + 1);
    {
        double total = 0.0;
        for (double w : weight) total += w;
        int it = 0;
        double before = 0.0;  // weight of the items before it
        cta_begin[0] = 0;
        for (int c = 1; c < grid; ++c) {
            const double target = total * c / grid;
            while (it < total_items && before + 0.5 * weight[it] <= target) before += weight[it++];
            cta_begin[c] = std::max(it, cta_begin[c - 1]);
        }
        cta_begin[grid] = total_items;
    }

    MmaHeader hdr_host = {};
    hdr_host.magic = kMmaMagic;
    hdr_host.count = n_prob;
    hdr_host.total_items = total_items;
    hdr_host.grid = grid;
    hdr_host.rows = rows;
    if (!(flags & BITLINEAR_BATCH_REUSE_PLAN)) {
        if (cudaMemcpyAsync(base, &hdr_host, sizeof(hdr_host), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.probs_off, mp.data(), mp.size() * sizeof(MmaProblem), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.items_off, items.data(), items.size() * sizeof(int2), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.cta_off, cta_begin.data(), cta_begin.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.row_prob_off, row_prob.data(), row_prob.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
    }
    const MmaHeader* hdr = reinterpret_cast<const MmaHeader*>(base);
    const MmaProblem* probs_dev = reinterpret_cast<const MmaProblem*>(base + L.probs_off);
    int* sw = device_status_word();

    // ---- launch 1: quantise every token into the 16-row tile images ----
    if (!(flags & BITLINEAR_BATCH_REUSE_ACT)) {
        const int vpt = (max_k / 8 + kQuantThreads - 1) / kQuantThreads;
        const dim3 g((unsigned)rows), b(kQuantThreads);
        const int* rp = reinterpret_cast<const int*>(base + L.row_prob_off);
        if (vpt <= 1) mma_quant_kernel<1><<<g, b, 0, st>>>(hdr, probs_dev, rp, n_prob, total_items, grid, sw);
        else if (vpt <= 2) mma_quant_kernel<2><<<g, b, 0, st>>>(hdr, probs_dev, rp, n_prob, total_items, grid, sw);
        else mma_quant_kernel<4><<<g, b, 0, st>>>(hdr, probs_dev, rp, n_prob, total_items, grid, sw);
        if (cudaGetLastError() != cudaSuccess) return BITLINEAR_ERR_CUDA;
    }

    // ---- launch 2: stream the weights through the tensor cores ----
    MmaParams prm;
    prm.hdr = hdr;
    prm.probs = probs_dev;
    prm.items = reinterpret_cast<const int2*>(base + L.items_off);
    prm.cta_begin = reinterpret_cast<const int*>(base + L.cta_off);
    prm.count = n_prob;
    prm.total_items = total_items;
    prm.rows = rows;
    prm.status_word = sw;
    decode_mma_kernel<<<grid, kMmaThreads, kMmaSmem, st>>>(prm);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

}  // namespace bitlinear
