// Batched decode for 2 to 16 tokens per matmul on the tensor cores.
// (Paper Section 5.1: packed weights are loaded from HBM into shared memory and unpacked right before the product
// with the 8-bit activations.  With more than a few tokens the dot-product-of-four kernel is bound by its arithmetic
// - one instruction per token per four weights - so here the product runs on tcgen05:
// D[128 weight rows x 16 tokens] += A[128 x 32 weight codes (u8)] x B[16 x 32 activations (s8)].
// The unpacked codes never touch shared memory: each unpack thread owns one weight row, expands its 2-bit codes in
// registers and stores them with tcgen05.st into tensor memory, from where the MMA takes its A operand; shared
// memory only carries the packed bytes and the token images, so the copy ring can be deep.)
//
// One persistent CTA per SM owns a contiguous, byte-balanced range of work items (128 weight rows of one matmul).
// Launch 1 (mma_quant_kernel, one warp per token) writes the quantised tokens as 16-row tile images; launch 2
// (decode_mma_kernel) is its programmatic dependent: only the threads that read launch 1's results wait for it, so
// where an SM has room for a CTA of launch 2 beside launch 1 (it needs almost all registers) the weights already flow.
//   producer warps : three warps, three bulk copies each (a thread starts a copy only every few hundred cycles):
//                    eight packed 16-row blocks x up to four 16x256 tiles (4 KiB each) and the matching slice of
//                    the token images, into a 4-slot ring of 48 KiB
// Tile g of every ring slot belongs to pipeline g (kLanes = 4 pipelines), each with its own unpack group, its own 64
// tensor-memory columns for the codes, its own MMA-issuing thread and its own partial accumulator (one thread can
// start a tcgen05.mma only every ~55 cycles whatever its shape, several threads scale; the integer partial sums are
// added in the epilogue, exactly):
//   unpack groups  : four warps each, the warp of tensor-memory lane quarter q expands weight rows 32q .. 32q+31
//                    (thread = row) into the pipeline's 64 columns, as 64 x code so that a left shift and one AND do
//   MMA warps      : one thread each issues the 8 tcgen05.mma (128 x 16 x 32, A from tensor memory) of a step
//   epilogue warps : tcgen05.ld of the finished partial accumulators (double buffered), their sum / 64 minus the
//                    code sum, two fp32 multiplies, stores coalesced along the weight rows
// The work items and matmul descriptors of the CTA are copied to shared memory first.
// Every wait is bounded; on a timeout the CTA raises the sticky status word and leaves.
#include <algorithm>
#include <vector>

#include "quant_row.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

constexpr int kRows = 128;        // weight rows per work item = tensor-memory lanes = UMMA M
constexpr int kItemRb = kRows / kTileRows;
constexpr int kTok = 16;          // tokens per matmul, padded (UMMA N)
constexpr int kStepTiles = 4;     // 16x256 tiles per row block per ring slot (1024 columns): one per pipeline
constexpr int kSlots = 4;         // ring slots of packed weights + token images (48 KiB each)
constexpr int kLanes = 4;         // pipelines: unpack group + tensor-memory stage(s) + MMA issuer + partial accumulator
// Code stages per pipeline.  Measured with three pipelines of two private stages each (the group expands step s + 1 while
// the MMAs of step s run; 3 tiles per slot, 5 slots): 155.5 / 168.8 us per 521 MB step at 4 / 16 tokens, against
// 140.8 / 156.2 us on the same GPU for four pipelines of one stage: the stage is not what the roles wait for.
constexpr int kAStages = 1;
constexpr int kUnpackWarps = 4 * kLanes;  // groups of four (one warp per tensor-memory lane quarter)
constexpr int kProdWarps = 3, kCopiesPerWarp = 3;  // 8 packed row blocks + the token images
constexpr int kFirstMmaWarp = kProdWarps + kUnpackWarps;
constexpr int kFirstEpiWarp = kFirstMmaWarp + kLanes;
constexpr int kMmaThreads = (kFirstEpiWarp + 4) * 32;
constexpr uint32_t kPackedSlot = kItemRb * kStepTiles * kTileBytes;  // 32 KiB of packed weights
constexpr uint32_t kXSlot = kStepTiles * 2 * kTok * 128;             // 16 KiB: 8 k-blocks of 16 x 128 token images
constexpr uint32_t kAStageCols = kTileCols / 4;                      // 64 columns: 256 codes per row, 4 per column
constexpr uint32_t kAColBase = 2 * kLanes * kTok;                    // after the two buffers of partial accumulators
constexpr uint32_t kTmemCols = 512;                                  // power of two >= kAColBase + kLanes * kAStages * 64
static_assert(kAColBase + kLanes * kAStages * kAStageCols <= kTmemCols, "tensor memory");
constexpr int kItemCap = 192;     // work items and matmul descriptors of the CTA kept in shared memory; what does
constexpr int kProbCap = 48;      // not fit is read from global memory where it is needed (slow, still correct)

struct MmaProblem {
    const uint8_t* packed;
    const uint8_t* x_img;  // quantised tokens as 16-row tile images, K / 128 images of 2 KiB
    const float* s_w;
    const float* d;
    const int32_t* xsum;
    void* y;
    const void* x;   // first operand of the input step (see RowOp)
    const __nv_bfloat16* gain;
    RowOp op;        // the element-wise step in front of the quantiser
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
    const int2* items;      // {problem, first row block of the item (a multiple of 8)}
    const int* cta_begin;   // [grid + 1]
    int count, total_items, rows;
    int* status_word;
};

// What the kernel's roles need of a matmul, copied to shared memory once: a descriptor fetched from global memory
// at every item boundary costs two dependent loads at loaded-HBM latency in every role, and the pipeline drains.
struct alignas(16) SProb {
    const uint8_t* packed;
    const uint8_t* x_img;
    const float* s_w;
    const float* d;
    const int32_t* xsum;
    void* y;
    int M, N, K, y_dtype;
};
constexpr int kNumBars = 3 * kSlots + 2 * kLanes * kAStages + 4;    // pfull, pempty, xempty; afull, aempty; tfull, tempty
constexpr size_t kBarBytes = 256;                                    // barriers, tensor-memory base, abort flag
static_assert(kNumBars * 8 + 8 <= kBarBytes, "barrier block");
constexpr size_t kMmaSmem = 1024 + kSlots * (size_t)(kPackedSlot + kXSlot) + kBarBytes + kItemCap * sizeof(int2) + kProbCap * sizeof(SProb);

__device__ __forceinline__ SProb load_prob(const MmaProblem& q) {
    SProb v;
    v.packed = q.packed; v.x_img = q.x_img; v.s_w = q.s_w; v.d = q.d; v.xsum = q.xsum; v.y = q.y;
    v.M = q.M; v.N = q.N; v.K = q.K; v.y_dtype = q.y_dtype;
    return v;
}

__device__ __forceinline__ bool mma_plan_matches(const MmaHeader* h, int count, int total_items, int grid, int rows) {
    return h->magic == kMmaMagic && h->count == count && h->total_items == total_items && h->grid == grid && h->rows == rows;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// A operand in tensor memory (lane = row, four 8-bit codes per 32-bit column), B operand in shared memory.
__device__ __forceinline__ void umma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Lane l of the warp writes 32 consecutive columns of tensor-memory lane (taddr lane + l).
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
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
// D = s32, A = u8 (64 x weight code, tensor memory), B = s8 (activations, K-major shared memory), M = 128, N = 16.
constexpr uint32_t kIdesc = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(kTok >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);

// One CTA per token, the row kept in registers (one read of the input): for calls with so few tokens that they do not
// even give every SM a CTA - a level of a decoder layer at 2 to 16 tokens - where the latency of a token's chain is all
// that counts.
template <int VPT>
__global__ void __launch_bounds__(kQuantThreads) mma_quant_row_kernel(const MmaHeader* __restrict__ hdr,
                                                                      const MmaProblem* __restrict__ probs,
                                                                      const int* __restrict__ row_prob, int count, int total_items,
                                                                      int grid, int rows, int* status_word) {
    __shared__ RowReduceSmem sm;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // see mma_quant_kernel
    if (!mma_plan_matches(hdr, count, total_items, grid, rows)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int row = blockIdx.x;
    const MmaProblem& p = probs[row_prob[row]];
    const int m = row - p.row_begin;
    with_row_source(p.op, p.x, m, p.K, [&](auto src) {
        quant_row_src<VPT, 3>(src, p.gain, p.eps, p.K, p.xq_out + (size_t)m * 128, p.d_out + m, p.xsum_out + m, sm, m & 7);
    });
}

// kQuantGroupWarps warps per token: there are at most a few thousand tokens here, and with one warp per token a
// 6,912-element token is a serial chain of thousands of instructions for its warp while most of the GPU idles.
// (Four warps per token while that still fits one wave of CTAs, two beyond.)
template <int kQuantGroupWarps>
__global__ void __launch_bounds__(kQuantThreads) mma_quant_kernel(const MmaHeader* __restrict__ hdr,
                                                                  const MmaProblem* __restrict__ probs,
                                                                  const int* __restrict__ row_prob, int count, int total_items,
                                                                  int grid, int rows, int* status_word) {
    constexpr int kQuantGroups = kQuantWarps / kQuantGroupWarps;  // tokens per CTA
    __shared__ GroupReduceSmem sm[kQuantGroups];
    // the kernel that follows may start now: it fetches weights first and waits for this grid before it reads
    // anything written here (programmatic dependent launch)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // this launch is itself a programmatic dependent of whatever runs before it on the stream (its launch overlaps that
    // kernel's tail); nothing is read before that kernel is complete
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!mma_plan_matches(hdr, count, total_items, grid, rows)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int group = threadIdx.x / (32 * kQuantGroupWarps);
    const int row = blockIdx.x * kQuantGroups + group;
    if (row >= rows) return;  // the whole group leaves: nobody is left waiting at its barrier
    const MmaProblem& p = probs[row_prob[row]];
    const int m = row - p.row_begin;
    with_row_source(p.op, p.x, m, p.K, [&](auto src) {
        quant_row_group_src<3, kQuantGroupWarps>(src, p.gain, p.eps, p.K, p.xq_out + (size_t)m * 128, p.d_out + m,
                                                 p.xsum_out + m, sm[group], 1 + group, m & 7);
    });
}

// 2 x 16 packed bytes (128 codes of one weight row) -> 32 tensor-memory columns of 64 x code.
__device__ __forceinline__ void expand_codes(const uint4& qa, const uint4& qb, uint32_t (&v)[32]) {
    const uint32_t w8[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[4 * i + j] = (w8[i] * (64u >> (2 * j))) & 0xC0C0C0C0u;
    }
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__global__ void __launch_bounds__(kMmaThreads, 1) decode_mma_kernel(const MmaParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t x_s = smem_u32(smem);            // [kSlots] token images
    const uint32_t p_s = x_s + kSlots * kXSlot;     // [kSlots] packed weights
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kSlots * (size_t)(kXSlot + kPackedSlot));
    const uint32_t pfull = smem_u32(bars), pempty = pfull + 8 * kSlots, xempty = pempty + 8 * kSlots;
    const uint32_t afull = xempty + 8 * kSlots, aempty = afull + 8 * kLanes * kAStages;  // [pipeline][stage]
    const uint32_t tfull = aempty + 8 * kLanes * kAStages, tempty = tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int2* items_s = reinterpret_cast<int2*>(reinterpret_cast<uint8_t*>(bars) + kBarBytes);
    SProb* probs_s = reinterpret_cast<SProb*>(items_s + kItemCap);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!mma_plan_matches(prm.hdr, prm.count, prm.total_items, (int)gridDim.x, prm.rows)) {  // uniform over the grid
        if (blockIdx.x == 0 && threadIdx.x == 0 && prm.status_word != nullptr)
            atomicExch(prm.status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    if (threadIdx.x == 0) {
        for (int b = 0; b < kSlots; ++b) {
            mbar_init(pfull + 8 * b, kProdWarps);
            mbar_init(pempty + 8 * b, kUnpackWarps);
            mbar_init(xempty + 8 * b, kLanes);
        }
        for (int b = 0; b < kLanes * kAStages; ++b) {
            mbar_init(afull + 8 * b, 4);
            mbar_init(aempty + 8 * b, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull + 8 * b, kLanes);
            mbar_init(tempty + 8 * b, 4);
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == kFirstMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const int item_lo = prm.cta_begin[blockIdx.x], item_hi = prm.cta_begin[blockIdx.x + 1];
    const int prob_lo = item_lo < item_hi ? prm.items[item_lo].x : 0;  // items are sorted by matmul
    for (int i = threadIdx.x; i < min(item_hi - item_lo, kItemCap); i += kMmaThreads) items_s[i] = prm.items[item_lo + i];
    for (int i = threadIdx.x; i < min(prm.count - prob_lo, kProbCap); i += kMmaThreads) probs_s[i] = load_prob(prm.probs[prob_lo + i]);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // item it of this CTA and its matmul, from shared memory when cached
    auto item_at = [&](int it) -> int2 { return it - item_lo < kItemCap ? items_s[it - item_lo] : prm.items[it]; };
    auto prob_at = [&](int pi) -> SProb { return pi - prob_lo < kProbCap ? probs_s[pi - prob_lo] : load_prob(prm.probs[pi]); };

    if (warp < kProdWarps) {
        // ------------------------------------------------------------------ producers: three copies per warp
        // (a thread starts a bulk copy only every ~200 cycles, and the lanes of a warp take turns)
        const int c = warp * kCopiesPerWarp + lane;  // copy 0 .. 7: packed row block c of the item; copy 8: token images
        // the token images are written by the quantiser launch before this kernel; the weights are not
        if (c == kItemRb) asm volatile("griddepcontrol.wait;" ::: "memory");
        uint32_t sc_idx = 0;
        bool ok = true;
        for (int it = item_lo; ok && it < item_hi; ++it) {
            const int2 item = item_at(it);
            const SProb p = prob_at(item.x);
            const int k_tiles = p.K / kTileCols, n_rb = min(kItemRb, p.N / kTileRows - item.y);
            const uint8_t* src_row = p.packed + (size_t)(item.y + c) * k_tiles * kTileBytes;
            for (int t0 = 0; t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                const int tiles = min(kStepTiles, k_tiles - t0);
                const uint32_t slot = sc_idx % kSlots, phase = (sc_idx / kSlots) & 1u;
                if (!mbar_wait(pempty + 8 * slot, phase ^ 1u, abort_flag) || !mbar_wait(xempty + 8 * slot, phase ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                if (lane == 0) {  // this warp's share of the slot's bytes
                    const int c0 = warp * kCopiesPerWarp;
                    const int n_packed = max(0, min(n_rb, c0 + kCopiesPerWarp) - c0);
                    const int has_x = (c0 <= kItemRb && kItemRb < c0 + kCopiesPerWarp) ? 1 : 0;
                    mbar_expect_tx(pfull + 8 * slot, (uint32_t)(n_packed * tiles * kTileBytes + has_x * tiles * 2 * kTok * 128));
                }
                __syncwarp();
                if (lane < kCopiesPerWarp) {
                    if (c < n_rb)
                        bulk_load_once(p_s + slot * kPackedSlot + c * (kStepTiles * kTileBytes), src_row + (size_t)t0 * kTileBytes,
                                       (uint32_t)tiles * kTileBytes, pfull + 8 * slot, l2_evict_first_policy());  // weights: read once
                    else if (c == kItemRb)
                        bulk_load(x_s + slot * kXSlot, p.x_img + (size_t)t0 * 2 * kTok * 128, (uint32_t)tiles * 2 * kTok * 128,
                                  pfull + 8 * slot);
                }
            }
        }
    } else if (warp < kFirstMmaWarp) {
        // ------------------------------------------------------------------ unpack: one thread per weight row
        const int quarter = warp & 3;                   // tensor-memory lanes 32*quarter .. +31 are the ones this warp may touch
        const int g = (warp - kProdWarps) >> 2;         // this warp's pipeline: tile g of every slot
        const int rbl = 2 * quarter + (lane >> 4), r16 = lane & 15;  // row block of the item, row inside it
        // the 256 codes of row r16 = 8h + g of a 16 x 256 tile are 64 consecutive packed bytes at 512h + 64g
        const uint32_t row_off = (uint32_t)rbl * (kStepTiles * kTileBytes) + (uint32_t)(r16 >> 3) * 512u + (uint32_t)(r16 & 7) * 64u +
                                 (uint32_t)g * kTileBytes;
        const uint32_t a_dst0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + kAColBase + (uint32_t)g * kAStages * kAStageCols;
        uint32_t sc_idx = 0, n_own = 0;
        bool ok = true;
        for (int it = item_lo; ok && it < item_hi; ++it) {
            const int2 item = item_at(it);
            const SProb p = prob_at(item.x);
            const int k_tiles = p.K / kTileCols;
            const bool have_row = rbl < min(kItemRb, p.N / kTileRows - item.y);
            for (int t0 = 0; t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                const uint32_t slot = sc_idx % kSlots, phase = (sc_idx / kSlots) & 1u;
                // every warp waits for every slot, also one in which it has no step: a warp can then never be a whole
                // ring lap ahead of another and arrive twice on pempty in one phase
                if (!mbar_wait(pfull + 8 * slot, phase, abort_flag)) { ok = false; break; }
                if (g < k_tiles - t0) {
                    uint4 pw[4] = {};
                    if (have_row) {
                        const uint32_t src = p_s + slot * kPackedSlot + row_off;
#pragma unroll
                        for (int t = 0; t < 4; ++t) pw[t] = lds128(src + 16u * t);
                    }
                    // word i of piece t, bit plane j, byte b = column 64t + 16i + 4j + b: tensor-memory column 16t + 4i + j.
                    // The 2-bit codes are moved to the TOP of their bytes (value 64 * code, still an unsigned byte):
                    // that takes a left shift, which the multiplier pipe executes, and one AND, where a right shift
                    // and an AND would both go to the logic pipe; the epilogue divides by 64.
                    // The first half is expanded BEFORE the wait for the tensor-memory stage (the MMAs of the
                    // pipeline's previous step are still reading it), the second half after the first is stored.
                    uint32_t v[32];
                    expand_codes(pw[0], pw[1], v);
                    // the pipeline's steps alternate between its two code stages: stage st is free once the MMAs of the
                    // step before last have retired
                    const uint32_t st = n_own % kAStages, a_dst = a_dst0 + st * kAStageCols;
                    if (!mbar_wait(aempty + 8 * (g * kAStages + st), ((n_own / kAStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    tmem_st_32x32(a_dst, v);
                    expand_codes(pw[2], pw[3], v);
                    tmem_st_32x32(a_dst + 32u, v);
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(afull + 8 * (g * kAStages + st));
                    ++n_own;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(pempty + 8 * slot);
            }
        }
    } else if (warp < kFirstEpiWarp) {
        // ------------------------------------------------------------------ MMA issuers: one pipeline each
        if (lane == 0) {
            const int g = warp - kFirstMmaWarp;
            const uint32_t a_tmem0 = tmem_base + kAColBase + (uint32_t)g * kAStages * kAStageCols;
            // token images of tile g of a slot: k-block kb at 2 KiB * (2g + kb), 32-byte slice k inside it
            const uint64_t x_desc = smem_desc_sw128(x_s) + (uint64_t)((g * 2 * kTok * 128) >> 4);
            uint32_t sc_idx = 0, n_own = 0, it_idx = 0;
            bool ok = true;
            for (int it = item_lo; ok && it < item_hi; ++it, ++it_idx) {
                const int k_tiles = prob_at(item_at(it).x).K / kTileCols;
                const uint32_t buf = it_idx & 1u;
                if (!mbar_wait(tempty + 8 * buf, ((it_idx >> 1) & 1u) ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (buf * kLanes + (uint32_t)g) * kTok;
                for (int t0 = 0; t0 < k_tiles; t0 += kStepTiles, ++sc_idx) {
                    const uint32_t slot = sc_idx % kSlots, phase = (sc_idx / kSlots) & 1u;
                    // every issuer waits for every slot, also one in which it has no step (see the unpack warps)
                    if (!mbar_wait(pfull + 8 * slot, phase, abort_flag)) { ok = false; break; }
                    if (g < k_tiles - t0) {
                        const uint32_t st = n_own % kAStages, a_tmem = a_tmem0 + st * kAStageCols;
                        if (!mbar_wait(afull + 8 * (g * kAStages + st), (n_own / kAStages) & 1u, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t b_desc = x_desc + (uint64_t)(slot * (kXSlot >> 4));
#pragma unroll
                        for (int s = 0; s < 8; ++s)
                            umma_i8_ts(d_tmem, a_tmem + 8u * s, b_desc + (uint64_t)((s >> 2) * ((kTok * 128) >> 4) + 2 * (s & 3)),
                                       kIdesc, (uint32_t)(t0 != 0 || s != 0));
                        umma_commit(aempty + 8 * (g * kAStages + st));  // the stage may be overwritten once these MMAs retire
                        ++n_own;
                    }
                    umma_commit(xempty + 8 * slot);  // counts kLanes arrivals: every issuer is done with the slot
                }
                if (ok) umma_commit(tfull + 8 * buf);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;  // tensor-memory lanes 32*quad .. 32*quad+31 belong to this warp
        asm volatile("griddepcontrol.wait;" ::: "memory");  // scales and code sums come from the quantiser launch
        uint32_t it_idx = 0;
        for (int it = item_lo; it < item_hi; ++it, ++it_idx) {
            const int2 item = item_at(it);
            const SProb p = prob_at(item.x);
            const int M = p.M, N = p.N, y_dtype = p.y_dtype;
            const int k_tiles = p.K / kTileCols;
            void* y = p.y;
            const float s_w = *p.s_w;
            const int xs_lane = lane < M ? p.xsum[lane] : 0;
            const float d_tok = lane < M ? p.d[lane] : 0.0f;
            const uint32_t buf = it_idx & 1u, bphase = (it_idx >> 1) & 1u;
            if (!mbar_wait(tfull + 8 * buf, bphase, abort_flag)) break;
            tc_fence_after();
            // the pipelines that had a step in this item hold its partial sums (integers: any order, same total)
            const uint32_t d_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kLanes * kTok;
            uint32_t r[16];
            tmem_ld_32x16(d_lane, r);
            for (int j = 1; j < min(kLanes, k_tiles); ++j) {
                uint32_t r2[16];
                tmem_ld_32x16(d_lane + (uint32_t)j * kTok, r2);
#pragma unroll
                for (int m = 0; m < kTok; ++m) r[m] += r2[m];
            }
#pragma unroll
            for (int m = 0; m < kTok; ++m) r[m] = (uint32_t)((int)r[m] >> 6);  // exact: the sums are multiples of 64
            const int n = item.y * kTileRows + quad * 32 + lane;  // this lane's weight row
#pragma unroll
            for (int m = 0; m < kTok; ++m) {
                const int xs = __shfl_sync(0xffffffffu, xs_lane, m);
                const float dm = __shfl_sync(0xffffffffu, d_tok, m);
                if (m < M && n < N) {
                    const float val = __fmul_rn(__fmul_rn((float)((int)r[m] - xs), s_w), dm);
                    const size_t idx = (size_t)m * N + n;
                    if (y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(val);
                    else reinterpret_cast<float*>(y)[idx] = val;
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
    if (warp == kFirstMmaWarp) {
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
    int sm_count = 0;
    if (const int rc = device_sm_count(&sm_count)) return rc;
    // the attribute is per device and cheap to set: done on every call, like the streaming kernel's launcher does
    if (cudaFuncSetAttribute(decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMmaSmem) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);

    // ---- host plan: descriptors, work items of 128 weight rows, token -> problem table, balanced CTA ranges ----
    std::vector<MmaProblem> mp;
    std::vector<int2> items;
    std::vector<double> weight;  // packed tiles of each item
    std::vector<int> row_prob;
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
            v.x = q.x;
            v.op.x2 = q.x2; v.op.x_out = q.x_out; v.op.op = q.x_op; v.op.arg0 = q.x_arg0; v.op.arg1 = q.x_arg1; v.op.pad = 0;
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
        const int* rp = reinterpret_cast<const int*>(base + L.row_prob_off);
        cudaLaunchConfig_t qcfg = {};
        qcfg.blockDim = dim3(kQuantThreads);
        qcfg.stream = st;
        cudaLaunchAttribute qattr[1];
        qattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        qattr[0].val.programmaticStreamSerializationAllowed = 1;
        qcfg.attrs = qattr;
        qcfg.numAttrs = 1;
        cudaError_t qe;
        if (rows <= sm_count) {  // a CTA per token (K <= 8192: at most four 16-byte vectors per thread)
            qcfg.gridDim = dim3((unsigned)rows);
            int max_k = 0;
            for (const MmaProblem& q : mp) max_k = std::max(max_k, q.K);
            qe = max_k <= 8 * 2 * kQuantThreads
                     ? cudaLaunchKernelEx(&qcfg, mma_quant_row_kernel<2>, hdr, probs_dev, rp, n_prob, total_items, grid, rows, sw)
                     : cudaLaunchKernelEx(&qcfg, mma_quant_row_kernel<4>, hdr, probs_dev, rp, n_prob, total_items, grid, rows, sw);
        } else if (rows <= 2 * 8 * sm_count) {  // two tokens per CTA, eight CTAs per SM
            qcfg.gridDim = dim3((unsigned)((rows + 1) / 2));
            qe = cudaLaunchKernelEx(&qcfg, mma_quant_kernel<4>, hdr, probs_dev, rp, n_prob, total_items, grid, rows, sw);
        } else {
            qcfg.gridDim = dim3((unsigned)((rows + 3) / 4));
            qe = cudaLaunchKernelEx(&qcfg, mma_quant_kernel<2>, hdr, probs_dev, rp, n_prob, total_items, grid, rows, sw);
        }
        if (qe != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
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
    // programmatic dependent launch: the kernel may begin (set-up, first weight copies) while the quantiser launch
    // before it is still running; the threads that read that launch's results call griddepcontrol.wait first
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = kMmaSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_mma_kernel, prm) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

}  // namespace bitlinear
