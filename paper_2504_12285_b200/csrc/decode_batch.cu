// Batched decode: many independent BitLinear forwards of ONE token each in two launches; with 2 to 8 tokens per
// problem the same weight stream feeds int8 mma.sync (decode_stream_mma_kernel below), with 9 to 16 tokens the call goes
// to the tcgen05 kernel of decode_mma.cu.
// (Paper Section 5.1: the decode cost is the packed weight bytes that must cross HBM; a single
// decode matmul is smaller than the memory system's bandwidth-delay product, so the weights of a
// whole batch of matmuls are streamed back to back by one persistent kernel.)
//
//   launch 1  batch_quant_kernel : one CTA per token of every problem - fused RMSNorm + absmax
//             int8 quantiser into the workspace (codes stored in the lane-interleaved order the
//             stream kernel reads, see quant_row).  A programmatic dependent of the launch before
//             it: in a decode loop its launch overlaps the previous step's stream kernel.
//   launch 2  decode_stream_kernel : one persistent CTA of 16 warps per SM.  The work list is every
//             block of 16 weight rows of every problem; each CTA owns a contiguous, byte-balanced
//             range of it.  A row block belongs to ONE warp, so 16 row blocks are in progress per CTA
//             and no partial sum ever crosses a warp.  Each warp runs its own pipeline: its lane 0
//             issues a linear bulk copy (cp.async.bulk, a few contiguous 16x256 tiles) into one of the
//             warp's two shared-memory slots; the warp waits on that slot's mbarrier, multiplies, and
//             refills the slot - across row-block and matrix boundaries, so HBM requests are always in
//             flight (16 issuing threads, ~160 KiB in flight per SM, nothing is handed from warp to warp).
//             Before the stream starts the CTA copies the descriptors of the few problems its range
//             touches, and their quantised activations, into shared memory once.
//             Unpack: word & (0x03030303 << 2j) is 4^j x the codes of four consecutive columns, fed
//             to a dot-product-of-four with the int8 activations (j = 0, 1) or, as one of four
//             operand registers, to an int8 mma.sync whose token columns all carry the one token
//             (j = 2, 3: the integer pipe, which does the masks and the quarter-rate dot products,
//             is the busiest unit; the tensor pipe is idle otherwise); one accumulator per j keeps
//             the scale uniform and the four are folded once per row block.
#include <algorithm>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <type_traits>
#include <vector>

#include "quant_row.cuh"
#include "decode_level.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

struct DevProblem {
    const uint8_t* packed;
    const float* s_w;
    void* y;
    const void* x;     // first operand of the problem's input step, all M rows of the ORIGINAL problem (see RowOp)
    const __nv_bfloat16* gain;
    RowOp op;          // the element-wise step in front of the quantiser
    int x_row0;        // row of x (and of the step's other operands) that token 0 of this entry is
    int pad0;
    int8_t* xq;
    float* d;
    int32_t* xsum;
    int32_t* acc_out;  // nullable: raw accumulators sum_k xq * Wq of this problem, [M][N] (parity hook)
    int M, N, K, y_dtype;
    float eps;
    int k_tiles;    // 1024-byte tiles per block of 16 weight rows: K / 256, or ceil(K / 320) in the dense layout
    int x_stride;   // bytes between the quantised rows of two tokens: K, or 320 * k_tiles in the dense layout (zero padded)
    int rb_begin;   // index of this problem's first row block in the global row-block list
    int rb_end;     // one past its last
    int row_begin;  // index of its first token in the global token list
};

// First bytes of the uploaded plan.  The kernels compare it with the values the host passes at
// launch, so a workspace that was overwritten between calls (with BITLINEAR_BATCH_REUSE_PLAN) is
// detected and reported instead of being followed into stale pointers.
struct PlanHeader {
    unsigned magic;
    int count, total_rb, grid, rows;
    int pad[3];
};
constexpr unsigned kPlanMagic = 0xB171A9E6u;

namespace {

__device__ __forceinline__ bool plan_matches(const PlanHeader* h, int count, int total_rb, int grid, int rows) {
    return h->magic == kPlanMagic && h->count == count && h->total_rb == total_rb && h->grid == grid && h->rows == rows;
}

constexpr int kDotJ = 2;  // of the four code positions j of a byte, how many the one-token kernel multiplies by dot-product-of-four
                          // (the rest goes to the tensor cores; 1 and 2 measured the same, 4 - no tensor cores - 3.5 % slower)
constexpr int kStreamWarps = 16;
constexpr int kStreamThreads = kStreamWarps * 32;
constexpr int kRing = 2;  // chunk slots per warp
constexpr int kBatchMaxK = 8192;
constexpr size_t kBarBytes = (size_t)kStreamWarps * kRing * 2 * 8 + 128;  // full + empty barriers, abort flag
constexpr size_t ring_bytes(int chunk_tiles) { return (size_t)kStreamWarps * kRing * chunk_tiles * kTileBytes + kBarBytes; }

// ------------------------------------------------------------------------------------ launch 1

// LAYOUT 1: codes in the lane-interleaved order of the 2-bit stream kernel; LAYOUT 0: plain column order with the row
// padded with zeros up to x_stride (the dense-layout kernel reads whole tiles of 320 columns).
template <int VPT, int LAYOUT>
__global__ void __launch_bounds__(kQuantThreads) batch_quant_kernel(const PlanHeader* __restrict__ hdr,
                                                                    const DevProblem* __restrict__ probs,
                                                                    const int* __restrict__ row_prob, int count,
                                                                    int total_rb, int grid, int* status_word) {
    __shared__ RowReduceSmem sm;
    // the stream kernel that follows may start now: it fetches weights first and waits for this grid before it reads
    // anything written here (programmatic dependent launch)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // itself a programmatic dependent of whatever runs before it on the stream (its launch overlaps that kernel's tail -
    // in a decode loop the previous step's stream kernel, which still reads what this kernel is about to overwrite):
    // nothing is read or written before that kernel is complete
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!plan_matches(hdr, count, total_rb, grid, (int)gridDim.x)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int row = blockIdx.x;
    const DevProblem& p = probs[row_prob[row]];
    const int m = row - p.row_begin;
    int8_t* xq_row = p.xq + (size_t)m * p.x_stride;
    with_row_source(p.op, p.x, p.x_row0 + m, p.K, [&](auto src) {
        quant_row_src<VPT, LAYOUT>(src, p.gain, p.eps, p.K, xq_row, p.d + m, p.xsum + m, sm);
    });
    if (LAYOUT == 0)
        for (int k = p.K + 4 * threadIdx.x; k < p.x_stride; k += 4 * kQuantThreads) *reinterpret_cast<uint32_t*>(xq_row + k) = 0u;
}

// The same for calls with more tokens than SMs (several tokens per problem): kQuantGroupWarps warps per token and
// several tokens per CTA, so that a wave of CTAs covers more tokens and a token's chain stays short.  Launched as a
// programmatic dependent of whatever runs before it (its launch overlaps that kernel's tail); it touches nothing
// before that kernel is complete.
template <int kQuantGroupWarps>
__global__ void __launch_bounds__(kQuantThreads) batch_quant_group_kernel(const PlanHeader* __restrict__ hdr,
                                                                          const DevProblem* __restrict__ probs,
                                                                          const int* __restrict__ row_prob, int count, int total_rb,
                                                                          int grid, int rows, int* status_word) {
    constexpr int kGroups = kQuantWarps / kQuantGroupWarps;  // tokens per CTA
    __shared__ GroupReduceSmem sm[kGroups];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!plan_matches(hdr, count, total_rb, grid, rows)) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    const int group = threadIdx.x / (32 * kQuantGroupWarps);
    const int row = blockIdx.x * kGroups + group;
    if (row >= rows) return;  // the whole group leaves: nobody is left waiting at its barrier
    const DevProblem& p = probs[row_prob[row]];
    const int m = row - p.row_begin;
    with_row_source(p.op, p.x, p.x_row0 + m, p.K, [&](auto src) {
        quant_row_group_src<1, kQuantGroupWarps>(src, p.gain, p.eps, p.K, p.xq + (size_t)m * p.x_stride, p.d + m, p.xsum + m, sm[group],
                                                 1 + group);
    });
}

// ------------------------------------------------------------------------------------ launch 2

__device__ __forceinline__ int dp4a_u8_s8(uint32_t a_u8x4, uint32_t b_s8x4, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_u8x4), "r"(b_s8x4), "r"(c));
    return d;
}

// d += a * b, 16 weight rows x 8 tokens x 32 columns: a = unsigned weight codes, b = int8 activations, exact in int32
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}

struct StreamParams {
    const DevProblem* probs;
    const int4* cta_range;  // [grid] {first row block, one past the last, first problem, last problem} of each CTA
    const PlanHeader* hdr;
    int count, total_rb, rows;
    int table_cap;  // problems of a CTA whose descriptors are cached in shared memory
    int arena_bytes;  // shared memory available for staged activations
    int* status_word;
    int fuse_prob;    // FUSE kernels: the plan entry that owns the one quantised row of the call
};

// Shared-memory copy of what the stream kernel needs of one problem (filled once per CTA).
struct alignas(16) SProb {
    const uint8_t* packed;
    void* y;
    const int8_t* xq;
    int32_t* acc_out;
    int rb_begin, rb_end, k_tiles, M, N, x_stride, y_dtype;
    int x_off;  // byte offset of token 0's codes in the CTA's activation arena
    float s_w;
    int pad;
    float d;   // the token's scale
    int xsum;  // and code sum
};

// Position of a warp in its sequence of weight chunks: row blocks rb, rb + par, ... of the CTA's range,
// every chunk (a few 16x256 tiles, contiguous in memory) of each.  Two of these walk the same
// sequence: one issues the bulk copies, one (kRing chunks behind) does the arithmetic.
struct ChunkCursor {
    int rb, c, p, rb_begin, rb_end, k_tiles, nc, ct;  // ct tiles per chunk, nc chunks per row block
    const uint8_t* base;                              // the current problem's packed matrix
    __device__ __forceinline__ void set_problem(int rb_begin_, int rb_end_, int k_tiles_, const void* packed,
                                                int chunk_tiles) {
        rb_begin = rb_begin_; rb_end = rb_end_; k_tiles = k_tiles_;
        nc = (k_tiles + chunk_tiles - 1) / chunk_tiles;
        ct = (k_tiles + nc - 1) / nc;
        base = static_cast<const uint8_t*>(packed);
    }
    __device__ __forceinline__ int tiles() const { return (k_tiles - c * ct) < ct ? (k_tiles - c * ct) : ct; }
    __device__ __forceinline__ const uint8_t* src() const {
        return base + ((size_t)(rb - rb_begin) * k_tiles + (size_t)c * ct) * kTileBytes;
    }
};

// One token per problem.  kChunkTiles = 16x256 tiles (1 KiB each) per bulk copy at most.
// The quantised activations of the problems the CTA touches are staged in shared memory once, as far as the arena
// reaches; those of the remaining problems are read through L1, which is slower.
// FMT 0: the 2-bit layout (tiles of 16 rows x 256 columns).  FMT 1: the dense layout, five values per byte (tiles of 16
// rows x 320 columns): a lane's 16 bytes are 80 columns of one row; the base-3 digits of the four bytes of a word are
// peeled off by repeated multiplication by 3 in two 16-bit fields per register (a byte times 3 leaves its digit in the
// byte above and the remainder in place), gathered into one operand of four codes per digit with a byte permute, and
// fed to the same dot-product-of-four against four consecutive activations.
// FUSE: the call has ONE input row (one token, every problem reads it through the same step with the same norm - q/k/v
// or gate/up of a layer, or a single matmul): there is no quantiser launch; every CTA quantises the row itself, into
// its arena, while its first weight chunks are in flight.  CTA 0 also writes the codes, the scale and the code sum
// where the quantiser launch would have put them, so that a later call may reuse them.
template <int kChunkTiles, int FMT, bool FUSE>
__global__ void __launch_bounds__(kStreamThreads, 1) decode_stream_kernel(const StreamParams prm) {
    constexpr int kCols = FMT ? kDenseTileCols : kTileCols;   // columns of a tile
    constexpr int kLaneBytes = FMT ? 80 : 16;                 // activation bytes of a column lane t inside a tile
    extern __shared__ __align__(128) uint8_t smem[];
    // [ring: 16 warps x kRing slots][full barriers][empty barriers][abort flag][descriptor table]
    // [activation arena]
    constexpr uint32_t kSlotBytes = kChunkTiles * kTileBytes;
    constexpr int par = kStreamWarps;  // row blocks in progress at a time in this CTA: one per warp
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)par * kRing * kSlotBytes);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kStreamWarps * kRing);
    SProb* table = reinterpret_cast<SProb*>(reinterpret_cast<uint8_t*>(bars) + kBarBytes);
    uint8_t* arena = reinterpret_cast<uint8_t*>(table) + (size_t)prm.table_cap * sizeof(SProb);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!plan_matches(prm.hdr, prm.count, prm.total_rb, (int)gridDim.x, prm.rows)) {  // uniform over the grid
        if (blockIdx.x == 0 && threadIdx.x == 0 && prm.status_word != nullptr)
            atomicExch(prm.status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    if (lane == 0 && warp < par) {  // warp i sets up the barriers of row-block lane i
        for (int r = 0; r < kRing; ++r) {
            mbar_init(smem_u32(bars + warp * kRing + r), 1);                          // full: the copy landed
            mbar_init(smem_u32(bars + kStreamWarps * kRing + warp * kRing + r), 1);   // empty: the warp has read it
        }
        if (warp == 0) *abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const int4 range = prm.cta_range[blockIdx.x];
    const int rb_lo = range.x, rb_hi = range.y, p_lo = range.z;
    const int n_local = rb_lo < rb_hi ? range.w - p_lo + 1 : 0;
    const int n_tab = n_local < prm.table_cap ? n_local : prm.table_cap;
    const DevProblem* probs = prm.probs;
    const int rl = warp;  // the row-block lane this warp works on
    const bool mine = rl < par && rb_lo + rl < rb_hi;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t ring_s = smem_u32(smem) + (uint32_t)rl * kRing * kSlotBytes;
    const uint32_t bar_s = smem_u32(bars + rl * kRing);                            // full barriers of this lane
    const uint32_t ebar_s = smem_u32(bars + kStreamWarps * kRing + rl * kRing);    // empty barriers
    const bool issuer = lane == 0;  // the thread of the warp that issues its copies

    // descriptor of the next problem that holds row block c.rb: from the shared-memory table when it is there
    auto enter = [&](ChunkCursor& c) {
        for (;;) {
            ++c.p;
            const int i = c.p - p_lo;
            if (i < n_tab) {
                if (c.rb < table[i].rb_end) {
                    c.set_problem(table[i].rb_begin, table[i].rb_end, table[i].k_tiles, table[i].packed, kChunkTiles);
                    return;
                }
            } else if (c.rb < probs[c.p].rb_end) {
                c.set_problem(probs[c.p].rb_begin, probs[c.p].rb_end, probs[c.p].k_tiles, probs[c.p].packed, kChunkTiles);
                return;
            }
        }
    };

    // ---- start the weight stream before anything else: the first chunks come from one problem ----
    ChunkCursor ld;  // where the next copy comes from
    ld.rb = rb_lo + rl; ld.c = 0; ld.p = p_lo;
    ld.rb_begin = 0; ld.rb_end = 0; ld.k_tiles = 1; ld.nc = 1; ld.ct = 1; ld.base = nullptr;
    bool ld_valid = mine;
    if (mine) {
        while (ld.rb >= probs[ld.p].rb_end) ++ld.p;
        ld.set_problem(probs[ld.p].rb_begin, probs[ld.p].rb_end, probs[ld.p].k_tiles, probs[ld.p].packed, kChunkTiles);
    }
    ChunkCursor cp = ld;  // where the arithmetic is
    const uint64_t once = l2_evict_first_policy();  // the weights pass through L2 once
    auto issue = [&](int slot) {  // lane 0 only
        const uint32_t bytes = (uint32_t)ld.tiles() * kTileBytes;
        mbar_expect_tx(bar_s + 8u * slot, bytes);
        bulk_load_once(ring_s + (uint32_t)slot * kSlotBytes, ld.src(), bytes, bar_s + 8u * slot, once);
    };
    auto advance_ld = [&](bool may_enter) {
        if (++ld.c == ld.nc) {
            ld.c = 0;
            ld.rb += par;
            if (ld.rb >= rb_hi) ld_valid = false;
            else if (may_enter && ld.rb >= ld.rb_end) enter(ld);
        }
    };
    int primed = 0;  // the first copies stay inside the first problem (the table is not there yet)
#pragma unroll
    for (int r = 0; r < kRing; ++r)
        if (ld_valid && ld.rb < ld.rb_end) {
            if (issuer) issue(r);
            primed = r + 1;
            advance_ld(false);
        }

    // ---- fill the descriptor table (one warp per problem) with what does not come from the quantiser launch ----
    for (int i = warp; i < n_tab; i += kStreamWarps) {
        const DevProblem& pr = probs[p_lo + i];
        if (lane == 0) {
            SProb& e = table[i];
            e.packed = pr.packed;
            e.y = pr.y; e.xq = pr.xq;
            e.acc_out = pr.acc_out;
            e.rb_begin = pr.rb_begin; e.rb_end = pr.rb_end; e.k_tiles = pr.k_tiles;
            e.M = pr.M; e.N = pr.N; e.x_stride = pr.x_stride; e.y_dtype = pr.y_dtype;
            e.x_off = 0;
            e.s_w = *pr.s_w;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int off = 0;
        for (int i = 0; i < n_tab; ++i) {
            const int bytes = table[i].M * table[i].x_stride;  // a multiple of 64
            if (FUSE) {
                table[i].x_off = 0;  // every problem reads the one row at the start of the arena
            } else if (off + bytes <= prm.arena_bytes) {
                table[i].x_off = off;
                off += bytes;
            } else {
                table[i].x_off = -1;  // does not fit: read through L1
            }
        }
    }

    // the quantiser launch that precedes this kernel must be complete before its results are read
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if constexpr (FUSE) {
        // ---- quantise the call's one input row into the arena (all threads), hand its scale and code sum to the table ----
        __shared__ RowReduceSmemT<kStreamWarps> qsm;
        __shared__ float d_s;
        __shared__ int xsum_s;
        const DevProblem& p0 = probs[prm.fuse_prob];
        RowOp op = p0.op;
        if (blockIdx.x != 0) op.x_out = nullptr;  // the step's own output (a new hidden state) is written once
        __syncthreads();  // the table is complete before the arena (which follows it) is written
        with_row_source(op, p0.x, p0.x_row0, p0.K, [&](auto src) {
            quant_row_src<2, FMT ? 0 : 1, decltype(src), kStreamThreads>(src, p0.gain, p0.eps, p0.K, reinterpret_cast<int8_t*>(arena), &d_s,
                                                                      &xsum_s, qsm);
        });
        if (FMT == 1)
            for (int k = p0.K + 4 * (int)threadIdx.x; k < p0.x_stride; k += 4 * kStreamThreads) *reinterpret_cast<uint32_t*>(arena + k) = 0u;
        __syncthreads();
        for (int i = threadIdx.x; i < n_tab; i += kStreamThreads) {
            table[i].d = d_s;
            table[i].xsum = xsum_s;
        }
        if (blockIdx.x == 0) {
            for (int o = threadIdx.x * 16; o < p0.x_stride; o += kStreamThreads * 16)
                *reinterpret_cast<uint4*>(p0.xq + o) = *reinterpret_cast<const uint4*>(arena + o);
            if (threadIdx.x == 0) {
                p0.d[0] = d_s;
                p0.xsum[0] = xsum_s;
            }
        }
        __syncthreads();
    } else {
    // ---- scales and code sums of the tokens, then stage the activations ----
    for (int i = warp; i < n_tab; i += kStreamWarps) {
        const DevProblem& pr = probs[p_lo + i];
        if (lane == 0) {
            table[i].d = pr.d[0];
            table[i].xsum = pr.xsum[0];
        }
    }
    {
        __syncthreads();
        const uint32_t arena_s = smem_u32(arena);
        for (int i = 0; i < n_tab; ++i) {
            if (table[i].x_off < 0) continue;
            const int bytes = table[i].M * table[i].x_stride;
            const int8_t* src = table[i].xq;
            const uint32_t dst = arena_s + (uint32_t)table[i].x_off;
            for (int o = threadIdx.x * 16; o < bytes; o += kStreamThreads * 16) cp_async16(dst + o, src + o);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
    }

    if (mine) {
        // top up the ring now that the cursor may cross into later problems
        if (ld_valid && ld.rb >= ld.rb_end) enter(ld);
#pragma unroll
        for (int r = 0; r < kRing; ++r)
            if (r >= primed && ld_valid) {
                if (issuer) issue(r);
                advance_ld(true);
            }

        // per-problem state of the arithmetic side
        int y_dtype = 0, xs = 0;
        void* y = nullptr;
        int32_t* acc_out = nullptr;
        float s_w = 0.0f, d = 0.0f;
        bool x_staged = false;
        const int8_t* xrow_g = nullptr;  // the token's codes in global memory
        uint32_t xrow_s = 0;             // and in the shared-memory arena (when staged)
        auto load_problem_state = [&]() {
            const int i = cp.p - p_lo;
            int x_off = -1;
            const int8_t* xq = nullptr;
            if (i < n_tab) {
                const SProb& e = table[i];
                y_dtype = e.y_dtype; y = e.y; s_w = e.s_w; x_off = e.x_off; xq = e.xq; acc_out = e.acc_out;
                d = e.d;
                xs = e.xsum;
            } else {
                const DevProblem& pr = probs[cp.p];
                y_dtype = pr.y_dtype; y = pr.y; s_w = *pr.s_w; xq = pr.xq; acc_out = pr.acc_out;
                d = pr.d[0];
                xs = pr.xsum[0];
            }
            x_staged = x_off >= 0;
            xrow_g = xq + t * kLaneBytes;
            xrow_s = smem_u32(arena) + (uint32_t)((x_staged ? x_off : 0) + t * kLaneBytes);
        };
        load_problem_state();

        int acc[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[h][j] = 0;
        // 2-bit layout: tensor-core accumulators of the codes j = 2, 3: [.][0] row g, [.][2] row g + 8, summed over the four
        // column lanes already and the same in each of them (every token column of the operand is this token)
        int macc[4 - kDotJ][4];
#pragma unroll
        for (int j = 0; j < 4 - kDotJ; ++j) macc[j][0] = macc[j][1] = macc[j][2] = macc[j][3] = 0;

        uint32_t n_chunk = 0;  // chunks consumed: slot = n_chunk % kRing, phase = (n_chunk / kRing) & 1
        bool ok = true;
        for (;;) {
            const uint32_t slot = n_chunk % kRing, phase = (n_chunk / kRing) & 1u;
            if (!mbar_wait(bar_s + 8u * slot, phase, abort_flag)) { ok = false; break; }
            const int tiles = cp.tiles();
            auto run_tiles = [&](auto staged) {
                constexpr bool XS = decltype(staged)::value;  // activations of this problem are in the arena
                uint32_t wa = ring_s + slot * kSlotBytes + (uint32_t)lane * 16u;
                uint32_t xo = (uint32_t)(cp.c * cp.ct) * kCols;
#pragma unroll 2
                for (int tile = 0; tile < tiles; ++tile, wa += kTileBytes, xo += kCols) {
                    const uint4 w0v = lds128(wa), w1v = lds128(wa + 512);
                    const uint32_t w0[4] = {w0v.x, w0v.y, w0v.z, w0v.w};
                    const uint32_t w1[4] = {w1v.x, w1v.y, w1v.z, w1v.w};
                    if constexpr (FMT == 1) {
                        // the lane's 80 activations: word 5 * i + e multiplies digit e of packed word i
                        uint32_t xw[20];
#pragma unroll
                        for (int q = 0; q < 5; ++q) {
                            uint4 v;
                            if (XS) v = lds128(xrow_s + xo + 16u * q);
                            else v = *reinterpret_cast<const uint4*>(xrow_g + xo + 16 * q);
                            xw[4 * q] = v.x; xw[4 * q + 1] = v.y; xw[4 * q + 2] = v.z; xw[4 * q + 3] = v.w;
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t ev[2] = {w0[i] & 0x00ff00ffu, w1[i] & 0x00ff00ffu};                // bytes 0 and 2
                            uint32_t od[2] = {__byte_perm(w0[i], 0u, 0x4341), __byte_perm(w1[i], 0u, 0x4341)};  // bytes 1 and 3
#pragma unroll
                            for (int e = 0; e < 5; ++e) {
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const uint32_t me = ev[h] * 3u, mo = od[h] * 3u;  // digit in bits 8-9 of each half
                                    acc[h][0] = dp4a_u8_s8(__byte_perm(me, mo, 0x7351), xw[5 * i + e], acc[h][0]);
                                    ev[h] = me & 0x00ff00ffu;
                                    od[h] = mo & 0x00ff00ffu;
                                }
                            }
                        }
                    } else {
                        // the token's codes are stored with the four 16-byte pieces of each lane's 64 columns interleaved
                        // (piece q of lane t at 64q + 16t inside the tile), so the four t lanes read 64 contiguous bytes
                        // The products are shared between two units: codes j = 0, 1 of every word go through the
                        // dot-product-of-four (a quarter-rate instruction of the integer pipe, which also does the masking),
                        // codes j = 2, 3 through an int8 mma.sync whose 8 token columns all carry this one token - a
                        // sixteenth of its products are used, and it still costs the integer pipe nothing.
#pragma unroll
                        for (int qp = 0; qp < 2; ++qp) {
                            uint4 va, vb;
                            if (XS) {
                                va = lds128(xrow_s + xo + 128u * qp);
                                vb = lds128(xrow_s + xo + 128u * qp + 64u);
                            } else {
                                va = *reinterpret_cast<const uint4*>(xrow_g + xo + 128 * qp);
                                vb = *reinterpret_cast<const uint4*>(xrow_g + xo + 128 * qp + 64);
                            }
                            const uint32_t xa[4] = {va.x, va.y, va.z, va.w}, xb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
                            for (int j = 0; j < kDotJ; ++j) {
                                const uint32_t mask = 0x03030303u << (2 * j);
                                acc[0][j] = dp4a_u8_s8(w0[2 * qp] & mask, xa[j], acc[0][j]);
                                acc[1][j] = dp4a_u8_s8(w1[2 * qp] & mask, xa[j], acc[1][j]);
                                acc[0][j] = dp4a_u8_s8(w0[2 * qp + 1] & mask, xb[j], acc[0][j]);
                                acc[1][j] = dp4a_u8_s8(w1[2 * qp + 1] & mask, xb[j], acc[1][j]);
                            }
#pragma unroll
                            for (int j = kDotJ; j < 4; ++j) {
                                const uint32_t mask = 0x03030303u << (2 * j);
                                mma_u8s8(macc[j - kDotJ], w0[2 * qp] & mask, w1[2 * qp] & mask, w0[2 * qp + 1] & mask, w1[2 * qp + 1] & mask,
                                         xa[j], xb[j]);
                            }
                        }
                    }
                }
            };
            if (x_staged) run_tiles(std::true_type{});
            else run_tiles(std::false_type{});
            __syncwarp();  // every lane of this warp has read the slot
            if (lane == 0) mbar_arrive(ebar_s + 8u * slot);
            if (ld_valid) {
                // refill the slot that has just been read
                if (issuer && mbar_wait(ebar_s + 8u * slot, phase, abort_flag)) issue((int)slot);
                advance_ld(true);
            }
            ++n_chunk;
            if (++cp.c == cp.nc) {
                // ---- end of a row block: fold the four scales (accumulator j holds 4^j x its share), the four
                //      column lanes, subtract the code offset, dequantise, store ----
                int v[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    // 64 x the sum: ((a0*4 + a1)*4 + a2)*4 + a3; |sum| <= 254*K/4 per lane: no overflow for K <= 8192
                    int sum = acc[h][0];
                    if constexpr (FMT == 0) {  // the dot-product-of-four part, this lane's share: accumulator j holds 4^j x its sum
                        sum = 0;
#pragma unroll
                        for (int j = 0; j < kDotJ; ++j) sum += acc[h][j] * (1 << (2 * (3 - j)));
                    }
                    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                    if constexpr (FMT == 0) {  // the tensor-core part, already summed over the lanes
#pragma unroll
                        for (int j = kDotJ; j < 4; ++j) {
                            sum += macc[j - kDotJ][2 * h] * (1 << (2 * (3 - j)));
                            macc[j - kDotJ][2 * h] = macc[j - kDotJ][2 * h + 1] = 0;
                        }
                    }
                    v[h] = FMT == 0 ? sum >> 6 : sum;  // 2-bit layout: exact, a multiple of 64
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[h][j] = 0;
                }
                if (t == 0) {
                    const int n0 = (cp.rb - cp.rb_begin) * kTileRows + g;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float val = __fmul_rn(__fmul_rn((float)(v[h] - xs), s_w), d);
                        const size_t idx = (size_t)(n0 + 8 * h);
                        if (acc_out != nullptr) acc_out[idx] = v[h] - xs;
                        if (y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(val);
                        else reinterpret_cast<float*>(y)[idx] = val;
                    }
                }
                cp.c = 0;
                cp.rb += par;
                if (cp.rb >= rb_hi) break;
                if (cp.rb >= cp.rb_end) {
                    enter(cp);
                    load_problem_state();
                }
            }
        }
        if (!ok) abort_drain();  // copies of this warp may still be in flight
    }
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0 && prm.status_word != nullptr) atomicExch(prm.status_word, BITLINEAR_ERR_TIMEOUT);
}

template <int kChunkTiles, int FMT, bool FUSE>
cudaError_t launch_stream(const StreamParams& prm, int grid, size_t smem, cudaStream_t st, bool dependent) {
    cudaError_t e = cudaFuncSetAttribute(decode_stream_kernel<kChunkTiles, FMT, FUSE>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // programmatic dependent launch: the kernel may begin (barrier set-up, first weight copies) while the quantiser
    // launch before it is still running; it calls griddepcontrol.wait before touching that launch's results
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, decode_stream_kernel<kChunkTiles, FMT, FUSE>, prm);
}

// Ring of the multi-token kernel: two slots of five tiles per warp, as for one token (four slots of two tiles in the same
// space were 20 % slower and three slots of four tiles 7 % slower: the cost per chunk, not the bytes in flight, is what counts); eight rows of 8,192 columns fit
// beside it.
constexpr int kMmaChunk = 5, kMmaRing = 2;
constexpr size_t mma_bar_bytes(int ring) { return (size_t)kStreamWarps * ring * 2 * 8 + 128; }
constexpr size_t mma_ring_bytes(int chunk_tiles, int ring) { return (size_t)kStreamWarps * ring * chunk_tiles * kTileBytes + mma_bar_bytes(ring); }

// Problems of 2 to 8 tokens (2-bit layout): the same weight stream, the products on the tensor cores.
// The tile layout already is the operand layout of an int8 mma.sync of 16 rows x 8 tokens x 32 columns: lane (g, t) holds
// word q of weight rows g and g + 8 - sixteen codes of columns 64q + 16t + 4j + b - and (word & mask_j) of rows g, g + 8
// and of two words q, q' are the four registers of the weight operand (the order of the columns inside a dot product is
// free); the activation operand of lane (g, t) is the matching four bytes of TOKEN g, which the interleaved activation
// layout puts into one 16-byte load per word.  As in the one-token kernel the codes are not shifted down: mask j leaves
// 4^j x the code (at most 128, an unsigned byte), one accumulator set per j keeps the scale uniform, and the four are
// folded once per row block - exact in int32.  Per tile and warp: 32 logic operations, 8 tensor-core instructions,
// 2 + 4 shared-memory loads; the integer pipe is the busiest unit (about half of its cycles).
// The arena holds the quantised rows of ONE problem at a time: the CTA goes through its problems in order, all warps meet
// before the arena is refilled, and the weight ring keeps prefetching across the meeting.  Problems that share their
// quantised input (q, k, v of a layer) share the copy.  A token's row in the arena is K + 64 bytes long, so that the
// 64-byte pieces of eight tokens fall into different banks.
// NT = 8-token groups per problem; only NT = 1 is instantiated (with two groups the kernel spills at its 128-register
// cap and is slower than the tcgen05 kernel, which therefore keeps 9 to 16 tokens).
template <int kChunkTiles, int RING, int NT>
__global__ void __launch_bounds__(kStreamThreads, 1) decode_stream_mma_kernel(const StreamParams prm) {
    extern __shared__ __align__(128) uint8_t smem[];
    // [ring: 16 warps x RING slots][full barriers][empty barriers][abort flag][activation arena]
    constexpr uint32_t kSlotBytes = kChunkTiles * kTileBytes;
    constexpr int par = kStreamWarps;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)par * RING * kSlotBytes);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kStreamWarps * RING);
    constexpr size_t kBars = (size_t)kStreamWarps * RING * 2 * 8 + 128;  // as mma_bar_bytes(RING) on the host
    uint8_t* arena = reinterpret_cast<uint8_t*>(bars) + kBars;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!plan_matches(prm.hdr, prm.count, prm.total_rb, (int)gridDim.x, prm.rows)) {  // uniform over the grid
        if (blockIdx.x == 0 && threadIdx.x == 0 && prm.status_word != nullptr)
            atomicExch(prm.status_word, BITLINEAR_ERR_WORKSPACE);
        return;
    }
    if (lane == 0) {
        for (int r = 0; r < RING; ++r) {
            mbar_init(smem_u32(bars + warp * RING + r), 1);                          // full: the copy landed
            mbar_init(smem_u32(bars + kStreamWarps * RING + warp * RING + r), 1);   // empty: the warp has read it
        }
        if (warp == 0) *abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const int4 range = prm.cta_range[blockIdx.x];
    const int rb_lo = range.x, rb_hi = range.y, p_lo = range.z, p_hi = range.w;
    const DevProblem* probs = prm.probs;
    const int rl = warp;
    const bool mine = rb_lo + rl < rb_hi;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t ring_s = smem_u32(smem) + (uint32_t)rl * RING * kSlotBytes;
    const uint32_t bar_s = smem_u32(bars + rl * RING);
    const uint32_t ebar_s = smem_u32(bars + kStreamWarps * RING + rl * RING);
    const bool issuer = lane == 0;

    // ---- the weight stream starts before anything else (the plan and the weights are not written by the launch in front)
    ChunkCursor ld;  // where the next copy comes from
    ld.rb = rb_lo + rl; ld.c = 0; ld.p = p_lo;
    ld.rb_begin = 0; ld.rb_end = 0; ld.k_tiles = 1; ld.nc = 1; ld.ct = 1; ld.base = nullptr;
    bool ld_valid = mine;
    auto enter_ld = [&]() {
        while (ld.rb >= probs[ld.p].rb_end) ++ld.p;
        ld.set_problem(probs[ld.p].rb_begin, probs[ld.p].rb_end, probs[ld.p].k_tiles, probs[ld.p].packed, kChunkTiles);
    };
    if (mine) enter_ld();
    const uint64_t once = l2_evict_first_policy();  // the weights pass through L2 once
    auto issue = [&](int slot) {  // lane 0 only
        const uint32_t bytes = (uint32_t)ld.tiles() * kTileBytes;
        mbar_expect_tx(bar_s + 8u * slot, bytes);
        bulk_load_once(ring_s + (uint32_t)slot * kSlotBytes, ld.src(), bytes, bar_s + 8u * slot, once);
    };
    auto advance_ld = [&]() {
        if (++ld.c == ld.nc) {
            ld.c = 0;
            ld.rb += par;
            if (ld.rb >= rb_hi) ld_valid = false;
            else if (ld.rb >= ld.rb_end) enter_ld();
        }
    };
#pragma unroll
    for (int r = 0; r < RING; ++r)
        if (ld_valid) {
            if (issuer) issue(r);
            advance_ld();
        }

    // the quantiser launch that precedes this kernel must be complete before its results are read
    asm volatile("griddepcontrol.wait;" ::: "memory");

    ChunkCursor cp;  // where the arithmetic is
    cp.rb = rb_lo + rl; cp.c = 0; cp.p = p_lo;
    cp.rb_begin = 0; cp.rb_end = 0; cp.k_tiles = 1; cp.nc = 1; cp.ct = 1; cp.base = nullptr;
    bool done = !mine, ok = true;
    uint32_t n_chunk = 0;  // chunks consumed: slot = n_chunk % RING, phase = (n_chunk / RING) & 1
    int macc[NT][4][4];    // [8-token group][scale 4^j][(row g, token 2t), (g, 2t + 1), (g + 8, 2t), (g + 8, 2t + 1)]
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 16; ++e) macc[nt][e >> 2][e & 3] = 0;
    const int8_t* staged_xq = nullptr;  // what the arena holds (uniform over the CTA)
    int staged_m = 0;
    const uint32_t arena_s = smem_u32(arena);

    if (rb_lo < rb_hi)
    for (int pi = p_lo; pi <= p_hi; ++pi) {  // uniform over the CTA
        const DevProblem& pr = probs[pi];
        const int M = pr.M, xst = pr.x_stride, pst = xst + 64;
        const bool fits = M * pst + 128 <= prm.arena_bytes;  // else the rows are read from global memory (slow, rare)
        if (fits && !(pr.xq == staged_xq && M == staged_m)) {
            __syncthreads();  // every warp is done with what the arena held
            const int bytes = M * xst;
            for (int o = threadIdx.x * 16; o < bytes; o += kStreamThreads * 16) cp_async16(arena_s + o + 64 * (o / xst), pr.xq + o);
            if ((int)threadIdx.x < M) {
                float* dx = reinterpret_cast<float*>(arena + M * pst);
                dx[threadIdx.x] = pr.d[threadIdx.x];
                reinterpret_cast<int*>(dx)[16 + threadIdx.x] = pr.xsum[threadIdx.x];
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
            staged_xq = pr.xq;
            staged_m = M;
        }
        if (done || cp.rb >= pr.rb_end) continue;  // this warp has no row block in the problem
        cp.p = pi;
        cp.c = 0;
        cp.set_problem(pr.rb_begin, pr.rb_end, pr.k_tiles, pr.packed, kChunkTiles);
        const int y_dtype = pr.y_dtype, n_out = pr.N;
        void* const y = pr.y;
        int32_t* const acc_out = pr.acc_out;
        const float s_w = *pr.s_w;
        // token 8 nt + g is this lane's column of the activation operand (the last token again where there is none);
        // the results this lane ends up with are those of tokens 8 nt + 2 t + e
        uint32_t xtok_s[NT];
        const int8_t* xtok_g[NT];
        float d_tok[NT][2];
        int xs_tok[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int tok = min(8 * nt + g, M - 1);
            xtok_s[nt] = arena_s + (uint32_t)(tok * pst + t * 16);
            xtok_g[nt] = pr.xq + (size_t)tok * xst + t * 16;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tk = min(8 * nt + 2 * t + e, M - 1);
                d_tok[nt][e] = fits ? reinterpret_cast<const float*>(arena + M * pst)[tk] : pr.d[tk];
                xs_tok[nt][e] = fits ? reinterpret_cast<const int*>(arena + M * pst)[16 + tk] : pr.xsum[tk];
            }
        }
        for (;;) {
            const uint32_t slot = n_chunk % RING, phase = (n_chunk / RING) & 1u;
            if (!mbar_wait(bar_s + 8u * slot, phase, abort_flag)) { ok = false; done = true; break; }
            const int tiles = cp.tiles();
            auto run_tiles = [&](auto staged) {
                constexpr bool XS = decltype(staged)::value;  // the problem's activations are in the arena
                uint32_t wa = ring_s + slot * kSlotBytes + (uint32_t)lane * 16u;
                uint32_t xo = (uint32_t)(cp.c * cp.ct) * kTileCols;
                for (int tile = 0; tile < tiles; ++tile, wa += kTileBytes, xo += kTileCols) {
                    const uint4 w0v = lds128(wa), w1v = lds128(wa + 512);
                    const uint32_t w0[4] = {w0v.x, w0v.y, w0v.z, w0v.w};  // row g
                    const uint32_t w1[4] = {w1v.x, w1v.y, w1v.z, w1v.w};  // row g + 8
#pragma unroll
                    for (int qp = 0; qp < 2; ++qp) {  // words 2 qp and 2 qp + 1 are the two column halves of an operand
                        uint32_t xa[NT][4], xb[NT][4];
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            uint4 va, vb;
                            if (XS) {
                                va = lds128(xtok_s[nt] + xo + 128u * qp);
                                vb = lds128(xtok_s[nt] + xo + 128u * qp + 64u);
                            } else {
                                va = *reinterpret_cast<const uint4*>(xtok_g[nt] + xo + 128 * qp);
                                vb = *reinterpret_cast<const uint4*>(xtok_g[nt] + xo + 128 * qp + 64);
                            }
                            xa[nt][0] = va.x; xa[nt][1] = va.y; xa[nt][2] = va.z; xa[nt][3] = va.w;
                            xb[nt][0] = vb.x; xb[nt][1] = vb.y; xb[nt][2] = vb.z; xb[nt][3] = vb.w;
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t mask = 0x03030303u << (2 * j);  // codes times 4^j: at most 128, an unsigned byte
                            const uint32_t a0 = w0[2 * qp] & mask, a1 = w1[2 * qp] & mask;
                            const uint32_t a2 = w0[2 * qp + 1] & mask, a3 = w1[2 * qp + 1] & mask;
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) mma_u8s8(macc[nt][j], a0, a1, a2, a3, xa[nt][j], xb[nt][j]);
                        }
                    }
                }
            };
            if (fits) run_tiles(std::true_type{});
            else run_tiles(std::false_type{});
            __syncwarp();  // every lane of this warp has read the slot
            if (lane == 0) mbar_arrive(ebar_s + 8u * slot);
            if (ld_valid) {
                // refill the slot that has just been read
                if (issuer && mbar_wait(ebar_s + 8u * slot, phase, abort_flag)) issue((int)slot);
                advance_ld();
            }
            ++n_chunk;
            if (++cp.c == cp.nc) {
                // ---- end of a row block: fold the two scales, subtract the code offset, dequantise, store ----
                const int n0 = (cp.rb - cp.rb_begin) * kTileRows + g;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int tok = 8 * nt + 2 * t + (e & 1);
                        // 64 x the sum, exactly: accumulator j holds 4^j x its share
                        const int a = ((((macc[nt][0][e] * 4 + macc[nt][1][e]) * 4 + macc[nt][2][e]) * 4 + macc[nt][3][e]) >> 6) - xs_tok[nt][e & 1];
                        macc[nt][0][e] = macc[nt][1][e] = macc[nt][2][e] = macc[nt][3][e] = 0;
                        if (tok < M) {
                            const float val = __fmul_rn(__fmul_rn((float)a, s_w), d_tok[nt][e & 1]);
                            const size_t idx = (size_t)tok * n_out + (size_t)(n0 + 8 * (e >> 1));
                            if (acc_out != nullptr) acc_out[idx] = a;
                            if (y_dtype == BITLINEAR_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(val);
                            else reinterpret_cast<float*>(y)[idx] = val;
                        }
                    }
                cp.c = 0;
                cp.rb += par;
                if (cp.rb >= rb_hi) { done = true; break; }
                if (cp.rb >= pr.rb_end) break;  // on to the next problem, with everybody else
            }
        }
    }
    if (!ok) abort_drain();  // copies of this warp may still be in flight
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0 && prm.status_word != nullptr) atomicExch(prm.status_word, BITLINEAR_ERR_TIMEOUT);
}

template <int kChunkTiles, int RING, int NT>
cudaError_t launch_stream_mma(const StreamParams& prm, int grid, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(decode_stream_mma_kernel<kChunkTiles, RING, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // behind this call's quantiser launch
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_stream_mma_kernel<kChunkTiles, RING, NT>, prm);
}

struct PlanLayout {
    size_t probs_off, cta_range_off, row_prob_off, xq_off, total;
};

PlanLayout plan_layout(int count, int grid, size_t xq_bytes, size_t rows) {
    PlanLayout L;
    size_t off = 256;  // the PlanHeader sits at offset 0
    L.probs_off = off;
    off = align_up(off + (size_t)count * sizeof(DevProblem), 256);
    L.cta_range_off = off;
    off = align_up(off + (size_t)(grid + 1) * sizeof(int4), 256);
    L.row_prob_off = off;
    off = align_up(off + (rows + 1) * sizeof(int), 256);
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

namespace bitlinear {

size_t prefill_group_workspace_bytes(const bitlinear_problem* problems, const int* idx, int n);
int prefill_group_forward(const bitlinear_problem* problems, const int* idx, int n, void* ws, bool skip_quant,
                          bool skip_unpack, cudaStream_t st);
// Sub-batches with a problem of more than kStreamMmaMaxTokens tokens run on the tcgen05 decode kernel (decode_mma.cu).
// Measured on the 210-matmul decode step: 100 to 121 us per step at 2 to 8 tokens through decode_stream_mma_kernel
// (141 to 153 us through the tcgen05 kernel); at 9 to 16 tokens the stream kernel needs a second accumulator set and twice the
// activation reads per tile, spills at its 128-register cap and takes 175 to 190 us against 156 to 166 us.
size_t decode_mma_workspace_bytes(const bitlinear_problem* problems, int count);
int decode_mma_forward(const bitlinear_problem* problems, int count, int flags, void* ws, size_t ws_bytes, void* stream);
constexpr int kStreamMmaMaxTokens = 8;

namespace {

// What identifies the quantised input of a plan entry: entries with equal keys share one quantised copy.
struct QuantKey {
    const void *x, *x2, *gain, *x_out;
    int M, K, op, arg0, arg1, row0;
    float eps;
    bool operator<(const QuantKey& o) const {
        return std::tie(x, x2, gain, x_out, M, K, op, arg0, arg1, row0, eps) <
               std::tie(o.x, o.x2, o.gain, o.x_out, o.M, o.K, o.op, o.arg0, o.arg1, o.row0, o.eps);
    }
};

// Bytes between the quantised rows of two tokens of a problem: K, or K padded to whole 320-column tiles (dense layout).
inline int x_stride_of(const bitlinear_problem& q) {
    return q.w_format == BITLINEAR_WEIGHTS_DENSE5 ? dense_k_tiles(q.K) * kDenseTileCols : q.K;
}

size_t decode_batch_workspace_bytes(const bitlinear_problem* problems, int count) {
    if (!problems || count <= 0) return 0;
    size_t xq = 0, rows = 0;
    int max_m = 0;
    const int fmt = problems[0].w_format;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.M < 0 || q.M > kGemvMaxTokens || !shape_ok(q.N, q.K) || q.K > kBatchMaxK || q.w_format != fmt) return 0;
        xq += align_up((size_t)q.M * x_stride_of(q), 16);
        rows += (size_t)q.M;
        if (q.M > max_m) max_m = q.M;
    }
    if (fmt == BITLINEAR_WEIGHTS_2BIT && max_m > kStreamMmaMaxTokens) return decode_mma_workspace_bytes(problems, count);
    // the dense-layout kernel takes one token per problem: a problem of M tokens is planned as M problems
    return plan_layout(fmt == BITLINEAR_WEIGHTS_DENSE5 ? (int)rows : count, kPlanGrid, xq, rows).total;
}

// What the host derives from the problem list of a call (everything the two launches need besides the plan in the
// workspace).  A call with BITLINEAR_BATCH_REUSE_PLAN whose problem list is the one an earlier call planned into the same
// workspace takes it from here instead of planning again (a 70-problem plan costs the host about as long as the kernel
// runs).  Keyed by workspace address and a hash of the descriptors; a few entries, replaced in turn.
struct PlanShape {
    int n_prob, total_rb, grid, rows, table_cap, table_need;
    size_t arena_max;
};
struct PlanCacheEntry {
    const void* ws = nullptr;
    uint64_t hash = 0;
    int count = 0;
    bool has_acc = false;
    PlanShape shape = {};
};
constexpr int kPlanCacheEntries = 16;
std::mutex g_plan_cache_mu;
PlanCacheEntry g_plan_cache[kPlanCacheEntries];
int g_plan_cache_next = 0;

uint64_t hash_problems(const bitlinear_problem* problems, int count) {
    // the descriptors word by word (their size is a multiple of 8); bytes of padding take part: a list that differs only
    // there is planned again, which is correct and merely slower
    static_assert(sizeof(bitlinear_problem) % 8 == 0, "hashed in 8-byte words");
    uint64_t h = 1469598103934665603ull;
    const size_t words = (size_t)count * sizeof(bitlinear_problem) / 8;
    for (size_t i = 0; i < words; ++i) {
        uint64_t w;
        memcpy(&w, reinterpret_cast<const char*>(problems) + 8 * i, 8);
        h = (h ^ w) * 1099511628211ull;
        h ^= h >> 29;
    }
    return h;
}

bool plan_cache_find(const void* ws, uint64_t hash, int count, bool has_acc, PlanShape* out) {
    std::lock_guard<std::mutex> lock(g_plan_cache_mu);
    for (const PlanCacheEntry& e : g_plan_cache)
        if (e.ws == ws && e.hash == hash && e.count == count && e.has_acc == has_acc) {
            *out = e.shape;
            return true;
        }
    return false;
}

void plan_cache_store(const void* ws, uint64_t hash, int count, bool has_acc, const PlanShape& shape) {
    std::lock_guard<std::mutex> lock(g_plan_cache_mu);
    PlanCacheEntry* slot = nullptr;
    for (PlanCacheEntry& e : g_plan_cache)
        if (e.ws == ws) slot = &e;  // one plan per workspace
    if (!slot) {
        slot = &g_plan_cache[g_plan_cache_next];
        g_plan_cache_next = (g_plan_cache_next + 1) % kPlanCacheEntries;
    }
    slot->ws = ws; slot->hash = hash; slot->count = count; slot->has_acc = has_acc; slot->shape = shape;
}

// acc_outs: nullptr, or one (nullable) device pointer per problem for the raw accumulators.
int decode_batch_forward(const bitlinear_problem* problems, int count, int flags, int32_t* const* acc_outs, void* ws,
                         size_t ws_bytes, void* stream) {
    size_t xq_bytes = 0, rows = 0;
    int max_m = 0, max_k = 0;
    const int fmt = problems[0].w_format;
    const bool dense = fmt == BITLINEAR_WEIGHTS_DENSE5;
    bool want_acc = false;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.y_dtype != BITLINEAR_F32 && q.y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
        if (q.w_format != fmt) return BITLINEAR_ERR_DTYPE;  // one weight layout per call
        if (q.M < 0 || q.M > kGemvMaxTokens || !shape_ok(q.N, q.K) || q.K > kBatchMaxK) return BITLINEAR_ERR_SHAPE;
        if (acc_outs && acc_outs[i]) {
            if (reinterpret_cast<uintptr_t>(acc_outs[i]) & 3u) return BITLINEAR_ERR_ALIGN;
            want_acc = true;
        }
        if (q.M == 0) continue;
        if (!q.x || !q.packed || !q.s_w || !q.y) return BITLINEAR_ERR_NULL;
        if (!aligned16(q.x) || !aligned16(q.packed) || !aligned16(q.y) || (q.gain && !aligned16(q.gain)) ||
            (reinterpret_cast<uintptr_t>(q.s_w) & 3u))
            return BITLINEAR_ERR_ALIGN;
        xq_bytes += align_up((size_t)q.M * x_stride_of(q), 16);
        rows += (size_t)q.M;
        if (q.M > max_m) max_m = q.M;
        if (q.K > max_k) max_k = q.K;
    }
    if (!dense && max_m > kStreamMmaMaxTokens) {
        if (want_acc) return BITLINEAR_ERR_SHAPE;  // the tcgen05 decode kernel has no accumulator output
        return decode_mma_forward(problems, count, flags, ws, ws_bytes, stream);
    }
    const int nt = dense || max_m <= 1 ? 0 : 1;  // 2 to 8 tokens: the multi-token stream kernel
    const PlanLayout L = plan_layout(dense ? (int)rows : count, kPlanGrid, xq_bytes, rows);
    if (!ws || !aligned16(ws) || ws_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    if (rows == 0) return BITLINEAR_OK;

    int sm_count = 0;
    if (const int rc = device_sm_count(&sm_count)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);

    // ---- a level of a decoder layer called again (REUSE_PLAN): up to four one-token problems on one input row need no host
    //      plan at all - the launch carries its descriptors, and the quantised row goes where the plan of the first call put it
    if ((flags & BITLINEAR_BATCH_REUSE_PLAN) && !(flags & BITLINEAR_BATCH_REUSE_ACT) && !dense && count <= kLevelMaxProblems &&
        rows == (size_t)count) {
        const bitlinear_problem& q0 = problems[0];
        bool one_input = true;
        int total_rb0 = 0;
        for (int i = 0; i < count; ++i) {
            const bitlinear_problem& q = problems[i];
            one_input = one_input && q.x == q0.x && q.x2 == q0.x2 && q.gain == q0.gain && q.x_out == q0.x_out && q.K == q0.K &&
                        q.x_op == q0.x_op && q.x_arg0 == q0.x_arg0 && q.x_arg1 == q0.x_arg1 && q.rms_eps == q0.rms_eps;
            total_rb0 += q.N / kTileRows;
        }
        if (one_input && decode_level_fits(count, total_rb0, q0.K, sm_count)) {
            LevelParams P = {};
            P.count = count;
            for (int i = 0; i < count; ++i) {
                const bitlinear_problem& q = problems[i];
                P.prob[i].packed = static_cast<const uint8_t*>(q.packed); P.prob[i].s_w = q.s_w; P.prob[i].y = q.y;
                P.prob[i].acc_out = acc_outs ? acc_outs[i] : nullptr;
                P.prob[i].N = q.N; P.prob[i].y_dtype = q.y_dtype;
            }
            P.x = q0.x;
            P.op.x2 = q0.x2; P.op.x_out = q0.x_out; P.op.op = q0.x_op; P.op.arg0 = q0.x_arg0; P.op.arg1 = q0.x_arg1; P.op.pad = 0;
            P.gain = static_cast<const __nv_bfloat16*>(q0.gain); P.eps = q0.rms_eps; P.K = q0.K; P.x_row0 = 0;
            // the places the plan gives the first entry's quantised row, scale and code sum (see below)
            P.xq_out = reinterpret_cast<int8_t*>(base + L.xq_off);
            P.d_out = reinterpret_cast<float*>(base + align_up(L.xq_off + xq_bytes, 256));
            P.xsum_out = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(P.d_out) + align_up(rows * sizeof(float), 256));
            P.total_rb = total_rb0;
            P.status_word = device_status_word();
            return decode_level_forward(P, sm_count, st, /*dependent=*/true);
        }
    }

    // ---- the plan of an earlier call on this workspace, if the caller says it is still there and the problems are the same
    //      (accumulator pointers are part of the device plan: calls that pass any are always planned)
    const uint64_t list_hash = want_acc ? 0 : hash_problems(problems, count);
    PlanShape shape = {};
    const bool planned = !want_acc && (flags & BITLINEAR_BATCH_REUSE_PLAN) && plan_cache_find(ws, list_hash, count, false, &shape) &&
                         shape.rows != 1;  // a single input row: the launch is built from the descriptors themselves

    // ---- host plan: device descriptors, token -> problem table, byte-balanced CTA ranges ----
    std::vector<DevProblem> dp;
    std::vector<int> row_prob;
    std::map<QuantKey, int> quantised;  // first entry of dp that quantises a given input
    int total_rb = 0, n_prob = 0, grid = 0, table_cap = 1, table_need = 1;
    size_t arena_max = 0;  // most activation bytes any CTA needs
    std::vector<int4> cta_range;
    if (planned) {
        n_prob = shape.n_prob; total_rb = shape.total_rb; grid = shape.grid; rows = (size_t)shape.rows;
        table_cap = shape.table_cap; table_need = shape.table_need; arena_max = shape.arena_max;
    } else {
    dp.reserve(count);
    row_prob.reserve(rows + 1);
    {
        char* xq_ptr = base + L.xq_off;
        float* d_ptr = reinterpret_cast<float*>(base + align_up(L.xq_off + xq_bytes, 256));
        int32_t* xs_ptr = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(d_ptr) + align_up(rows * sizeof(float), 256));
        int row = 0;
        for (int i = 0; i < count; ++i) {
            const bitlinear_problem& q = problems[i];
            if (q.M == 0) continue;
            const int stride = x_stride_of(q);
            const size_t y_row = (size_t)q.N * (q.y_dtype == BITLINEAR_BF16 ? 2 : 4);
            // the dense-layout kernel multiplies one token per problem: every token becomes a problem of its own
            // (its weights are then streamed once per token)
            const int parts = dense ? q.M : 1, m_each = dense ? 1 : q.M;
            for (int part = 0; part < parts; ++part) {
                DevProblem v;
                v.packed = static_cast<const uint8_t*>(q.packed);
                v.s_w = q.s_w;
                v.y = static_cast<char*>(q.y) + (size_t)part * y_row;
                v.x = q.x;
                v.x_row0 = part;
                v.pad0 = 0;
                v.op.x2 = q.x2; v.op.x_out = q.x_out; v.op.op = q.x_op; v.op.arg0 = q.x_arg0; v.op.arg1 = q.x_arg1; v.op.pad = 0;
                v.gain = static_cast<const __nv_bfloat16*>(q.gain);
                // entries that read the same rows through the same step with the same norm share one quantised copy
                const QuantKey key{q.x, q.x2, q.gain, q.x_out, q.M, q.K, q.x_op, q.x_arg0, q.x_arg1, part, q.rms_eps};
                const auto seen = quantised.find(key);
                if (seen != quantised.end()) {
                    const DevProblem& first = dp[seen->second];
                    v.xq = first.xq; v.d = first.d; v.xsum = first.xsum;
                    v.acc_out = (acc_outs && acc_outs[i]) ? acc_outs[i] + (size_t)part * q.N : nullptr;
                    v.M = m_each; v.N = q.N; v.K = q.K; v.y_dtype = q.y_dtype;
                    v.eps = q.rms_eps;
                    v.k_tiles = dense ? dense_k_tiles(q.K) : q.K / kTileCols;
                    v.x_stride = stride;
                    v.rb_begin = total_rb;
                    v.rb_end = total_rb + q.N / kTileRows;
                    v.row_begin = first.row_begin;
                    dp.push_back(v);
                    total_rb = v.rb_end;
                    continue;
                }
                quantised.emplace(key, (int)dp.size());
                v.xq = reinterpret_cast<int8_t*>(xq_ptr) + (size_t)part * stride;
                v.d = d_ptr + row;
                v.xsum = xs_ptr + row;
                v.acc_out = (acc_outs && acc_outs[i]) ? acc_outs[i] + (size_t)part * q.N : nullptr;
                v.M = m_each; v.N = q.N; v.K = q.K; v.y_dtype = q.y_dtype;
                v.eps = q.rms_eps;
                v.k_tiles = dense ? dense_k_tiles(q.K) : q.K / kTileCols;
                v.x_stride = stride;
                v.rb_begin = total_rb;
                v.rb_end = total_rb + q.N / kTileRows;
                v.row_begin = row;
                for (int m = 0; m < m_each; ++m) row_prob.push_back((int)dp.size());
                dp.push_back(v);
                total_rb = v.rb_end;
                row += m_each;
            }
            xq_ptr += align_up((size_t)q.M * stride, 16);
        }
        rows = (size_t)row;  // tokens actually quantised (shared copies counted once)
        row_prob.push_back(0);
    }
    n_prob = (int)dp.size();
    grid = sm_count < total_rb ? sm_count : total_rb;
    cta_range.resize(grid);
    table_cap = 1;  // most problems any CTA touches
    {
        std::vector<int> cta_rb(grid + 1);
        double total_tiles = 0.0;
        for (int i = 0; i < n_prob; ++i) total_tiles += (double)(dp[i].rb_end - dp[i].rb_begin) * dp[i].k_tiles;
        int pi = 0;
        double before = 0.0;  // tiles before problem pi
        cta_rb[0] = 0;
        for (int c = 1; c < grid; ++c) {
            const double target = total_tiles * c / grid;
            while (pi < n_prob - 1 && before + (double)(dp[pi].rb_end - dp[pi].rb_begin) * dp[pi].k_tiles <= target) {
                before += (double)(dp[pi].rb_end - dp[pi].rb_begin) * dp[pi].k_tiles;
                ++pi;
            }
            int rb = dp[pi].rb_begin + (int)((target - before) / (double)dp[pi].k_tiles + 0.5);
            if (rb > dp[pi].rb_end) rb = dp[pi].rb_end;
            if (rb < cta_rb[c - 1]) rb = cta_rb[c - 1];
            cta_rb[c] = rb;
        }
        cta_rb[grid] = total_rb;
        int pf = 0;
        for (int c = 0; c < grid; ++c) {
            const int lo = cta_rb[c], hi = cta_rb[c + 1];
            while (pf < n_prob - 1 && lo >= dp[pf].rb_end) ++pf;
            int pl = pf;
            while (pl < n_prob - 1 && hi - 1 >= dp[pl].rb_end) ++pl;
            cta_range[c] = make_int4(lo, hi, pf, pl);
            if (lo < hi) {
                if (pl - pf + 1 > table_cap) table_cap = pl - pf + 1;
                size_t a = 0;
                for (int i = pf; i <= pl; ++i) {
                    const size_t one = (size_t)dp[i].M * (dp[i].x_stride + 64) + 128;  // multi-token: one problem at a time, padded rows
                    if (nt) a = std::max(a, one);
                    else a += (size_t)dp[i].M * dp[i].x_stride;
                }
                if (a > arena_max) arena_max = a;
            }
        }
    }
    // shared memory: chunk ring + descriptor table + activation arena; activations that do not fit the arena are read
    // through L1 instead, and only as many descriptors as fit a quarter of the space are cached
    // (the multi-token kernel caches no descriptors and keeps the rows of one problem at a time in its arena)
    {
        const size_t smem_limit = 227 * 1024 - (nt == 0 ? ring_bytes(5) : mma_ring_bytes(kMmaChunk, kMmaRing)) - 128;
        if (nt) table_cap = 0;
        table_need = table_cap;  // with fewer cached descriptors some problems of a CTA are read from global memory
        if ((size_t)table_cap * sizeof(SProb) > smem_limit / 4) table_cap = (int)(smem_limit / 4 / sizeof(SProb));
        if (arena_max > smem_limit - (size_t)table_cap * sizeof(SProb)) arena_max = smem_limit - (size_t)table_cap * sizeof(SProb);
        if (nt) arena_max = std::min(align_up(arena_max, 256), smem_limit & ~(size_t)255);
        else arena_max &= ~(size_t)255;
    }
    {   // (a call with accumulator pointers leaves no entry: its plan carries them)
        const PlanShape made = {n_prob, total_rb, grid, (int)rows, table_cap, table_need, arena_max};
        plan_cache_store(ws, want_acc ? 0 : list_hash, want_acc ? -1 : count, false, made);
    }
    }  // planned or not
    constexpr int chunk_tiles = 5;
    const size_t ring_total = nt == 0 ? ring_bytes(chunk_tiles) : mma_ring_bytes(kMmaChunk, kMmaRing);

    PlanHeader hdr_host;
    hdr_host.magic = kPlanMagic;
    hdr_host.count = n_prob;
    hdr_host.total_rb = total_rb;
    hdr_host.grid = grid;
    hdr_host.rows = (int)rows;
    hdr_host.pad[0] = hdr_host.pad[1] = hdr_host.pad[2] = 0;
    if (!(flags & BITLINEAR_BATCH_REUSE_PLAN)) {
        if (cudaMemcpyAsync(base, &hdr_host, sizeof(hdr_host), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.probs_off, dp.data(), dp.size() * sizeof(DevProblem), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.cta_range_off, cta_range.data(), cta_range.size() * sizeof(int4), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(base + L.row_prob_off, row_prob.data(), row_prob.size() * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
    }
    const DevProblem* probs_dev = reinterpret_cast<const DevProblem*>(base + L.probs_off);

    // One input row in the whole call (a single token, every problem reading it the same way - the usual shape of one level
    // of a decoder layer at one token): no quantiser launch, the stream kernel quantises the row itself (FUSE).
    const bool fuse = rows == 1 && !(flags & BITLINEAR_BATCH_REUSE_ACT) && table_cap == table_need && max_k <= 16 * kStreamThreads;
    if (fuse) arena_max = std::max(arena_max, align_up((size_t)dp[0].x_stride, 256));  // (never with a cached shape: rows != 1)

    // ... and when the problems are few (a level of a decoder layer) the whole call is one launch that carries its
    // descriptors in its arguments (decode_level.cu); the plan uploaded above stays valid for calls that reuse activations
    // A fused launch reads weights, scales and gain before it waits for the launch in front of it, which is only safe
    // when that launch does not write them: the steady state of a decode loop, which BITLINEAR_BATCH_REUSE_PLAN names.
    const bool static_weights = (flags & BITLINEAR_BATCH_REUSE_PLAN) != 0;
    if (fuse && !dense && decode_level_fits(n_prob, total_rb, max_k, sm_count)) {
        LevelParams P = {};
        P.count = n_prob;
        for (int i = 0; i < n_prob; ++i) {
            P.prob[i].packed = dp[i].packed; P.prob[i].s_w = dp[i].s_w; P.prob[i].y = dp[i].y; P.prob[i].acc_out = dp[i].acc_out;
            P.prob[i].N = dp[i].N; P.prob[i].y_dtype = dp[i].y_dtype;
        }
        P.x = dp[0].x; P.op = dp[0].op; P.gain = dp[0].gain; P.eps = dp[0].eps; P.K = dp[0].K; P.x_row0 = dp[0].x_row0;
        P.xq_out = dp[0].xq; P.d_out = dp[0].d; P.xsum_out = dp[0].xsum;
        P.total_rb = total_rb;
        P.status_word = device_status_word();
        return decode_level_forward(P, sm_count, st, static_weights);
    }

    // ---- launch 1: quantise every token of every problem ----
    if (!fuse && !(flags & BITLINEAR_BATCH_REUSE_ACT)) {
        const int vpt = (max_k / 8 + kQuantThreads - 1) / kQuantThreads;
        const dim3 g((unsigned)rows), b(kQuantThreads);
        const PlanHeader* h = reinterpret_cast<const PlanHeader*>(base);
        const int* rp = reinterpret_cast<const int*>(base + L.row_prob_off);
        int* sw = device_status_word();
        if (nt && (int)rows > sm_count) {
            // more tokens than SMs: groups of warps per token (two tokens per CTA while eight CTAs per SM hold them all)
            cudaLaunchConfig_t qcfg = {};
            qcfg.blockDim = dim3(kQuantThreads);
            qcfg.stream = st;
            cudaLaunchAttribute qattr[1];
            qattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            qattr[0].val.programmaticStreamSerializationAllowed = 1;
            qcfg.attrs = qattr;
            qcfg.numAttrs = 1;
            cudaError_t qe;
            if ((int)rows <= 2 * 8 * sm_count) {
                qcfg.gridDim = dim3((unsigned)((rows + 1) / 2));
                qe = cudaLaunchKernelEx(&qcfg, batch_quant_group_kernel<4>, h, probs_dev, rp, n_prob, total_rb, grid, (int)rows, sw);
            } else {
                qcfg.gridDim = dim3((unsigned)((rows + 3) / 4));
                qe = cudaLaunchKernelEx(&qcfg, batch_quant_group_kernel<2>, h, probs_dev, rp, n_prob, total_rb, grid, (int)rows, sw);
            }
            if (qe != cudaSuccess) {
                cudaGetLastError();
                return BITLINEAR_ERR_CUDA;
            }
        } else {
            cudaLaunchConfig_t qcfg = {};
            qcfg.gridDim = g;
            qcfg.blockDim = b;
            qcfg.stream = st;
            cudaLaunchAttribute qattr[1];
            qattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            qattr[0].val.programmaticStreamSerializationAllowed = 1;
            qcfg.attrs = qattr;
            qcfg.numAttrs = 1;
            auto launch_q = [&](auto kernel) { return cudaLaunchKernelEx(&qcfg, kernel, h, probs_dev, rp, n_prob, total_rb, grid, sw); };
            const cudaError_t qe = dense ? (vpt <= 1 ? launch_q(batch_quant_kernel<1, 0>) : vpt <= 2 ? launch_q(batch_quant_kernel<2, 0>)
                                                                                                : launch_q(batch_quant_kernel<4, 0>))
                                         : (vpt <= 1 ? launch_q(batch_quant_kernel<1, 1>) : vpt <= 2 ? launch_q(batch_quant_kernel<2, 1>)
                                                                                                : launch_q(batch_quant_kernel<4, 1>));
            if (qe != cudaSuccess) {
                cudaGetLastError();
                return BITLINEAR_ERR_CUDA;
            }
        }
    }

    // ---- launch 2: stream the weights ----
    StreamParams prm;
    prm.probs = probs_dev;
    prm.cta_range = reinterpret_cast<const int4*>(base + L.cta_range_off);
    prm.hdr = reinterpret_cast<const PlanHeader*>(base);
    prm.count = n_prob;
    prm.total_rb = total_rb;
    prm.rows = (int)rows;
    prm.status_word = device_status_word();
    prm.table_cap = table_cap;
    prm.arena_bytes = (int)arena_max;
    const size_t smem = ring_total + (size_t)table_cap * sizeof(SProb) + arena_max + 128;
    prm.fuse_prob = 0;
    if (nt) {
        const cudaError_t em = launch_stream_mma<kMmaChunk, kMmaRing, 1>(prm, grid, smem, st);
        return em == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
    }  // the first entry owns the quantised copy of the one row
    // behind the quantiser launch of this call the stream kernel is always a dependent (that launch writes no weights);
    // a fused launch only under the promise above
    const bool dep = !fuse || static_weights;
    const cudaError_t e = fuse ? (dense ? launch_stream<chunk_tiles, 1, true>(prm, grid, smem, st, dep)
                                        : launch_stream<chunk_tiles, 0, true>(prm, grid, smem, st, dep))
                               : (dense ? launch_stream<chunk_tiles, 1, false>(prm, grid, smem, st, dep)
                                        : launch_stream<chunk_tiles, 0, false>(prm, grid, smem, st, dep));
    return e == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

namespace {

// The element-wise step in front of a problem's quantiser (x_op and its operands), checked on the host.
int check_input_step(const bitlinear_problem& q) {
    if (q.x_op < BITLINEAR_X_PLAIN || q.x_op > BITLINEAR_X_ATTN_STANDIN) return BITLINEAR_ERR_DTYPE;
    if (q.x_op == BITLINEAR_X_PLAIN || q.M == 0) return BITLINEAR_OK;
    if (!q.x2) return BITLINEAR_ERR_NULL;
    if (!aligned16(q.x2) || (q.x_out && !aligned16(q.x_out))) return BITLINEAR_ERR_ALIGN;
    if (q.x_out == q.x) return BITLINEAR_ERR_SHAPE;  // rows are read more than once: the result cannot replace them
    if (q.x_op == BITLINEAR_X_ATTN_STANDIN) {
        if (q.x_arg0 <= 0 || q.x_arg0 % 8 || q.x_arg1 <= 0 || q.K % q.x_arg0 || (q.K / q.x_arg0) % q.x_arg1) return BITLINEAR_ERR_SHAPE;
        if (((size_t)(q.K / q.x_arg1) * sizeof(float)) % 16) return BITLINEAR_ERR_ALIGN;  // rows of v stay 16-byte aligned
    }
    return BITLINEAR_OK;
}

// Up to this many tokens a problem of the 2-bit layout is cut into problems of 16 tokens for the tensor-core decode
// kernel, which streams the packed weights once per 16 tokens; above it the weights are expanded to byte codes and
// multiplied by the tcgen05 GEMM on 256-token tiles.  Measured on the FFN down projection (2560 x 6912) in a batch of 32
// such matmuls: 2.2 us per matmul at 32 tokens and 4.0 us at 64 through the decode kernel, 7.7 us through the GEMM at
// either (a 256 x 256 tile is mostly padding below 128 tokens); at 256 tokens the GEMM takes 7.8 us.
constexpr int kDecodeChunkMaxTokens = 96;

// Row m0 onwards of a problem as a problem of its own (m rows): every operand advanced by its own row size.
bitlinear_problem rows_of(const bitlinear_problem& q, int m0, int m) {
    bitlinear_problem c = q;
    const size_t K = (size_t)q.K;
    auto adv = [&](const void* p, size_t row_bytes) {
        return p ? static_cast<const void*>(static_cast<const char*>(p) + (size_t)m0 * row_bytes) : nullptr;
    };
    const bool x_is_f32 = q.x_op == BITLINEAR_X_RELU2 || q.x_op == BITLINEAR_X_ATTN_STANDIN;
    c.x = adv(q.x, K * (x_is_f32 ? 4 : 2));
    c.x2 = adv(q.x2, (q.x_op == BITLINEAR_X_ATTN_STANDIN ? K / q.x_arg1 : K) * 4);
    c.x_out = const_cast<void*>(adv(q.x_out, K * 2));
    c.y = const_cast<void*>(adv(q.y, (size_t)q.N * (q.y_dtype == BITLINEAR_BF16 ? 2 : 4)));
    c.M = m;
    return c;
}

// Splits the problems of a call into those of the decode kernels (at most 16 tokens each, longer ones cut into chunks
// where that is the faster path) and those of the grouped GEMM (indices).  Returns a status.
int partition_problems(const bitlinear_problem* problems, int count, int32_t* const* acc_out, std::vector<bitlinear_problem>& dec,
                       std::vector<int32_t*>& dec_acc, std::vector<int>& pre) {
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.y_dtype != BITLINEAR_F32 && q.y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
        if (q.w_format != BITLINEAR_WEIGHTS_2BIT && q.w_format != BITLINEAR_WEIGHTS_DENSE5) return BITLINEAR_ERR_DTYPE;
        if (q.M < 0 || !shape_ok(q.N, q.K)) return BITLINEAR_ERR_SHAPE;
        if (const int rc = check_input_step(q)) return rc;
        int32_t* acc = acc_out ? acc_out[i] : nullptr;
        if (q.M <= kGemvMaxTokens) {
            if (q.K > kBatchMaxK) return BITLINEAR_ERR_SHAPE;
            dec.push_back(q);
            dec_acc.push_back(acc);
            continue;
        }
        if (q.w_format != BITLINEAR_WEIGHTS_2BIT || acc) return BITLINEAR_ERR_SHAPE;  // dense layout / accumulators: decode sizes only
        if (q.M <= kDecodeChunkMaxTokens && q.K <= kBatchMaxK) {
            for (int m0 = 0; m0 < q.M; m0 += kGemvMaxTokens) {
                dec.push_back(rows_of(q, m0, std::min(kGemvMaxTokens, q.M - m0)));
                dec_acc.push_back(nullptr);
            }
            continue;
        }
        if (q.N % 128) return BITLINEAR_ERR_SHAPE;
        if (!q.x || !q.packed || !q.s_w || !q.y) return BITLINEAR_ERR_NULL;
        if (!aligned16(q.x) || !aligned16(q.packed) || !aligned16(q.y) || (q.gain && !aligned16(q.gain)) ||
            (reinterpret_cast<uintptr_t>(q.s_w) & 3u))
            return BITLINEAR_ERR_ALIGN;
        pre.push_back(i);
    }
    return BITLINEAR_OK;
}

}  // namespace

namespace {

// ---- bitlinear_forward_batch_host in segments: while one segment's kernels run, the next one's inputs come in and the
//      previous one's outputs go out (the copy engines work beside the SMs).
constexpr int kHostSegments = 3;
constexpr int kHostSegmentMinProblems = 8;  // per segment; smaller calls are not worth three pairs of launches

struct HostSegments {
    int cut[kHostSegments + 1];        // problems [cut[s], cut[s + 1])
    size_t xcut[kHostSegments + 1];    // bytes [xcut[s], xcut[s + 1]) of the x arena belong to segment s
    size_t ycut[kHostSegments + 1];
    size_t ws_off[kHostSegments + 1];  // its slice of the workspace
};

// Decode-sized problems with a plain input whose operands lie in the arenas in the order of the problems: cut where a
// third and two thirds of the packed bytes have gone by (cuts at 45 and 80 % measured the same: the call is bound by the
// host's enqueue time either way).  A segment's part of an arena begins where its lowest operand
// begins and ends where the next segment's does, so the parts are disjoint and together the whole arena.  False where
// any of that does not hold (the call then runs unsegmented).
size_t batch_workspace_core(const bitlinear_problem* problems, int count);

// which problems go into which segment (by shapes alone, so that the workspace can be sized without the arenas)
bool host_segment_cuts(const bitlinear_problem* problems, int count, int (&cut)[kHostSegments + 1]) {
    if (count < kHostSegments * kHostSegmentMinProblems) return false;
    double total = 0.0;
    for (int i = 0; i < count; ++i) {
        const bitlinear_problem& q = problems[i];
        if (q.M < 1 || q.M > kGemvMaxTokens || q.x_op != BITLINEAR_X_PLAIN || !shape_ok(q.N, q.K)) return false;
        total += (double)q.N * q.K;
    }
    cut[0] = 0;
    double run = 0.0;
    int s = 1;
    for (int i = 0; i < count && s < kHostSegments; ++i) {
        run += (double)problems[i].N * problems[i].K;
        if (run >= total * s / kHostSegments) cut[s++] = i + 1;
    }
    for (; s <= kHostSegments; ++s) cut[s] = count;
    for (s = 0; s < kHostSegments; ++s)
        if (cut[s + 1] - cut[s] < kHostSegmentMinProblems) return false;
    return true;
}

// the workspace the segments of a call need together (0: the call is not segmented)
size_t host_segments_workspace(const bitlinear_problem* problems, int count) {
    int cut[kHostSegments + 1];
    if (!problems || !host_segment_cuts(problems, count, cut)) return 0;
    size_t total = 0;
    for (int s = 0; s < kHostSegments; ++s) {
        const size_t need = batch_workspace_core(problems + cut[s], cut[s + 1] - cut[s]);
        if (need == 0) return 0;
        total += align_up(need, 1024);
    }
    return total;
}

bool plan_host_segments(const bitlinear_problem* problems, int count, const void* x_dev, size_t x_bytes, const void* y_dev,
                        size_t y_bytes, size_t ws_bytes, HostSegments* out) {
    HostSegments sg;
    if (!host_segment_cuts(problems, count, sg.cut)) return false;
    const char* xb = static_cast<const char*>(x_dev);
    const char* yb = static_cast<const char*>(y_dev);
    for (int i = 0; i < count; ++i)
        if (!problems[i].x || !problems[i].y) return false;
    const char *x_lo[kHostSegments], *x_hi[kHostSegments], *y_lo[kHostSegments], *y_hi[kHostSegments];
    sg.ws_off[0] = 0;
    for (int s = 0; s < kHostSegments; ++s) {
        const int n = sg.cut[s + 1] - sg.cut[s];
        x_lo[s] = x_hi[s] = y_lo[s] = y_hi[s] = nullptr;
        for (int i = sg.cut[s]; i < sg.cut[s + 1]; ++i) {
            const bitlinear_problem& q = problems[i];
            const char* x0 = static_cast<const char*>(q.x);
            const char* x1 = x0 + (size_t)q.M * q.K * 2;
            const char* y0 = static_cast<const char*>(q.y);
            const char* y1 = y0 + (size_t)q.M * q.N * (q.y_dtype == BITLINEAR_BF16 ? 2 : 4);
            if (x0 < xb || x1 > xb + x_bytes || y0 < yb || y1 > yb + y_bytes) return false;
            if (!x_lo[s] || x0 < x_lo[s]) x_lo[s] = x0;
            if (!x_hi[s] || x1 > x_hi[s]) x_hi[s] = x1;
            if (!y_lo[s] || y0 < y_lo[s]) y_lo[s] = y0;
            if (!y_hi[s] || y1 > y_hi[s]) y_hi[s] = y1;
        }
        if (s > 0 && (x_hi[s - 1] > x_lo[s] || y_hi[s - 1] > y_lo[s])) return false;  // a part reaches into the next one
        sg.xcut[s] = s == 0 ? 0 : (size_t)(x_lo[s] - xb);
        sg.ycut[s] = s == 0 ? 0 : (size_t)(y_lo[s] - yb);
        const size_t need = batch_workspace_core(problems + sg.cut[s], n);
        if (need == 0) return false;
        sg.ws_off[s + 1] = sg.ws_off[s] + align_up(need, 1024);
    }
    sg.xcut[kHostSegments] = x_bytes;
    sg.ycut[kHostSegments] = y_bytes;
    if (sg.ws_off[kHostSegments] > ws_bytes) return false;
    *out = sg;
    return true;
}

struct HostPipe {
    cudaStream_t side[kHostSegments - 1];
    cudaEvent_t fork, done[kHostSegments - 1];
    bool tried = false, ok = false;
};
std::mutex g_host_pipe_mu;  // held while a call enqueues its segments: the streams and events are shared per device
HostPipe g_host_pipe[64];

HostPipe* host_pipe_locked() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return nullptr;
    }
    HostPipe& hp = g_host_pipe[dev];
    if (!hp.tried) {
        hp.tried = true;
        bool ok = cudaEventCreateWithFlags(&hp.fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < kHostSegments - 1 && ok; ++i)
            ok = cudaStreamCreateWithFlags(&hp.side[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) cudaGetLastError();
        hp.ok = ok;
    }
    return hp.ok ? &hp : nullptr;
}

}  // namespace

namespace {
size_t batch_workspace_core(const bitlinear_problem* problems, int count) {
    if (!problems || count <= 0) return 0;
    std::vector<bitlinear_problem> dec;
    std::vector<int32_t*> dec_acc;
    std::vector<int> pre;
    if (partition_problems(problems, count, nullptr, dec, dec_acc, pre) != BITLINEAR_OK) return 0;
    size_t total = 0;
    if (!dec.empty()) total += align_up(decode_batch_workspace_bytes(dec.data(), (int)dec.size()), 1024);
    if (!pre.empty()) total += prefill_group_workspace_bytes(problems, pre.data(), (int)pre.size());
    return total;
}
}  // namespace

extern "C" {

size_t bitlinear_batch_workspace_bytes(const bitlinear_problem* problems, int count) {
    // bitlinear_forward_batch_host may run a long decode call as kHostSegments calls with a plan each
    return std::max(batch_workspace_core(problems, count), host_segments_workspace(problems, count));
}

int bitlinear_forward_batch(const bitlinear_problem* problems, int count, int flags, void* ws, size_t ws_bytes,
                            void* stream) {
    return bitlinear_forward_batch_acc(problems, count, flags, nullptr, ws, ws_bytes, stream);
}

int bitlinear_forward_batch_acc(const bitlinear_problem* problems, int count, int flags, int32_t* const* acc_out,
                                void* ws, size_t ws_bytes, void* stream) {
    if (count < 0) return BITLINEAR_ERR_SHAPE;
    if (count == 0) return BITLINEAR_OK;
    if (!problems) return BITLINEAR_ERR_NULL;
    if (flags & ~(BITLINEAR_BATCH_REUSE_PLAN | BITLINEAR_BATCH_REUSE_ACT | BITLINEAR_BATCH_REUSE_WEIGHTS)) return BITLINEAR_ERR_DTYPE;
    std::vector<bitlinear_problem> dec;
    std::vector<int32_t*> dec_acc;
    std::vector<int> pre;
    if (const int rc = partition_problems(problems, count, acc_out, dec, dec_acc, pre)) return rc;
    const size_t dec_bytes = dec.empty() ? 0 : align_up(decode_batch_workspace_bytes(dec.data(), (int)dec.size()), 1024);
    const size_t pre_bytes = pre.empty() ? 0 : prefill_group_workspace_bytes(problems, pre.data(), (int)pre.size());
    if (!ws || !aligned16(ws) || ws_bytes < dec_bytes + pre_bytes) return BITLINEAR_ERR_WORKSPACE;
    if (!dec.empty()) {
        const int rc = decode_batch_forward(dec.data(), (int)dec.size(), flags & ~BITLINEAR_BATCH_REUSE_WEIGHTS, acc_out ? dec_acc.data() : nullptr, ws, dec_bytes, stream);
        if (rc != BITLINEAR_OK) return rc;
    }
    if (!pre.empty()) {
        if (int rc = [] {
                int dev = 0, major = 0;
                if (cudaGetDevice(&dev) != cudaSuccess ||
                    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
                    cudaGetLastError();
                    return (int)BITLINEAR_ERR_CUDA;
                }
                return major == 10 ? (int)BITLINEAR_OK : (int)BITLINEAR_ERR_ARCH;
            }())
            return rc;
        return prefill_group_forward(problems, pre.data(), (int)pre.size(), static_cast<char*>(ws) + dec_bytes,
                                     (flags & BITLINEAR_BATCH_REUSE_ACT) != 0, (flags & BITLINEAR_BATCH_REUSE_WEIGHTS) != 0,
                                     static_cast<cudaStream_t>(stream));
    }
    return BITLINEAR_OK;
}

int bitlinear_forward_batch_host(const bitlinear_problem* problems, int count, int flags, const void* x_host,
                                 void* x_dev, size_t x_bytes, const void* y_dev, void* y_host, size_t y_bytes, void* ws,
                                 size_t ws_bytes, void* stream) {
    if (count > 0 && (!x_host || !x_dev || !y_dev || !y_host)) return BITLINEAR_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    HostSegments sg;
    if (count > 0 && problems && ws && plan_host_segments(problems, count, x_dev, x_bytes, y_dev, y_bytes, ws_bytes, &sg)) {
        std::unique_lock<std::mutex> lock(g_host_pipe_mu);
        if (HostPipe* hp = host_pipe_locked()) {
            // segment 0 runs on the caller's stream, the others on side streams that start after the caller's earlier work
            // and that the caller's stream waits for at the end
            bool cuda_ok = cudaEventRecord(hp->fork, st) == cudaSuccess;
            for (int i = 0; i < kHostSegments - 1 && cuda_ok; ++i) cuda_ok = cudaStreamWaitEvent(hp->side[i], hp->fork, 0) == cudaSuccess;
            int rc = BITLINEAR_OK;
            for (int s = 0; s < kHostSegments && cuda_ok && rc == BITLINEAR_OK; ++s) {
                cudaStream_t ss = s == 0 ? st : hp->side[s - 1];
                const size_t xn = sg.xcut[s + 1] - sg.xcut[s], yn = sg.ycut[s + 1] - sg.ycut[s];
                if (xn > 0)
                    cuda_ok = cudaMemcpyAsync(static_cast<char*>(x_dev) + sg.xcut[s], static_cast<const char*>(x_host) + sg.xcut[s], xn,
                                              cudaMemcpyHostToDevice, ss) == cudaSuccess;
                if (cuda_ok)
                    rc = bitlinear_forward_batch(problems + sg.cut[s], sg.cut[s + 1] - sg.cut[s], flags, static_cast<char*>(ws) + sg.ws_off[s],
                                                 sg.ws_off[s + 1] - sg.ws_off[s], ss);
                if (cuda_ok && rc == BITLINEAR_OK && yn > 0)
                    cuda_ok = cudaMemcpyAsync(static_cast<char*>(y_host) + sg.ycut[s], static_cast<const char*>(y_dev) + sg.ycut[s], yn,
                                              cudaMemcpyDeviceToHost, ss) == cudaSuccess;
            }
            // join whatever was started, also after an error
            for (int i = 0; i < kHostSegments - 1; ++i)
                if (cudaEventRecord(hp->done[i], hp->side[i]) != cudaSuccess || cudaStreamWaitEvent(st, hp->done[i], 0) != cudaSuccess)
                    cuda_ok = false;
            lock.unlock();
            if (cudaStreamSynchronize(st) != cudaSuccess) cuda_ok = false;
            if (rc != BITLINEAR_OK) return rc;
            if (!cuda_ok) {
                cudaGetLastError();
                return BITLINEAR_ERR_CUDA;
            }
            return BITLINEAR_OK;
        }
    }
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
