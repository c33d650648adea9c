// Prefill contraction (M > 16 tokens): int8 activations x uint8 weight codes on the 5th-generation
// tensor cores (tcgen05.mma kind::i8, s8 x u8 -> s32) with accumulators in tensor memory.
// (Paper Section 5.1: the packed weights are expanded to a form the matrix units can consume right
// before the product with the 8-bit activations; here the expansion target is the code c = Wq + 1,
// and the epilogue removes the offset with the per-token code sum.)
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0   : producer      - per stage a 128B-swizzled TMA tile of A (tokens x K) and one linear 32 KiB
//              bulk copy of B (the weight codes are laid out in global memory as the shared-memory images
//              of their 256 x 128 tiles) into a 4-stage shared-memory ring, completion on mbarriers
//   warp 1   : MMA issuer    - one elected thread issues tcgen05.mma 128 x 256 x 32 and commits
//   warps 2-5: epilogue      - tcgen05.ld of a finished 128 x 256 int32 accumulator, subtract the
//              code sum, two fp32 multiplies, store; tensor memory is double buffered so the
//              epilogue of tile i overlaps the main loop of tile i+1.
// Every wait is bounded: if one runs out the CTA raises a sticky status word and leaves cleanly.
#include <cuda.h>

#include <cstring>
#include <mutex>

#include "common.cuh"
#include "sm100_sync.cuh"
#include "tensor_map.cuh"

namespace bitlinear {

namespace {

constexpr int BM = 128;   // tokens per tile (UMMA M, one per tensor-memory lane)
constexpr int BN = 256;   // weight rows per tile (UMMA N, one per tensor-memory column)
constexpr int BK = 128;   // bytes of K per pipeline stage = one 128-byte swizzle row
constexpr int UMMA_K = 32;
constexpr int STAGES = 4;
constexpr uint32_t A_BYTES = BM * BK;
constexpr uint32_t B_BYTES = BN * BK;
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;  // two accumulator buffers of 256 columns
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + 256 /*barriers*/ + 4 * 32 * 144 /*epilogue staging*/ + 3072 /*group table*/;
// ---- thin PTX wrappers (mbarrier, bulk copy and the bounded wait come from sm100_sync.cuh) --------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
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

__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes with the 128-byte
// swizzle: 8-row groups are 1024 bytes apart (stride offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t desc = 0;
    desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    desc |= (uint64_t)1 << 16;                    // leading byte offset (unused with swizzle): 1
    desc |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
    desc |= (uint64_t)1 << 46;                    // descriptor version for this architecture
    desc |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return desc;
}

// Instruction descriptor: D = s32, A = s8 (activations), B = u8 (weight codes), both K-major.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
    return (2u << 4) | (1u << 7) | (0u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Epilogue staging: a warp holds a 32-row x 32-column block with one row per lane.  It is written to shared
// memory (row stride 144 bytes keeps the eight 16-byte stores of a quarter warp on distinct banks), read back with
// eight lanes per row, and stored with each instruction covering four whole 128-byte row segments.
constexpr uint32_t STAGE_ROW_B32 = 144;
constexpr uint32_t STAGE_ROW_B16 = 80;
constexpr uint32_t STAGE_OUT_BYTES = 32 * STAGE_ROW_B32;  // per epilogue warp

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// vals: this lane's row (32 x 32-bit).  dst: element (row 0, column 0) of the block in a row-major matrix of
// leading dimension ld (elements); rows >= rows_ok are not stored.
__device__ __forceinline__ void store_block_b32(const uint32_t (&vals)[32], uint32_t stage_s, uint32_t* dst, int ld,
                                                int rows_ok, int lane) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
        sts128(stage_s + lane * STAGE_ROW_B32 + 16 * i, vals[4 * i], vals[4 * i + 1], vals[4 * i + 2], vals[4 * i + 3]);
    __syncwarp();
    const int sub = lane >> 3, piece = lane & 7;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const int row = 4 * it + sub;
        const uint4 v = lds128(stage_s + row * STAGE_ROW_B32 + 16 * piece);
        if (row < rows_ok) *reinterpret_cast<uint4*>(dst + (size_t)row * ld + 4 * piece) = v;
    }
    __syncwarp();
}

// Same for 16-bit elements: vals holds this lane's 32 columns as 16 packed words (64 bytes per row).
__device__ __forceinline__ void store_block_b16(const uint32_t (&vals)[16], uint32_t stage_s, uint16_t* dst, int ld,
                                                int rows_ok, int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
        sts128(stage_s + lane * STAGE_ROW_B16 + 16 * i, vals[4 * i], vals[4 * i + 1], vals[4 * i + 2], vals[4 * i + 3]);
    __syncwarp();
    const int sub = lane >> 2, piece = lane & 3;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = 8 * it + sub;
        const uint4 v = lds128(stage_s + row * STAGE_ROW_B16 + 16 * piece);
        if (row < rows_ok) *reinterpret_cast<uint4*>(dst + (size_t)row * ld + 8 * piece) = v;
    }
    __syncwarp();
}

// Epilogue of one warp for one accumulator: 32 tensor-memory lanes (token rows m_warp .. m_warp+31) x 256 columns
// (weight rows n0 .. n0+255) starting at tensor-memory address taddr.  Subtracts the code offset, dequantises, stores.
__device__ __forceinline__ void drain_accumulator(const GemmProblem& p, uint32_t taddr, int m_warp, int n0, uint32_t stage_s,
                                                  int lane) {
    const int M = p.M, N = p.N, y_dtype = p.y_dtype;
    void* y = p.y;
    int32_t* acc_out = p.acc_out;
    const float s_w = *p.s_w;
    const int m = m_warp + lane;
    const bool row_ok = m < M;
    // read through L2: the quantiser launch that wrote them may still be running beside this kernel (other rows)
    const int xs = row_ok ? __ldcg(p.xsum + m) : 0;
    const float dm = row_ok ? __ldcg(p.d + m) : 0.0f;
    const int rows_ok = (M - m_warp) < 32 ? (M - m_warp) : 32;
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(taddr + c * 32, r);
        tmem_ld_wait();
        const int n = n0 + c * 32;
        if (n < N && rows_ok > 0) {  // warp-uniform
            // Each lane holds 32 consecutive columns of ONE row.  The block goes through this warp's
            // shared-memory staging area so that every global store covers whole 128-byte row segments.
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = (uint32_t)((int)r[i] - xs);
            if (acc_out != nullptr)
                store_block_b32(r, stage_s, reinterpret_cast<uint32_t*>(acc_out) + (size_t)m_warp * N + n, N, rows_ok, lane);
            if (y_dtype == BITLINEAR_BF16) {
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float v0 = __fmul_rn(__fmul_rn((float)(int)r[2 * i], s_w), dm);
                    const float v1 = __fmul_rn(__fmul_rn((float)(int)r[2 * i + 1], s_w), dm);
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(v0, v1);
                    w[i] = *reinterpret_cast<const uint32_t*>(&pk);
                }
                store_block_b16(w, stage_s, reinterpret_cast<uint16_t*>(y) + (size_t)m_warp * N + n, N, rows_ok, lane);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__fmul_rn(__fmul_rn((float)(int)r[i], s_w), dm));
                store_block_b32(r, stage_s, reinterpret_cast<uint32_t*>(y) + (size_t)m_warp * N + n, N, rows_ok, lane);
            }
        }
    }
}

// Tile -> (problem, token rows, weight rows).  Tiles of one problem are numbered with the token tile
// fastest, so CTAs that run side by side share the weight tile; problems follow each other in table order.
__device__ __forceinline__ int ld_acquire_gpu_s32(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

struct TileWalk {
    const GemmProblem* probs;
    int count, pi;
    __device__ __forceinline__ const GemmProblem& find(int tile) {
        while (pi + 1 < count && tile >= probs[pi + 1].tile_begin) ++pi;
        return probs[pi];
    }
};

// A_TILED: the activations come as tile images and are fetched with linear bulk copies (any group size);
// otherwise the group holds one problem whose row-major activations are fetched through the tensor map.
template <bool A_TILED>
__global__ void __launch_bounds__(THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const uint8_t* __restrict__ table_g, int* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t* full_bar = bars;                 // [STAGES] TMA bytes landed
    uint64_t* empty_bar = bars + STAGES;       // [STAGES] MMAs that read the stage retired
    uint64_t* tfull_bar = bars + 2 * STAGES;   // [2] accumulator buffer complete
    uint64_t* tempty_bar = tfull_bar + 2;      // [2] accumulator buffer drained by the epilogue
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* table_s = smem + (size_t)STAGES * STAGE_BYTES + 256 + 4 * STAGE_OUT_BYTES;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the group table goes to shared memory once; every role walks it on its own
    for (int o = threadIdx.x * 16; o < (int)kGroupTableBytes; o += THREADS * 16)
        *reinterpret_cast<uint4*>(table_s + o) = *reinterpret_cast<const uint4*>(table_g + o);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(tfull_bar + b), 1);
            mbar_init(smem_u32(tempty_bar + b), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const GemmGroupHeader hdr = *reinterpret_cast<const GemmGroupHeader*>(table_s);
    const int total_tiles = hdr.total_tiles;
    TileWalk walk{reinterpret_cast<const GemmProblem*>(table_s + sizeof(GemmGroupHeader)), hdr.count, 0};

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
                const GemmProblem& p = walk.find(tile);
                const int lt = tile - p.tile_begin, mt = lt % p.m_tiles, nt = lt / p.m_tiles;
                const int k_blocks = p.K / BK;
                const uint8_t* a_src = A_TILED ? p.a_tiles + (size_t)mt * k_blocks * A_BYTES : nullptr;
                const uint8_t* b_src = p.codes + (size_t)nt * k_blocks * B_BYTES;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = smem_u32(full_bar + stage);
                    mbar_expect_tx(fb, STAGE_BYTES);
                    const uint32_t sa = smem_u32(smem + (size_t)stage * STAGE_BYTES);
                    if (A_TILED) bulk_load(sa, a_src + (size_t)kb * A_BYTES, A_BYTES, fb);
                    else tma_load_2d(sa, &map_a, kb * BK, mt * BM, fb);
                    bulk_load(sa + A_BYTES, b_src + (size_t)kb * B_BYTES, B_BYTES, fb);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BM, BN);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int iter = 0;
            for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++iter) {
                const int k_blocks = walk.find(tile).K / BK;
                const uint32_t buf = (uint32_t)iter & 1u, bphase = ((uint32_t)iter >> 1) & 1u;
                if (!mbar_wait(smem_u32(tempty_bar + buf), bphase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(full_bar + stage), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)stage * STAGE_BYTES);
                    const uint64_t a_desc = make_smem_desc(sa);
                    const uint64_t b_desc = make_smem_desc(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // advance both operands by 32 bytes of K inside the swizzled row
                        umma_i8(d_tmem, a_desc + (uint64_t)(k * UMMA_K / 16), b_desc + (uint64_t)(k * UMMA_K / 16), idesc,
                                (uint32_t)((kb | k) != 0));
                    }
                    umma_commit(smem_u32(empty_bar + stage));  // frees the stage once these MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(tfull_bar + buf));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;  // tensor-memory lanes 32*quad .. 32*quad+31 belong to this warp
        const uint32_t stage_s = smem_u32(smem + (size_t)STAGES * STAGE_BYTES + 256) + (uint32_t)quad * STAGE_OUT_BYTES;
        bool ok = true;
        int iter = 0;
        for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++iter) {
            const GemmProblem& p = walk.find(tile);
            const int lt = tile - p.tile_begin, mt = lt % p.m_tiles, nt = lt / p.m_tiles;
            const uint32_t buf = (uint32_t)iter & 1u, bphase = ((uint32_t)iter >> 1) & 1u;
            const int m_warp = mt * BM + quad * 32;  // first token row of this warp's 32 tensor-memory lanes
            if (!mbar_wait(smem_u32(tfull_bar + buf), bphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            drain_accumulator(p, tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN, m_warp, nt * BN, stage_s, lane);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(tempty_bar + buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        abort_drain();  // copies that may still be in flight land before shared memory is released
        if (threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ================================================================================================
// CTA-pair variant (cta_group::2): two CTAs of a cluster share one 256 x 256 tile.  Each CTA stages its
// own 128 token rows of A and HALF of the weight tile (128 rows of B) per k-block, so a CTA ingests 32 KB
// per 512 tensor-pipe cycles (64 B/clk) instead of 48 KB; the leader CTA (cluster rank 0) issues the MMAs
// for both, each CTA drains its own 128 x 256 accumulator.  Operands are tile images (the grouped path);
// they are fetched with tensor-map copies in the .cta_group::2 form, which may signal the leader's
// mbarrier from either CTA: the tensor map views the whole workspace region as rows of 128 bytes, no
// swizzle (the images are stored swizzled).
// ================================================================================================
// PACKED variant: the CTA's half of the weight tile arrives as PACKED 2-bit codes (4 KiB per k-block, fetched with one
// 4-D tensor-map copy straight out of the packed matrix) and four more warps expand it in shared memory into the
// swizzled byte-code image the MMA reads.  No expansion launch, no code images in global memory, and a quarter of the
// weight bytes on the L2 -> SM path, which is what bounds this kernel.
constexpr uint32_t P_HALF_BYTES = 128 * BK;              // 128 rows x 128 bytes
constexpr uint32_t P_PACKED_BYTES = 128 * BK / 4;        // the same rows as 2-bit codes
template <bool PACKED> struct PairCfg {
    static constexpr int kStages = PACKED ? 5 : 6;
    static constexpr uint32_t kStageBytes = 2 * P_HALF_BYTES + (PACKED ? P_PACKED_BYTES : 0);  // A rows + half of B (+ packed)
    static constexpr int kThreads = PACKED ? THREADS + 128 : THREADS;
    static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256 + 4 * 32 * 144 + 3072;
};
constexpr uint32_t kPeerMask = 0xFEFFFFFFu;  // clears the cluster-rank bit of a shared::cluster address: the pair's rank-0 CTA

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// tensor-map copy whose completion bytes are counted on the LEADER CTA's mbarrier (same offset, rank bit cleared)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_local) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_local & kPeerMask)
        : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives (once the MMAs issued so far have retired) on the barrier at this offset in BOTH CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"((uint16_t)3)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar_local) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_local & kPeerMask) : "memory");
}
// 4-D tensor-map copy into this CTA's shared memory, completion bytes on this CTA's own mbarrier
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
        : "memory");
}

// A single matmul needs no table in global memory: header, problem and the tensor map of its packed weights travel as
// kernel parameters, so a single call is the launch alone (no host-to-device copies in front of it).
struct PairInline {
    GemmGroupHeader hdr;
    GemmProblem prob;
    alignas(64) CUtensorMap w_map;
    int use;  // 1: take the table from here instead of table_g / w_maps
};

template <bool PACKED>
__global__ void __launch_bounds__(PairCfg<PACKED>::kThreads, 1)
gemm_i8_pair_kernel(const __grid_constant__ CUtensorMap map, const uint8_t* __restrict__ table_g, const CUtensorMap* __restrict__ w_maps_g,
                    int* status_word, const __grid_constant__ PairInline inl) {
    constexpr int P_STAGES = PairCfg<PACKED>::kStages;
    constexpr uint32_t P_STAGE_BYTES = PairCfg<PACKED>::kStageBytes;
    constexpr int kThreadsAll = PairCfg<PACKED>::kThreads;
    extern __shared__ uint8_t smem_raw[];
    // the rounding of the base is the same in both CTAs (same launch, same dynamic offset), so operand offsets match
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)P_STAGES * P_STAGE_BYTES);
    uint64_t* full_bar = bars;                    // [P_STAGES] leader: both CTAs' operand bytes landed
    uint64_t* empty_bar = bars + P_STAGES;        // [P_STAGES] each CTA: the MMAs that read the stage retired
    uint64_t* tfull_bar = bars + 2 * P_STAGES;    // [2] each CTA: accumulator buffer complete
    uint64_t* tempty_bar = tfull_bar + 2;         // [2] leader: drained by the 8 epilogue warps of the pair
    uint64_t* pfull_bar = tempty_bar + 2;         // [P_STAGES] each CTA (PACKED): its packed weight bytes landed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pfull_bar + P_STAGES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* table_s = smem + (size_t)P_STAGES * P_STAGE_BYTES + 256 + 4 * STAGE_OUT_BYTES;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = (int)blockIdx.x >> 1, n_pairs = (int)gridDim.x >> 1;
    const CUtensorMap* w_maps = inl.use ? &inl.w_map : w_maps_g;
    if (inl.use) {
        if (threadIdx.x == 0) {
            *reinterpret_cast<GemmGroupHeader*>(table_s) = inl.hdr;
            *reinterpret_cast<GemmProblem*>(table_s + sizeof(GemmGroupHeader)) = inl.prob;
        }
    } else {
        for (int o = threadIdx.x * 16; o < (int)kGroupTableBytes; o += kThreadsAll * 16)
            *reinterpret_cast<uint4*>(table_s + o) = *reinterpret_cast<const uint4*>(table_g + o);
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) {
            // PACKED: the leader's barrier also counts the eight expander warps of the pair (the code image is written)
            mbar_init(smem_u32(full_bar + s), PACKED ? 9 : 1);
            mbar_init(smem_u32(empty_bar + s), 1);
            mbar_init(smem_u32(pfull_bar + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(tfull_bar + b), 1);
            mbar_init(smem_u32(tempty_bar + b), 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // the same warp of both CTAs allocates for the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const GemmGroupHeader hdr = *reinterpret_cast<const GemmGroupHeader*>(table_s);
    const int total_tiles = hdr.total_tiles;  // counted in 256 x 256 pair tiles (m_tiles = ceil(M / 256))
    TileWalk walk{reinterpret_cast<const GemmProblem*>(table_s + sizeof(GemmGroupHeader)), hdr.count, 0};

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int ready_idx = -1;  // last weight tile whose codes are known to be complete
            if (hdr.wait_primary) asm volatile("griddepcontrol.wait;" ::: "memory");  // token images: quantiser launch
            for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
                const GemmProblem& p = walk.find(tile);
                const int lt = tile - p.tile_begin, mt = lt % p.m_tiles, nt = lt / p.m_tiles;
                const int k_blocks = p.K / BK;
                if (hdr.ready != nullptr && p.nt_begin + nt != ready_idx) {
                    // the expansion launch may still be writing this weight tile's codes: wait for its word count (bounded)
                    const int target = min(BN, p.N - nt * BN) * (p.K / 16);
                    const unsigned long long t0 = globaltimer_ns();
                    unsigned spins = 0;
                    while (ld_acquire_gpu_s32(hdr.ready + p.nt_begin + nt) < target) {
                        if ((++spins & 63u) == 0u) {
                            if (*abort_flag) { ok = false; break; }
                            if (globaltimer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; ok = false; break; }
                        }
                    }
                    if (!ok) break;
                    asm volatile("fence.proxy.async;" ::: "memory");  // the copies below read what generic stores wrote
                    ready_idx = p.nt_begin + nt;
                }
                if (hdr.a_ready != nullptr) {
                    // the quantiser launch may still be writing this token tile: wait for its token count (bounded)
                    const int target = min(256, p.M - mt * 256);
                    const unsigned long long t0 = globaltimer_ns();
                    unsigned spins = 0;
                    while (ld_acquire_gpu_s32(hdr.a_ready + p.at_begin + mt) < target) {
                        if ((++spins & 63u) == 0u) {
                            if (*abort_flag) { ok = false; break; }
                            if (globaltimer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; ok = false; break; }
                        }
                    }
                    if (!ok) break;
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                // rows (of 128 bytes) of this CTA's operand images inside the mapped region
                const int a_row = (int)((reinterpret_cast<unsigned long long>(p.a_tiles) - hdr.region_base) >> 7) +
                                  (2 * mt + (int)rank) * k_blocks * 128;
                const int b_row = (int)((reinterpret_cast<unsigned long long>(p.codes) - hdr.region_base) >> 7) +
                                  nt * k_blocks * 256 + (int)rank * 128;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = smem_u32(full_bar + stage);
                    const uint32_t sa = smem_u32(smem + (size_t)stage * P_STAGE_BYTES);
                    if constexpr (PACKED) {
                        if (leader) mbar_expect_tx(fb, 2 * P_HALF_BYTES);  // the token rows of both CTAs
                        // tokens: a tile image (already swizzled, the map has rows of 128 bytes) or, for a single matmul on
                        // row-major activations, a 128-row x 128-byte box of the [M][K] matrix through a swizzling map
                        if (hdr.a_row_major) tma_load_2d_pair(sa, &map, kb * BK, mt * 256 + (int)rank * 128, fb);
                        else tma_load_2d_pair(sa, &map, 0, a_row + kb * 128, fb);
                        // this CTA's 128 weight rows x 128 columns as packed codes: 8 row blocks x 16 rows x 32 bytes of the
                        // packed matrix (half of the 16 x 256 tile kb / 2 of each row block)
                        const uint32_t pb = smem_u32(pfull_bar + stage);
                        mbar_expect_tx(pb, P_PACKED_BYTES);
                        tma_load_4d(sa + 2 * P_HALF_BYTES, w_maps + walk.pi, 32 * (kb & 1), 0, kb >> 1, 16 * nt + 8 * (int)rank, pb);
                    } else {
                        if (leader) mbar_expect_tx(fb, 2 * P_STAGE_BYTES);  // its own copies and the peer's
                        tma_load_2d_pair(sa, &map, 0, a_row + kb * 128, fb);
                        tma_load_2d_pair(sa + P_HALF_BYTES, &map, 0, b_row + kb * 256, fb);
                    }
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && lane == 0) {
            constexpr uint32_t idesc = make_idesc(256, BN);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int iter = 0;
            for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++iter) {
                const int k_blocks = walk.find(tile).K / BK;
                const uint32_t buf = (uint32_t)iter & 1u, bphase = ((uint32_t)iter >> 1) & 1u;
                if (!mbar_wait(smem_u32(tempty_bar + buf), bphase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(full_bar + stage), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)stage * P_STAGE_BYTES);
                    const uint64_t a_desc = make_smem_desc(sa);
                    const uint64_t b_desc = make_smem_desc(sa + P_HALF_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_i8_pair(d_tmem, a_desc + (uint64_t)(k * UMMA_K / 16), b_desc + (uint64_t)(k * UMMA_K / 16), idesc,
                                     (uint32_t)((kb | k) != 0));
                    umma_commit_pair(smem_u32(empty_bar + stage));  // frees the stage in both CTAs
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit_pair(smem_u32(tfull_bar + buf));
            }
        }
        __syncwarp();
    } else if (PACKED && warp >= 6) {
        // ------------------------------------------------------------------ expanders (PACKED; both CTAs, own half of B)
        // Packed staging: [8 row blocks][16 rows][32 bytes]; word w of row r holds columns 16 w .. 16 w + 15 of the
        // k-block, byte b bits 2j = column 4 j + b: (word >> 2 j) & 0x03030303 is the 4 bytes 4 j .. 4 j + 3 of the
        // 16-byte piece w of the row's 128-byte code row, which sits swizzled at r * 128 + ((w ^ (r & 7)) * 16).
        const int et = (int)threadIdx.x - 192;   // 0..127
        const int piece = et & 7, r0 = et >> 3;  // a quarter warp writes one whole 128-byte row per store
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
            const int k_blocks = walk.find(tile).K / BK;
            for (int kb = 0; kb < k_blocks; ++kb) {
                if (!mbar_wait(smem_u32(pfull_bar + stage), phase, abort_flag)) { ok = false; break; }
                const uint32_t sb = smem_u32(smem + (size_t)stage * P_STAGE_BYTES) + P_HALF_BYTES;
                const uint32_t sp = sb + P_HALF_BYTES;
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[i]) : "r"(sp + (uint32_t)(r0 + 16 * i) * 32u + 4u * piece));
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = r0 + 16 * i;
                    sts128(sb + (uint32_t)r * 128u + (uint32_t)((piece ^ (r & 7)) << 4), w[i] & 0x03030303u, (w[i] >> 2) & 0x03030303u,
                           (w[i] >> 4) & 0x03030303u, (w[i] >> 6) & 0x03030303u);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMA reads what these stores wrote
                __syncwarp();
                if (lane == 0) mbar_arrive_leader(smem_u32(full_bar + stage));
                if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        const int quad = warp & 3;
        const uint32_t stage_s = smem_u32(smem + (size_t)P_STAGES * P_STAGE_BYTES + 256) + (uint32_t)quad * STAGE_OUT_BYTES;
        bool ok = true;
        int iter = 0;
        if (hdr.wait_primary) asm volatile("griddepcontrol.wait;" ::: "memory");  // scales, code sums: quantiser launch
        for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++iter) {
            const GemmProblem& p = walk.find(tile);
            const int lt = tile - p.tile_begin, mt = lt % p.m_tiles, nt = lt / p.m_tiles;
            const uint32_t buf = (uint32_t)iter & 1u, bphase = ((uint32_t)iter >> 1) & 1u;
            const int m_warp = mt * 256 + (int)rank * 128 + quad * 32;
            if (!mbar_wait(smem_u32(tfull_bar + buf), bphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            drain_accumulator(p, tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN, m_warp, nt * BN, stage_s, lane);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(smem_u32(tempty_bar + buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        abort_drain();
        if (threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
        __syncthreads();
    }
    cluster_sync_all();  // neither CTA frees tensor memory or leaves while the other may still use the pair's resources
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ================================================================================================
// Rate probe: how fast this GPU issues and retires tcgen05.mma kind::i8 when nothing else limits it.  Every CTA
// (one per SM) fills one 128 x 128-byte A image and one 256 x 128-byte B image in shared memory once, then one thread
// issues n_mma MMAs of 128 x 256 x 32 on them, alternating between the two accumulator halves of tensor memory; no
// global memory traffic, no epilogue.  The benchmark divides the operations by the launch's device time and uses the
// result as the denominator of the prefill numbers (a measured int8 peak instead of a datasheet figure).
// ================================================================================================
__global__ void __launch_bounds__(128, 1) int8_mma_rate_kernel(int n_mma, int* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t done_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    for (uint32_t o = threadIdx.x * 16; o < STAGE_BYTES; o += blockDim.x * 16)
        *reinterpret_cast<uint4*>(smem + o) = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&done_bar), 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read what generic stores wrote
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    if (threadIdx.x == 0) {
        constexpr uint32_t idesc = make_idesc(BM, BN);
        const uint64_t a_desc = make_smem_desc(smem_u32(smem)), b_desc = make_smem_desc(smem_u32(smem) + A_BYTES);
        for (int i = 0; i < n_mma; ++i)
            umma_i8(tmem_base + (uint32_t)(i & 1) * BN, a_desc + (uint64_t)((i & 3) * UMMA_K / 16),
                    b_desc + (uint64_t)((i & 3) * UMMA_K / 16), idesc, (uint32_t)(i > 1));
        umma_commit(smem_u32(&done_bar));  // arrives once every MMA above has retired
        mbar_wait(smem_u32(&done_bar), 0u, &abort_flag);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
    if (threadIdx.x < 32) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------

// 2-D map over a row-major [rows][K] byte matrix; box = box_rows x 128 bytes, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t gemm_codes_bytes(int N, int K) { return (size_t)((N + BN - 1) / BN) * BN * K; }  // whole 256-row tiles
size_t gemm_a_tiles_bytes(int M, int K) { return (size_t)((M + 255) / 256) * 256 * K; }  // whole pairs of 128-row tiles
size_t gemm_scratch_bytes(int N, int K) { return align_up(gemm_codes_bytes(N, K), 256) + align_up(kGroupTableDevBytes, 256); }

// The whole region [base, base + bytes) as a matrix of 128-byte rows, box = 128 rows, no swizzle: a tile image (stored
// swizzled) is copied as it is.
bool make_map_rows128(CUtensorMap* map, const void* base, size_t bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || (reinterpret_cast<uintptr_t>(base) & 127u) || bytes < 128 * 128) return false;
    const cuuint64_t dims[2] = {128, (cuuint64_t)(bytes / 128)};
    const cuuint64_t strides[1] = {128};
    const cuuint32_t box[2] = {128, 128};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 4-D view of a packed [N][K] matrix for the PACKED pair kernel: x = 64 bytes of a tile row, y = the 16 rows of a tile,
// z = the K / 256 tiles of a row block, w = the N / 16 row blocks; box = 32 bytes x 16 rows x 1 tile x 8 row blocks, i.e.
// 128 weight rows x 128 columns of 2-bit codes (4 KiB) per copy.
bool make_map_packed(CUtensorMap* map, const void* packed, int N, int K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || (reinterpret_cast<uintptr_t>(packed) & 15u)) return false;
    const cuuint64_t k_tiles = (cuuint64_t)(K / kTileCols);
    const cuuint64_t dims[4] = {64, 16, k_tiles, (cuuint64_t)(N / kTileRows)};
    const cuuint64_t strides[3] = {64, (cuuint64_t)kTileBytes, k_tiles * kTileBytes};
    const cuuint32_t box[4] = {32, 16, 1, 8};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(packed), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int gemm_launch(GemmProblem* probs, int count, bool a_tiled, const int8_t* xq_row_major, uint8_t* table_dev,
                cudaStream_t st, const void* region_base, size_t region_bytes, const int* ready, GemmBeforeKernel before,
                void* before_ctx, bool wait_primary, const int* a_ready, const void* const* packed) {
    // kernel attributes and the SM count are per device: set / looked up once for each device a process uses
    int sm_count = 0;
    {
        static std::mutex mu;
        static int sm_of[64];  // 0 = this device has not been set up yet
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        std::lock_guard<std::mutex> lock(mu);
        if (sm_of[dev] == 0) {
            int n = 0;
            if (cudaFuncSetAttribute(gemm_i8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess ||
                cudaFuncSetAttribute(gemm_i8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess ||
                cudaFuncSetAttribute(gemm_i8_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairCfg<false>::kSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(gemm_i8_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairCfg<true>::kSmemBytes) != cudaSuccess ||
                cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
                cudaGetLastError();
                return BITLINEAR_ERR_CUDA;
            }
            sm_of[dev] = n;
        }
        sm_count = sm_of[dev];
    }
    if (count < 1 || count > kMaxGroup || (!a_tiled && count != 1)) return BITLINEAR_ERR_SHAPE;
    alignas(16) uint8_t host[kGroupTableBytes] = {};
    GemmGroupHeader* hdr = reinterpret_cast<GemmGroupHeader*>(host);
    GemmProblem* tab = reinterpret_cast<GemmProblem*>(host + sizeof(GemmGroupHeader));
    // CTA pairs (256 x 256 tiles) when the operands are tile images inside one mapped region and the SMs pair up
    const bool pairs = (sm_count % 2) == 0 && ((a_tiled && region_base != nullptr) || (!a_tiled && packed != nullptr));
    const int tile_m = pairs ? 256 : BM;
    int tiles = 0, n_tiles = 0;
    for (int i = 0; i < count; ++i) {
        probs[i].m_tiles = (probs[i].M + tile_m - 1) / tile_m;
        probs[i].tile_begin = tiles;
        probs[i].nt_begin = n_tiles;
        tiles += probs[i].m_tiles * ((probs[i].N + BN - 1) / BN);
        n_tiles += (probs[i].N + BN - 1) / BN;
        tab[i] = probs[i];
    }
    hdr->count = count;
    hdr->total_tiles = tiles;
    hdr->region_base = reinterpret_cast<unsigned long long>(region_base);
    // PACKED mode: the weights are read as packed codes through one tensor map per problem and expanded in the kernel
    const bool packed_mode = pairs && packed != nullptr;
    hdr->ready = (pairs && !packed_mode) ? ready : nullptr;
    hdr->a_ready = pairs ? a_ready : nullptr;
    hdr->a_row_major = (pairs && !a_tiled) ? 1 : 0;
    // griddepcontrol.wait in the kernel: only where the launch before it is the quantiser and no token-tile counters follow it
    const bool dependent = pairs && (hdr->ready != nullptr || hdr->a_ready != nullptr);
    hdr->wait_primary = (dependent && hdr->a_ready == nullptr && wait_primary) ? 1 : 0;
    // a single matmul on packed weights carries its table in the kernel parameters: nothing to upload
    const bool inline_table = packed_mode && count == 1;
    PairInline inl;
    memset(&inl, 0, sizeof(inl));
    if (inline_table) {
        inl.hdr = *hdr;
        inl.prob = tab[0];
        inl.use = 1;
        if (!make_map_packed(&inl.w_map, packed[0], probs[0].N, probs[0].K)) return BITLINEAR_ERR_CUDA;
    } else if (cudaMemcpyAsync(table_dev, host, kGroupTableBytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    CUtensorMap* w_maps_dev = reinterpret_cast<CUtensorMap*>(table_dev + kGroupMapsOffset);
    if (packed_mode && !inline_table) {
        alignas(64) CUtensorMap maps[kMaxGroup];
        for (int i = 0; i < count; ++i)
            if (!make_map_packed(&maps[i], packed[i], probs[i].N, probs[i].K)) return BITLINEAR_ERR_CUDA;
        if (cudaMemcpyAsync(w_maps_dev, maps, sizeof(CUtensorMap) * count, cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
    }
    if (before != nullptr) {
        const int rc = before(before_ctx);
        if (rc != BITLINEAR_OK) return rc;
    }
    CUtensorMap map_a;
    memset(&map_a, 0, sizeof(map_a));
    if (pairs) {
        if (a_tiled ? !make_map_rows128(&map_a, region_base, region_bytes) : !make_map(&map_a, xq_row_major, probs[0].M, probs[0].K, 128))
            return BITLINEAR_ERR_CUDA;
        int n_pairs = tiles < sm_count / 2 ? tiles : sm_count / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * n_pairs));
        cfg.blockDim = dim3(packed_mode ? PairCfg<true>::kThreads : PairCfg<false>::kThreads);
        cfg.dynamicSmemBytes = packed_mode ? PairCfg<true>::kSmemBytes : PairCfg<false>::kSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // beside the expansion launch: the kernel waits per problem on the ready counters, not on the whole launch
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = dependent ? 2 : 1;
        const cudaError_t e = packed_mode ? cudaLaunchKernelEx(&cfg, gemm_i8_pair_kernel<true>, map_a, (const uint8_t*)table_dev,
                                                               (const CUtensorMap*)w_maps_dev, device_status_word(), inl)
                                          : cudaLaunchKernelEx(&cfg, gemm_i8_pair_kernel<false>, map_a, (const uint8_t*)table_dev,
                                                               (const CUtensorMap*)w_maps_dev, device_status_word(), inl);
        if (e != cudaSuccess) cudaGetLastError();
        return e == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
    }
    if (!a_tiled && !make_map(&map_a, xq_row_major, probs[0].M, probs[0].K, BM)) return BITLINEAR_ERR_CUDA;
    const int grid = tiles < sm_count ? tiles : sm_count;
    if (a_tiled) gemm_i8_kernel<true><<<grid, THREADS, SMEM_BYTES, st>>>(map_a, table_dev, device_status_word());
    else gemm_i8_kernel<false><<<grid, THREADS, SMEM_BYTES, st>>>(map_a, table_dev, device_status_word());
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

// Launches the rate probe on every SM; ops_out (host) receives the integer operations of the launch (2 per MAC).
int int8_mma_rate_probe(int n_mma, double* ops_out, cudaStream_t st) {
    int sm_count = 0;
    if (const int rc = device_sm_count(&sm_count)) return rc;
    const size_t smem = STAGE_BYTES + 1024;
    if (cudaFuncSetAttribute(int8_mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    int8_mma_rate_kernel<<<sm_count, 128, smem, st>>>(n_mma, device_status_word());
    if (cudaGetLastError() != cudaSuccess) return BITLINEAR_ERR_CUDA;
    if (ops_out) *ops_out = 2.0 * BM * BN * UMMA_K * (double)n_mma * sm_count;
    return BITLINEAR_OK;
}

// One matmul on row-major int8 activations; `scratch` holds the code tiles followed by the group table.
int gemm_tcgen05(const int8_t* xq, const float* d, const int32_t* xsum, const uint8_t* scratch, const float* s_w, int M,
                 int N, int K, void* y, int y_dtype, int32_t* acc_out, cudaStream_t st) {
    GemmProblem p = {};
    p.codes = scratch;
    p.d = d; p.xsum = xsum; p.s_w = s_w; p.y = y; p.acc_out = acc_out;
    p.M = M; p.N = N; p.K = K; p.y_dtype = y_dtype;
    uint8_t* table_dev = const_cast<uint8_t*>(scratch) + align_up(gemm_codes_bytes(N, K), 256);
    return gemm_launch(&p, 1, false, xq, table_dev, st);
}

// The same through the CTA-pair kernel that reads the packed weights themselves (no code tiles): `table_dev` holds
// kGroupTableDevBytes.  Returns BITLINEAR_ERR_ARCH-free status; the caller checks pairs_available() first.
int gemm_tcgen05_packed(const int8_t* xq, const float* d, const int32_t* xsum, const void* packed, const float* s_w, int M,
                        int N, int K, void* y, int y_dtype, int32_t* acc_out, uint8_t* table_dev, cudaStream_t st) {
    GemmProblem p = {};
    p.d = d; p.xsum = xsum; p.s_w = s_w; p.y = y; p.acc_out = acc_out;
    p.M = M; p.N = N; p.K = K; p.y_dtype = y_dtype;
    const void* packed_ptrs[1] = {packed};
    return gemm_launch(&p, 1, false, xq, table_dev, st, nullptr, 0, nullptr, nullptr, nullptr, false, nullptr, packed_ptrs);
}

bool gemm_pairs_available() {
    int sm_count = 0;
    return device_sm_count(&sm_count) == BITLINEAR_OK && (sm_count % 2) == 0;
}

}  // namespace bitlinear
