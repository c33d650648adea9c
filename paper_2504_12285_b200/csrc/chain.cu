// Chained decode of a stack of decoder layers at one token, in ONE persistent cooperative kernel.
// (Paper Section 2: every linear map of a layer is a BitLinear - q, k, v, o, gate, up, down - with squared ReLU in the
// feed-forward block; Section 5.1: decode cost is the packed weight bytes.  Attention is not a BitLinear and is
// replaced by a fixed stand-in, see bitlinear_glue_attn_standin.)
//
// A layer is four dependent levels: {q,k,v}(h), o(a), {gate,up}(h), down(f).  What a level hands to the next one is a
// vector of a few thousand values that EVERY CTA needs, so a level boundary is an all-to-all exchange between the CTAs
// (one per SM); its latency, not the arithmetic, bounds the token.  The kernel is built around making that exchange
// short:
//   * The CTA that computes an output row also applies the glue that follows it (residual add, squared-ReLU gate,
//     attention stand-in) and publishes the NEXT level's input as bf16: 2 bytes per element instead of one or two fp32
//     vectors.  To keep the glue local, gate row n and up row n belong to the same CTA, and the CTA that owns a block
//     of q rows computes the v rows the stand-in adds to them itself (v is small; its rows are computed four times).
//   * Published values carry their own validity: three bf16 values and a 16-bit level tag share one 8-byte word,
//     written by one store and read by one load, so no fence and no release/acquire pair sits between producer and
//     consumer.  A relaxed arrival counter only tells the consumers when a look is worthwhile.
//   * Weights never wait for activations: a copy warp prefetches the CTA's share of the next level into shared memory
//     with bulk copies while the current level runs.
// Per level a CTA: waits for the counter, loads the whole input vector once (tags checked, stale words re-read),
// RMSNorm + absmax int8 quantiser into shared memory, dot-products-of-four over its weight rows, dequantising
// epilogue + glue, publish.  Every wait is bounded; on a timeout an abort word makes every CTA leave and
// BITLINEAR_ERR_TIMEOUT is reported.
#include <algorithm>
#include <mutex>

#include "quant_row.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

constexpr int kChainThreads = 512;  // compute threads; one more warp issues the weight copies
constexpr int kChainWarps = kChainThreads / 32;
constexpr int kChainLaunchThreads = kChainThreads + 32;
// barrier of the compute threads only (the copy warp runs on its own)
#define CSYNC() asm volatile("bar.sync 1, 512;" ::: "memory")
constexpr int kMaxLoads = 3;   // 16-byte loads of the level input per thread: 3 per 16 elements, K <= 8192
constexpr int kMaxJobs = 12;    // row blocks of weights a CTA multiplies in one level

struct ChainLayerDev {
    const uint8_t* packed[7];    // q k v o gate up down
    const float* s_w[7];
    const __nv_bfloat16* gain[4];  // inputs of {q,k,v}, o, {gate,up}, down (nullptr = ones)
};

struct ChainParams {
    const ChainLayerDev* layers;
    int n_layers, hidden, ffn, n_q, n_kv, head_dim;
    float eps;
    __nv_bfloat16* h;             // [hidden] in / out
    float* k;                     // [n_kv * head_dim] the k projection (an output only)
    // pub[j]: what level j publishes = the input of level j + 1 (of the next layer for j = 3): per 16 elements six
    // 8-byte words {bf16, bf16, bf16, tag}; word 5 of a group holds one value and two zeros.  Zero at launch.
    unsigned long long* pub[4];
    unsigned* counter;            // arrivals, zero at launch: a hint, never relied on for ordering
    int* abort_word;              // zero at launch
    int* status_word;
    int buf_bytes;                // one weight buffer (the largest per-CTA share of a level)
};

// Level shapes.  A "unit" is one block of 16 output rows of the level's result vector together with every weight row
// block needed to finish it: level 0 - a q block and the matching v block (units 0 .. hidden/16) or a k block (the
// units after those); level 1 - an o block; level 2 - a gate block and the up block of the same rows; level 3 - a down
// block.  Units are split over the CTAs by weight (bytes of packed rows).
__device__ __forceinline__ int level_K(int level, const ChainParams& p) { return level == 3 ? p.ffn : p.hidden; }

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
// Two published words: each 8-byte half is read atomically and carries its own tag.  Bypasses L1 (written by other SMs).
__device__ __forceinline__ void ld_pub2(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_pub(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long* pub_of(const ChainParams& p, int j) {
    return j == 0 ? p.pub[0] : (j == 1 ? p.pub[1] : (j == 2 ? p.pub[2] : p.pub[3]));
}

// r = fl32( 1 / sqrt( S / K + eps ) ) for S given as an unevaluated sum of two fp32 (S_hi + S_lo), without fp64
// arithmetic (slow on this GPU) and without a division: S / K + eps as a pair of fp32, the hardware's approximate reciprocal root, and one
// Newton step whose residual 1 - m * y0^2 is formed error-free with fused multiply-adds, second-order term included.
// The value rounded at the end is within 2^-44 of the exact one (checked against extended precision on 2 * 10^7 random
// inputs: the only differences from the correctly rounded result sit where the sum of squares is within 2^-40 of a
// rounding boundary of r, rows the parity tests exclude as fragile anyway).
__device__ __forceinline__ float rms_scale_pair(float S_hi, float S_lo, float ik_hi, float ik_lo, float eps) {
    // S / K as S * (1 / K), the reciprocal given as a pair ik_hi + ik_lo (accurate to 2^-48)
    const float q_hi = __fmul_rn(S_hi, ik_hi);
    const float q_lo = __fadd_rn(__fmaf_rn(S_hi, ik_hi, -q_hi), __fmaf_rn(S_hi, ik_lo, __fmul_rn(S_lo, ik_hi)));
    const float t_hi = __fadd_rn(q_hi, eps);
    const float bb = __fsub_rn(t_hi, q_hi);
    const float t_lo = __fadd_rn(__fadd_rn(__fsub_rn(q_hi, __fsub_rn(t_hi, bb)), __fsub_rn(eps, bb)), q_lo);
    float y0;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y0) : "f"(t_hi));
    const float p_hi = __fmul_rn(y0, y0), p_lo = __fmaf_rn(y0, y0, -p_hi);
    const float u_hi = __fmul_rn(t_hi, p_hi), u_lo = __fmaf_rn(t_hi, p_hi, -u_hi);
    const float small = __fmaf_rn(t_hi, p_lo, __fmul_rn(t_lo, p_hi));
    const float e = __fsub_rn(__fsub_rn(__fsub_rn(1.0f, u_hi), u_lo), small);
    const float c = __fmul_rn(y0, __fmaf_rn(__fmul_rn(e, e), 0.375f, __fmul_rn(0.5f, e)));
    return __fadd_rn(y0, c);
}

struct BlockScratch {
    float sq_hi[kChainWarps], sq_lo[kChainWarps];
    unsigned amax_bits[2];  // absolute maximum of the normalised input as fp32 bits (non-negative: ordered like integers)
    int csum[2];            // sum of the int8 codes; both indexed by level parity, the other slot is cleared meanwhile
    int ok;          // CTA-local abort flag
    int desc_ready;  // highest layer whose descriptor is in shared memory
    // this CTA's units of each level: [u_lo, u_hi); level 0 has a second range of k units [k_lo, k_hi)
    int u_lo[4], u_hi[4], k_lo, k_hi;
};

__device__ __forceinline__ uint32_t bf16_bits_rn(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Error-free accumulation of fp32 values that are exact squares: (hi, lo) += x.
__device__ __forceinline__ void acc_pair(float& hi, float& lo, float x_hi, float x_lo) {
    const float s = __fadd_rn(hi, x_hi);
    const float bb = __fsub_rn(s, hi);
    const float err = __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(x_hi, bb));
    lo = __fadd_rn(lo, __fadd_rn(err, x_lo));
    hi = s;
}

// Which packed matrix and which of its 16-row blocks job j of this CTA's level is; unit_local / part say where its
// accumulators go in the epilogue.
struct Job {
    int mat, rb;
};
__device__ __forceinline__ int v_block_of_q_block(int q_rb, const ChainParams& p) {
    const int per_head = p.head_dim / kTileRows;
    const int head = q_rb / per_head, jb = q_rb - head * per_head;
    return (head / (p.n_q / p.n_kv)) * per_head + jb;
}
__device__ __forceinline__ int level_jobs(int level, const BlockScratch* sc) {
    const int n = sc->u_hi[level] - sc->u_lo[level];
    if (level == 0) return 2 * n + (sc->k_hi - sc->k_lo);
    return level == 2 ? 2 * n : n;
}
__device__ __forceinline__ Job level_job(int level, int j, const BlockScratch* sc, const ChainParams& p) {
    Job jb;
    if (level == 0) {
        const int nqv = sc->u_hi[0] - sc->u_lo[0];
        if (j < 2 * nqv) {
            const int unit = sc->u_lo[0] + (j >> 1);
            jb.mat = (j & 1) ? 2 : 0;
            jb.rb = (j & 1) ? v_block_of_q_block(unit, p) : unit;
        } else {
            jb.mat = 1;
            jb.rb = sc->k_lo + (j - 2 * nqv);
        }
    } else if (level == 1) {
        jb.mat = 3;
        jb.rb = sc->u_lo[1] + j;
    } else if (level == 2) {
        jb.mat = 4 + (j & 1);
        jb.rb = sc->u_lo[2] + (j >> 1);
    } else {
        jb.mat = 6;
        jb.rb = sc->u_lo[3] + j;
    }
    return jb;
}

__global__ void __launch_bounds__(kChainLaunchThreads, 1) decode_chain_kernel(const ChainParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int kmax = p.hidden > p.ffn ? p.hidden : p.ffn;
    uint8_t* wbuf = smem;                                                      // [2][buf_bytes]
    uint8_t* xq_s = wbuf + 2 * (size_t)p.buf_bytes;                            // [kmax] int8 codes, lane-interleaved
    __nv_bfloat16* h_s = reinterpret_cast<__nv_bfloat16*>(xq_s + kmax);        // [hidden] running hidden state
    int* acc_s = reinterpret_cast<int*>(h_s + p.hidden);                       // [kMaxJobs][16]
    ChainLayerDev* desc_s = reinterpret_cast<ChainLayerDev*>(acc_s + kMaxJobs * 16);  // [2]
    float* sw_s = reinterpret_cast<float*>(desc_s + 2);                        // [2][8]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sw_s + 16);                   // [2] weight buffer landed, [2] buffer read
    BlockScratch* sc = reinterpret_cast<BlockScratch*>(bars + 4);
    volatile int* abort_s = reinterpret_cast<volatile int*>(&sc->ok);  // CTA-local abort flag for the mbarrier waits

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    const int total_levels = 4 * p.n_layers;

    // ---- prologue: barriers, first descriptor, its scales, the hidden state, this CTA's shares ----
    if (tid == 0) {
        for (int b = 0; b < 4; ++b) mbar_init(smem_u32(bars + b), 1);
        sc->ok = 0;
        sc->desc_ready = 0;
        sc->amax_bits[0] = sc->amax_bits[1] = 0u;
        sc->csum[0] = sc->csum[1] = 0;
        mbar_init_fence();
        // level 0: q+v units weigh two row blocks, k units one; a unit belongs to the CTA in whose weight range it starts
        const int nq = p.hidden / kTileRows, nk = p.n_kv * p.head_dim / kTileRows;
        const long long w_total = 2LL * nq + nk;
        const int w_lo = (int)(w_total * cta / grid), w_hi = (int)(w_total * (cta + 1) / grid);
        const int q_lo_w = w_lo < 2 * nq ? w_lo : 2 * nq, q_hi_w = w_hi < 2 * nq ? w_hi : 2 * nq;
        sc->u_lo[0] = (q_lo_w + 1) / 2;
        sc->u_hi[0] = (q_hi_w + 1) / 2;
        sc->k_lo = (w_lo > 2 * nq ? w_lo : 2 * nq) - 2 * nq;
        sc->k_hi = (w_hi > 2 * nq ? w_hi : 2 * nq) - 2 * nq;
        const int n1 = p.hidden / kTileRows, n2 = p.ffn / kTileRows;
        sc->u_lo[1] = (int)((long long)n1 * cta / grid); sc->u_hi[1] = (int)((long long)n1 * (cta + 1) / grid);
        sc->u_lo[2] = (int)((long long)n2 * cta / grid); sc->u_hi[2] = (int)((long long)n2 * (cta + 1) / grid);
        sc->u_lo[3] = sc->u_lo[1]; sc->u_hi[3] = sc->u_hi[1];
    }
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(p.layers);
        uint32_t* dst = reinterpret_cast<uint32_t*>(desc_s);
        for (int i = tid; i < (int)(sizeof(ChainLayerDev) / 4); i += kChainLaunchThreads) dst[i] = src[i];
    }
    for (int i = tid; i < p.hidden; i += kChainLaunchThreads) h_s[i] = p.h[i];
    __syncthreads();
    if (tid < 7) sw_s[tid] = *desc_s[0].s_w[tid];
    __syncthreads();

    // bulk copies of this CTA's share of level L into weight buffer L & 1 (the copy warp, all lanes)
    auto issue_level = [&](int L) {
        const int layer = L >> 2, level = L & 3;
        const ChainLayerDev& dsc = desc_s[layer & 1];
        const int n_jobs = level_jobs(level, sc);
        const uint32_t rb_bytes = (uint32_t)(level_K(level, p) / kTileCols) * kTileBytes;
        const uint32_t bar = smem_u32(bars + (L & 1));
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)n_jobs * rb_bytes);
        __syncwarp();
        for (int j = lane; j < n_jobs; j += 32) {
            const Job jb = level_job(level, j, sc, p);
            bulk_load_once(smem_u32(wbuf + (size_t)(L & 1) * p.buf_bytes) + (uint32_t)j * rb_bytes,
                           dsc.packed[jb.mat] + (size_t)jb.rb * rb_bytes, rb_bytes, bar, l2_evict_first_policy());  // weights: read once
        }
    };
    bool ok = true;
    // Load index l = tid + i * 512 of a level input covers elements 16 * (l / 3) + 6 * (l % 3) + 0..5 (the last of the
    // three loads of a 16-element group covers four).  None of this depends on the level.
    int ld_part[kMaxLoads], ld_elem[kMaxLoads], ld_piece[kMaxLoads];
#pragma unroll
    for (int i = 0; i < kMaxLoads; ++i) {
        const int l = tid + i * kChainThreads, rb = l / 3;
        ld_part[i] = l - 3 * rb;
        ld_elem[i] = rb * kTileRows + 6 * ld_part[i];
        // the 16 codes of a group are one 16-byte piece of the lane-interleaved order (piece 4t+q of a block of 256
        // columns at byte 64q + 16t); this thread owns bytes 6 * part .. of it
        const int c0 = rb * kTileRows, rr = c0 & 255;
        ld_piece[i] = (c0 & ~255) + 64 * ((rr >> 4) & 3) + 16 * (rr >> 6);
    }
    // 1 / K as a pair of fp32 for the two input widths
    const float ikh_hi = __fdiv_rn(1.0f, (float)p.hidden), ikh_lo = __fdiv_rn(__fmaf_rn(-ikh_hi, (float)p.hidden, 1.0f), (float)p.hidden);
    const float ikf_hi = __fdiv_rn(1.0f, (float)p.ffn), ikf_lo = __fdiv_rn(__fmaf_rn(-ikf_hi, (float)p.ffn, 1.0f), (float)p.ffn);
    if (warp == kChainWarps) {
        // ---- copy warp: one level ahead of the arithmetic, as soon as the buffer has been read and the layer's
        //      descriptor is in shared memory ----
        for (int L = 0; L < total_levels; ++L) {
            const int layer = L >> 2;
            if (L >= 2 && !mbar_wait(smem_u32(bars + 2 + (L & 1)), (uint32_t)((L >> 1) - 1) & 1u, abort_s)) break;
            const unsigned long long t0 = globaltimer_ns();
            bool ready = true;
            while (*reinterpret_cast<volatile int*>(&sc->desc_ready) < layer) {
                if (*abort_s || globaltimer_ns() - t0 > kWaitLimitNs) { ready = false; break; }
            }
            if (!ready) { *abort_s = 1; break; }
            issue_level(L);
        }
    } else
    for (int L = 0; L < total_levels && ok; ++L) {
        const int layer = L >> 2, level = L & 3;
        const int K = level_K(level, p), k_tiles = K / kTileCols;
        const int n_jobs = level_jobs(level, sc);
        const unsigned tag = (unsigned)L & 0xffffu;  // what the producers of this level's input wrote: their level + 1

        // ---- descriptor / scale prefetch for the next layer ----
        // level 3 needs the next layer's descriptor, level 0 this layer's scales: the asynchronous copies that fetch them
        // are awaited here and become visible to everybody at the barrier that follows the counter wait
        if (level == 3 || level == 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (level == 0 && layer + 1 < p.n_layers && tid < (int)(sizeof(ChainLayerDev) / 16)) {
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(&desc_s[(layer + 1) & 1]) + 16u * tid),
                         "l"(reinterpret_cast<const uint8_t*>(p.layers + layer + 1) + 16 * tid)
                         : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }

        // ---- the gains of this level's input: loads issued before the wait so that they overlap it ----
        const __nv_bfloat16* gain = desc_s[layer & 1].gain[level];
        const int n_loads = 3 * (K / kTileRows);
        // whether load i concerns this WARP at all (warp-uniform): whole iterations are skipped where it does not
        const bool act[kMaxLoads] = {(warp << 5) < n_loads, (warp << 5) + kChainThreads < n_loads,
                                     (warp << 5) + 2 * kChainThreads < n_loads};
        uint32_t gw[kMaxLoads][3];
#pragma unroll
        for (int i = 0; i < kMaxLoads; ++i) {
            gw[i][0] = gw[i][1] = gw[i][2] = 0x3f803f80u;  // bf16 ones
            if (act[i] && gain != nullptr && tid + i * kChainThreads < n_loads) {
                const uint32_t* gp = reinterpret_cast<const uint32_t*>(gain + ld_elem[i]);
                gw[i][0] = gp[0];
                gw[i][1] = gp[1];
                if (ld_part[i] < 2) gw[i][2] = gp[2];
            }
        }

        // ---- wait until the arrival counter says that a look at the input is worthwhile (bounded) ----
        if (L > 0) {
            if (tid == 0) {
                const unsigned target = (unsigned)grid * (unsigned)L;
                const unsigned long long t0 = globaltimer_ns();
                unsigned spins = 0;
                while (ld_relaxed_u32(p.counter) < target) {
                    if ((++spins & 255u) == 0u) {
                        if (*reinterpret_cast<volatile int*>(p.abort_word) != 0) { sc->ok = 1; break; }
                        if (globaltimer_ns() - t0 > kWaitLimitNs) {
                            atomicExch(p.abort_word, 1);
                            sc->ok = 1;
                            break;
                        }
                    }
                }
            }
            CSYNC();
            if (sc->ok) { ok = false; break; }
        }
        if (level == 3 && tid == 0) {
            __threadfence_block();
            *reinterpret_cast<volatile int*>(&sc->desc_ready) = layer + 1;  // the copy warp may go on to the next layer
        }
        // the next layer's scales: their addresses are in the descriptor that the barrier above has made visible
        if (level == 3 && layer + 1 < p.n_layers && tid < 7) {
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(sw_s + 8 * ((layer + 1) & 1) + tid)),
                         "l"(desc_s[(layer + 1) & 1].s_w[tid])
                         : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (tid < kMaxJobs * 16) acc_s[tid] = 0;
        if (tid == 0) { sc->amax_bits[(L + 1) & 1] = 0u; sc->csum[(L + 1) & 1] = 0; }

        // ---- the level's input: every word checked against the level tag, stale words read again ----
        float xv[kMaxLoads][6];
        if (L == 0) {
#pragma unroll
            for (int i = 0; i < kMaxLoads; ++i) {
                const int l = tid + i * kChainThreads;
#pragma unroll
                for (int e = 0; e < 6; ++e)
                    xv[i][e] = (l < n_loads && 6 * ld_part[i] + e < kTileRows) ? __bfloat162float(h_s[ld_elem[i] + e]) : 0.0f;
            }
        } else {
            const unsigned long long* src = pub_of(p, (level + 3) & 3);
            unsigned long long wa[kMaxLoads], wb[kMaxLoads];
#pragma unroll
            for (int i = 0; i < kMaxLoads; ++i) {
                const int l = tid + i * kChainThreads;
                wa[i] = wb[i] = (unsigned long long)tag << 48;
                if (act[i] && l < n_loads) ld_pub2(src + 2 * l, wa[i], wb[i]);
            }
#pragma unroll
            for (int i = 0; i < kMaxLoads; ++i) {
                const int l = tid + i * kChainThreads;
                if (!act[i]) continue;
                if (l < n_loads && ((unsigned)(wa[i] >> 48) != tag || (unsigned)(wb[i] >> 48) != tag)) {
                    const unsigned long long t0 = globaltimer_ns();
                    unsigned spins = 0;
                    for (;;) {
                        ld_pub2(src + 2 * l, wa[i], wb[i]);
                        if ((unsigned)(wa[i] >> 48) == tag && (unsigned)(wb[i] >> 48) == tag) break;
                        if ((++spins & 15u) == 0u) {
                            if (*reinterpret_cast<volatile int*>(p.abort_word) != 0) { sc->ok = 1; break; }
                            if (globaltimer_ns() - t0 > kWaitLimitNs) {
                                atomicExch(p.abort_word, 1);
                                sc->ok = 1;
                                break;
                            }
                        }
                    }
                }
                const uint32_t a0 = (uint32_t)wa[i], a1 = (uint32_t)(wa[i] >> 32), b0 = (uint32_t)wb[i], b1 = (uint32_t)(wb[i] >> 32);
                xv[i][0] = bf16_lo(a0); xv[i][1] = bf16_hi(a0); xv[i][2] = bf16_lo(a1);
                xv[i][3] = bf16_lo(b0); xv[i][4] = bf16_hi(b0); xv[i][5] = bf16_lo(b1);
                if ((level == 0 || level == 2) && l < n_loads) {
                    // the input of levels 0 and 2 is the hidden state itself: keep it for the residual adds of this CTA's rows
                    // (ld_elem is even: two values per 32-bit store)
                    uint32_t* hp = reinterpret_cast<uint32_t*>(reinterpret_cast<uint16_t*>(h_s) + ld_elem[i]);
                    hp[0] = a0;
                    hp[1] = (a1 & 0xffffu) | (b0 << 16);
                    if (ld_part[i] < 2) hp[2] = (b0 >> 16) | (b1 << 16);
                }
            }
        }

        // ---- RMSNorm: sum of the exact squares as an error-free pair of fp32, root in fp64 by one thread ----
        float s_hi = 0.0f, s_lo = 0.0f;
#pragma unroll
        for (int i = 0; i < kMaxLoads; ++i) {
            if (!act[i]) continue;
            // one chain per load: independent of the others, so their latencies overlap
            float c_hi = __fmul_rn(xv[i][0], xv[i][0]), c_lo = 0.0f;
#pragma unroll
            for (int e = 1; e < 6; ++e) acc_pair(c_hi, c_lo, __fmul_rn(xv[i][e], xv[i][e]), 0.0f);
            if (i == 0) { s_hi = c_hi; s_lo = c_lo; }
            else acc_pair(s_hi, s_lo, c_hi, c_lo);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float o_hi = __shfl_xor_sync(0xffffffffu, s_hi, o), o_lo = __shfl_xor_sync(0xffffffffu, s_lo, o);
            acc_pair(s_hi, s_lo, o_hi, o_lo);
        }
        if (lane == 0) { sc->sq_hi[warp] = s_hi; sc->sq_lo[warp] = s_lo; }
        CSYNC();
        if (sc->ok) { if (tid == 0) atomicExch(p.abort_word, 1); ok = false; break; }  // a tag wait ran out
        // every warp adds the sixteen partial pairs in the same order and takes lane 0's result, so all agree on r
        s_hi = sc->sq_hi[lane & (kChainWarps - 1)];
        s_lo = sc->sq_lo[lane & (kChainWarps - 1)];
#pragma unroll
        for (int o = kChainWarps / 2; o > 0; o >>= 1) {
            const float o_hi = __shfl_xor_sync(0xffffffffu, s_hi, o), o_lo = __shfl_xor_sync(0xffffffffu, s_lo, o);
            acc_pair(s_hi, s_lo, o_hi, o_lo);
        }
        const float r = __shfl_sync(0xffffffffu, rms_scale_pair(s_hi, s_lo, level == 3 ? ikf_hi : ikh_hi, level == 3 ? ikf_lo : ikh_lo, p.eps), 0);
        float amax = 0.0f;
#pragma unroll
        for (int i = 0; i < kMaxLoads; ++i) {
            if (!act[i]) continue;
            const float gv[6] = {bf16_lo(gw[i][0]), bf16_hi(gw[i][0]), bf16_lo(gw[i][1]),
                                 bf16_hi(gw[i][1]), bf16_lo(gw[i][2]), bf16_hi(gw[i][2])};
#pragma unroll
            for (int e = 0; e < 6; ++e) {
                xv[i][e] = __fmul_rn(__fmul_rn(xv[i][e], r), gv[e]);  // the normalised value (0 where there is no element)
                amax = fmaxf(amax, fabsf(xv[i][e]));
            }
        }
        {
            const unsigned wmax = __reduce_max_sync(0xffffffffu, __float_as_uint(amax));
            if (lane == 0) atomicMax(&sc->amax_bits[L & 1], wmax);
        }
        CSYNC();
        const float a = fmaxf(__uint_as_float(sc->amax_bits[L & 1]), 1e-5f);
        const float sc_q = __fdiv_rn(127.0f, a), d = __fdiv_rn(a, 127.0f);
        int csum = 0;
#pragma unroll
        for (int i = 0; i < kMaxLoads; ++i) {
            if (act[i] && tid + i * kChainThreads < n_loads) {
                const int part = ld_part[i];
                uint32_t c[6];
#pragma unroll
                for (int e = 0; e < 6; ++e) c[e] = round_code(__fmul_rn(xv[i][e], sc_q));
                uint8_t* piece = xq_s + ld_piece[i];
                const uint32_t w4 = pack_codes4(c[0], c[1], c[2], c[3], csum);
                if (part == 0) {
                    *reinterpret_cast<uint32_t*>(piece) = w4;
                    const uint32_t w2 = pack_codes4(c[4], c[5], 0u, 0u, csum);
                    *reinterpret_cast<uint16_t*>(piece + 4) = (uint16_t)w2;
                } else if (part == 1) {
                    // bytes 6..11: codes 0,1 then 2..5
                    const uint32_t w2 = pack_codes4(c[4], c[5], 0u, 0u, csum);
                    *reinterpret_cast<uint16_t*>(piece + 6) = (uint16_t)w4;
                    *reinterpret_cast<uint32_t*>(piece + 8) = (w4 >> 16) | (w2 << 16);
                } else {
                    *reinterpret_cast<uint32_t*>(piece + 12) = w4;
                }
            }
        }
        csum = __reduce_add_sync(0xffffffffu, csum);
        if (lane == 0) atomicAdd(&sc->csum[L & 1], csum);

        // ---- the level's weights: wait for the prefetched share, multiply ----
        mbar_wait(smem_u32(bars + (L & 1)), (uint32_t)(L >> 1) & 1u, abort_s);
        CSYNC();  // codes, code sums and the zeroed accumulators are visible; every thread has passed the weight wait
        if (sc->ok) {  // the copy did not land in time: tell the other CTAs and leave
            if (tid == 0) atomicExch(p.abort_word, 1);
            ok = false;
            break;
        }
        const int xsum = sc->csum[L & 1];
        const uint32_t buf_s = smem_u32(wbuf + (size_t)(L & 1) * p.buf_bytes);
        const uint32_t xq_a = smem_u32(xq_s) + 16u * t;
        {
            // a warp takes a contiguous run of the CTA's 16 x 256 tiles, so it folds its accumulators once per row block
            const int n_tiles = n_jobs * k_tiles;
            const int t_lo = n_tiles * warp / kChainWarps, t_hi = n_tiles * (warp + 1) / kChainWarps;
            int acc[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
            int job = t_lo / k_tiles, kt = t_lo - job * k_tiles;
            for (int tix = t_lo; tix < t_hi; ++tix) {
                const uint4 w0v = lds128(buf_s + (uint32_t)tix * kTileBytes + 16u * lane);
                const uint4 w1v = lds128(buf_s + (uint32_t)tix * kTileBytes + 512u + 16u * lane);
                const uint32_t w0[4] = {w0v.x, w0v.y, w0v.z, w0v.w};
                const uint32_t w1[4] = {w1v.x, w1v.y, w1v.z, w1v.w};
#pragma unroll
                for (int qd = 0; qd < 4; ++qd) {
                    const uint4 xw4 = lds128(xq_a + (uint32_t)kt * kTileCols + 64u * qd);
                    const uint32_t xw[4] = {xw4.x, xw4.y, xw4.z, xw4.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t mask = 0x03030303u << (2 * j);
                        acc[0][j] = dp4a_u8_s8(w0[qd] & mask, xw[j], acc[0][j]);
                        acc[1][j] = dp4a_u8_s8(w1[qd] & mask, xw[j], acc[1][j]);
                    }
                }
                if (++kt == k_tiles || tix + 1 == t_hi) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        int sum = acc[hh][0] * 4 + acc[hh][1];  // accumulator j holds 4^j x its share: 64 x the sum
                        sum = sum * 4 + acc[hh][2];
                        sum = sum * 4 + acc[hh][3];
                        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                        if (t == 0) atomicAdd(&acc_s[job * 16 + 8 * hh + g], sum >> 6);
                        acc[hh][0] = acc[hh][1] = acc[hh][2] = acc[hh][3] = 0;
                    }
                    if (kt == k_tiles) { kt = 0; ++job; }
                }
            }
        }
        CSYNC();
        if (tid == 0) mbar_arrive(smem_u32(bars + 2 + (L & 1)));  // the buffer has been read: it may be refilled

        // ---- dequantising epilogue + the glue that follows this level, published as the next level's input ----
        // One thread per output row (a unit's 16 rows are a half warp); lanes 0..5 of each half then gather three rows each
        // into the 8-byte words of the unit.  The k rows of level 0 are stored by the second half of the CTA.
        {
            const int n_units = sc->u_hi[level] - sc->u_lo[level];
            const float* sw = sw_s + 8 * (layer & 1);
            const bool last = L + 1 == total_levels;
            if (warp < (n_units + 1) / 2) {  // warp-uniform
                const int ul = tid >> 4, row16 = tid & 15, unit = sc->u_lo[level] + ul;
                uint32_t bits = 0u;
                if (ul < n_units) {
                    const int row = unit * kTileRows + row16;
                    const int jpu = (level == 0 || level == 2) ? 2 : 1;  // jobs per unit
                    const float s0 = level == 0 ? sw[0] : (level == 1 ? sw[3] : (level == 2 ? sw[4] : sw[6]));
                    const float y0 = __fmul_rn(__fmul_rn((float)(acc_s[(ul * jpu) * 16 + row16] - xsum), s0), d);
                    float val;
                    if (level == 0) {
                        const float y1 = __fmul_rn(__fmul_rn((float)(acc_s[(ul * 2 + 1) * 16 + row16] - xsum), sw[2]), d);
                        val = __fadd_rn(y0, y1);  // attention stand-in: q + v of the matching KV head
                    } else if (level == 2) {
                        const float y1 = __fmul_rn(__fmul_rn((float)(acc_s[(ul * 2 + 1) * 16 + row16] - xsum), sw[5]), d);
                        const float rl = fmaxf(y0, 0.0f);
                        val = __fmul_rn(__fmul_rn(rl, rl), y1);  // squared-ReLU gate times up
                    } else {
                        val = __fadd_rn(__bfloat162float(h_s[row]), y0);  // residual
                    }
                    bits = bf16_bits_rn(val);
                    if (last) reinterpret_cast<uint16_t*>(p.h)[row] = (uint16_t)bits;
                }
                const int wd = lane & 15, base = lane & 16;  // word wd of this half warp's unit: rows 3 wd .. 3 wd + 2
                const int r0 = 3 * wd;
                const uint32_t b0 = __shfl_sync(0xffffffffu, bits, base + (r0 < 16 ? r0 : 15));
                const uint32_t b1 = __shfl_sync(0xffffffffu, bits, base + (r0 + 1 < 16 ? r0 + 1 : 15));
                const uint32_t b2 = __shfl_sync(0xffffffffu, bits, base + (r0 + 2 < 16 ? r0 + 2 : 15));
                if (!last && ul < n_units && wd < 6)
                    st_pub(pub_of(p, level) + 6 * (size_t)unit + wd,
                           (unsigned long long)(b0 | ((wd < 5 ? b1 : 0u) << 16)) |
                               ((unsigned long long)((wd < 5 ? b2 : 0u) | (((unsigned)(L + 1) & 0xffffu) << 16)) << 32));
            }
            if (level == 0 && tid >= kChainThreads / 2) {  // k rows: an output of the layer, consumed by nobody here
                const int nqv = sc->u_hi[0] - sc->u_lo[0], nk = sc->k_hi - sc->k_lo;
                const int o = tid - kChainThreads / 2;
                if (o < nk * 16)
                    p.k[(sc->k_lo + (o >> 4)) * kTileRows + (o & 15)] =
                        __fmul_rn(__fmul_rn((float)(acc_s[(2 * nqv + (o >> 4)) * 16 + (o & 15)] - xsum), sw[1]), d);
            }
            // arrival hint (not ordered with the stores above: the tags say when the data is there)
            if (tid == 0 && !last) asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p.counter) : "memory");
        }
    }

    __syncthreads();
    if (!ok || sc->ok) abort_drain();  // bulk copies of this CTA may still be in flight
    if (tid == 0 && cta == 0 && *reinterpret_cast<volatile int*>(p.abort_word) != 0 && p.status_word != nullptr)
        atomicExch(p.status_word, BITLINEAR_ERR_TIMEOUT);
}

struct ChainLayout {
    size_t layers_off, k_off, pub_off[4], sync_off, zero_begin, zero_bytes, total;
};

ChainLayout chain_layout(int n_layers, int hidden, int ffn, int kv) {
    ChainLayout L;
    size_t off = 0;
    L.layers_off = off;
    off = align_up(off + (size_t)n_layers * sizeof(ChainLayerDev), 256);
    L.k_off = off;
    off = align_up(off + (size_t)kv * sizeof(float), 256);
    L.zero_begin = off;  // everything from here on is cleared at every launch: tags and the sync words
    const int widths[4] = {hidden, hidden, ffn, hidden};  // a, h after attention, f, h after the feed-forward block
    for (int i = 0; i < 4; ++i) {
        L.pub_off[i] = off;
        off = align_up(off + (size_t)(widths[i] / kTileRows) * 6 * sizeof(unsigned long long), 256);
    }
    L.sync_off = off;
    off += 256;
    L.zero_bytes = off - L.zero_begin;
    L.total = off;
    return L;
}

bool chain_dims_ok(int n_layers, int hidden, int ffn, int n_q, int n_kv, int hd) {
    if (n_layers <= 0 || n_layers > 16000 || n_q <= 0 || n_kv <= 0 || hd <= 0 || n_q % n_kv) return false;
    if (hidden != n_q * hd || hd % kTileRows) return false;  // a block of 16 q rows lies inside one head
    return shape_ok(hidden, hidden) && shape_ok(ffn, hidden) && shape_ok(hidden, ffn) &&
           3 * (hidden / kTileRows) <= kMaxLoads * kChainThreads && 3 * (ffn / kTileRows) <= kMaxLoads * kChainThreads;
}

// Per-device facts, looked up once per device (a process may drive several GPUs).
struct ChainDevice {
    int sm_count = 0, coop = 0, major = 0;
    bool known = false;
};
int chain_device(ChainDevice& out) {
    static ChainDevice cache[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    ChainDevice& c = cache[dev];
    if (!c.known) {
        if (cudaDeviceGetAttribute(&c.major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c.coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        c.known = true;
    }
    out = c;
    return BITLINEAR_OK;
}

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

size_t bitlinear_decode_chain_workspace_bytes(int n_layers, int hidden, int ffn, int n_q_heads, int n_kv_heads, int head_dim) {
    if (!chain_dims_ok(n_layers, hidden, ffn, n_q_heads, n_kv_heads, head_dim)) return 0;
    return chain_layout(n_layers, hidden, ffn, n_kv_heads * head_dim).total;
}

int bitlinear_decode_chain(const bitlinear_chain_layer* layers, int n_layers, int hidden, int ffn, int n_q_heads,
                           int n_kv_heads, int head_dim, float rms_eps, void* h_bf16, float* k_out, int flags, void* ws,
                           size_t ws_bytes, void* stream) {
    if (!chain_dims_ok(n_layers, hidden, ffn, n_q_heads, n_kv_heads, head_dim)) return BITLINEAR_ERR_SHAPE;
    if (flags & ~BITLINEAR_BATCH_REUSE_PLAN) return BITLINEAR_ERR_DTYPE;
    if (!layers || !h_bf16) return BITLINEAR_ERR_NULL;
    const int kv = n_kv_heads * head_dim;
    const ChainLayout L = chain_layout(n_layers, hidden, ffn, kv);
    if (!ws || !aligned16(ws) || ws_bytes < L.total) return BITLINEAR_ERR_WORKSPACE;
    if (!aligned16(h_bf16) || (reinterpret_cast<uintptr_t>(k_out) & 3u)) return BITLINEAR_ERR_ALIGN;
    static_assert(sizeof(ChainLayerDev) == sizeof(bitlinear_chain_layer), "host and device layer descriptors differ");
    for (int l = 0; l < n_layers; ++l)
        for (int j = 0; j < 7; ++j) {
            if (!layers[l].packed[j] || !layers[l].s_w[j]) return BITLINEAR_ERR_NULL;
            if (!aligned16(layers[l].packed[j]) || (j < 4 && layers[l].gain[j] && !aligned16(layers[l].gain[j])))
                return BITLINEAR_ERR_ALIGN;
        }
    ChainDevice devinfo;
    if (const int rc = chain_device(devinfo)) return rc;
    if (devinfo.major != 10) return BITLINEAR_ERR_ARCH;
    if (!devinfo.coop) return BITLINEAR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);
    if (!(flags & BITLINEAR_BATCH_REUSE_PLAN) &&
        cudaMemcpyAsync(base + L.layers_off, layers, (size_t)n_layers * sizeof(ChainLayerDev), cudaMemcpyHostToDevice, st) !=
            cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (cudaMemsetAsync(base + L.zero_begin, 0, L.zero_bytes, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    ChainParams prm;
    prm.layers = reinterpret_cast<const ChainLayerDev*>(base + L.layers_off);
    prm.n_layers = n_layers; prm.hidden = hidden; prm.ffn = ffn; prm.n_q = n_q_heads; prm.n_kv = n_kv_heads;
    prm.head_dim = head_dim; prm.eps = rms_eps;
    prm.h = static_cast<__nv_bfloat16*>(h_bf16);
    prm.k = reinterpret_cast<float*>(base + L.k_off);
    for (int i = 0; i < 4; ++i) prm.pub[i] = reinterpret_cast<unsigned long long*>(base + L.pub_off[i]);
    prm.counter = reinterpret_cast<unsigned*>(base + L.sync_off);
    prm.abort_word = reinterpret_cast<int*>(base + L.sync_off + 64);
    prm.status_word = device_status_word();
    // the largest per-CTA share of a level, in row blocks of packed weights: level 0 splits 2 * hidden/16 + kv/16
    // weight units and a q+v unit (two row blocks) is not divided; level 2 pairs a gate block with an up block
    const int grid = devinfo.sm_count;
    auto ceil_div = [](long long a, long long b) { return (a + b - 1) / b; };
    const size_t rb_h = (size_t)(hidden / kTileCols) * kTileBytes, rb_f = (size_t)(ffn / kTileCols) * kTileBytes;
    const long long jobs0 = ceil_div(2LL * (hidden / kTileRows) + kv / kTileRows, grid) + 2;
    const long long jobs1 = ceil_div(hidden / kTileRows, grid);
    const long long jobs2 = 2 * ceil_div(ffn / kTileRows, grid);
    if (jobs0 > kMaxJobs || jobs1 > kMaxJobs || jobs2 > kMaxJobs) return BITLINEAR_ERR_SHAPE;
    size_t buf = std::max({(size_t)jobs0 * rb_h, (size_t)jobs1 * rb_h, (size_t)jobs2 * rb_h, (size_t)jobs1 * rb_f});
    prm.buf_bytes = (int)buf;
    const int kmax = hidden > ffn ? hidden : ffn;
    const size_t smem = 2 * buf + kmax + (size_t)hidden * 2 + kMaxJobs * 64 + 2 * sizeof(ChainLayerDev) + 64 + 32 +
                        sizeof(BlockScratch) + 1024;
    if (smem > 227 * 1024) return BITLINEAR_ERR_SHAPE;
    if (cudaFuncSetAttribute(decode_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    void* args[] = {&prm};
    if (cudaLaunchCooperativeKernel(reinterpret_cast<void*>(decode_chain_kernel), dim3(grid), dim3(kChainLaunchThreads), args, smem,
                                    st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (k_out && cudaMemcpyAsync(k_out, prm.k, (size_t)kv * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

}  // extern "C"
