// Chained decode of a stack of decoder layers at one token, in ONE persistent cooperative kernel.
// (Paper Section 2: every linear map of a layer is a BitLinear - q, k, v, o, gate, up, down - with squared ReLU in the
// feed-forward block; Section 5.1: decode cost is the packed weight bytes.  Attention is not a BitLinear and is
// replaced by a fixed stand-in, see bitlinear_glue_attn_standin.)
//
// A layer is four dependent levels: {q,k,v}(h), o(a), {gate,up}(h), down(f).  A level's matrices are stacked and their
// 16-row blocks split evenly over the CTAs (one per SM).  Per level every CTA
//   1. waits for the level's share of packed weights, which it prefetched into shared memory with bulk copies while
//      the previous level ran (weight addresses do not depend on activations),
//   2. waits at a grid barrier for the previous level's outputs, then rebuilds the level's input vector itself
//      (residual / stand-in / squared-ReLU glue, RMSNorm, absmax int8 quantiser - a few thousand elements, cheaper to
//      redo per CTA than to exchange),
//   3. multiplies its row blocks (dot-product-of-four on word & (0x03030303 << 2j), as in the streaming decode kernel),
//      applies the dequantising epilogue and stores its slice of the level's output.
// So a token costs 4 x n_layers grid barriers instead of 12 x n_layers kernel launches.
// Every wait is bounded; on a timeout an abort word makes every CTA leave and BITLINEAR_ERR_TIMEOUT is reported.
#include <algorithm>

#include "quant_row.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

constexpr int kChainThreads = 512;  // compute threads; one more warp issues the weight copies
constexpr int kChainWarps = kChainThreads / 32;
constexpr int kChainLaunchThreads = kChainThreads + 32;
// barrier of the compute threads only (the copy warp runs on its own)
#define CSYNC() asm volatile("bar.sync 1, 512;" ::: "memory")
constexpr int kMaxEpt = 16;  // input elements per thread: K <= 8192

struct ChainLayerDev {
    const uint8_t* packed[7];    // q k v o gate up down
    const float* s_w[7];
    const __nv_bfloat16* gain[4];  // inputs of {q,k,v}, o, {gate,up}, down (nullptr = ones)
};

struct ChainParams {
    const ChainLayerDev* layers;
    int n_layers, hidden, ffn, n_q, n_kv, head_dim;
    float eps;
    __nv_bfloat16* h;                 // [hidden] in / out
    float *q, *k, *v, *o, *g, *u, *dn;  // level outputs (fp32)
    unsigned* barrier;                // grid barrier counter, zero at launch
    int* abort_word;                  // zero at launch
    int* status_word;
    int buf_bytes;                    // one weight buffer (the largest per-CTA share of a level)
};

// matrices of a level: indices into the layer's 7, and their row counts
struct LevelShape {
    int n_mats, first, K;
    int rows[3];
};

__device__ __forceinline__ LevelShape level_shape(int level, const ChainParams& p) {
    LevelShape s;
    const int kv = p.n_kv * p.head_dim;
    if (level == 0) { s.n_mats = 3; s.first = 0; s.K = p.hidden; s.rows[0] = p.hidden; s.rows[1] = kv; s.rows[2] = kv; }
    else if (level == 1) { s.n_mats = 1; s.first = 3; s.K = p.hidden; s.rows[0] = p.hidden; s.rows[1] = s.rows[2] = 0; }
    else if (level == 2) { s.n_mats = 2; s.first = 4; s.K = p.hidden; s.rows[0] = p.ffn; s.rows[1] = p.ffn; s.rows[2] = 0; }
    else { s.n_mats = 1; s.first = 6; s.K = p.ffn; s.rows[0] = p.hidden; s.rows[1] = s.rows[2] = 0; }
    return s;
}

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
// bypass L1: written by other CTAs
__device__ __forceinline__ float ldcg_f32(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ldcg_f32x4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

struct BlockScratch {
    double sq[kChainWarps];
    float mx[kChainWarps];
    int sum[kChainWarps];
    float r, d;
    int xsum;
    int ok;
    int desc_ready;  // highest layer whose descriptor is in shared memory
    int rb_lo[4], rb_hi[4];  // this CTA's share of the row blocks of each of the four levels of a layer
};

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Same rounding as the stand-alone quantisers (see round_code in quant_row.cuh): low byte = int8 code.
__device__ __forceinline__ uint32_t chain_round_code(float v) { return __float_as_uint(__fadd_rn(v, 12582912.0f)); }

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void __launch_bounds__(kChainLaunchThreads, 1) decode_chain_kernel(const ChainParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int kmax = p.hidden > p.ffn ? p.hidden : p.ffn;
    const int max_rb = p.buf_bytes / ((p.hidden / kTileCols) * kTileBytes);  // most row blocks a CTA can own in a level
    uint8_t* wbuf = smem;                                                      // [2][buf_bytes]
    uint8_t* xq_s = wbuf + 2 * (size_t)p.buf_bytes;                            // [kmax] int8 codes, lane-interleaved
    __nv_bfloat16* h_s = reinterpret_cast<__nv_bfloat16*>(xq_s + kmax);        // [hidden] running hidden state
    int* acc_s = reinterpret_cast<int*>(h_s + p.hidden);                       // [max_rb][16]
    ChainLayerDev* desc_s = reinterpret_cast<ChainLayerDev*>(acc_s + (size_t)max_rb * 16);  // [2]
    float* sw_s = reinterpret_cast<float*>(desc_s + 2);                        // [2][8]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sw_s + 16);                   // [2] weight buffer landed, [2] buffer read
    BlockScratch* sc = reinterpret_cast<BlockScratch*>(bars + 4);
    volatile int* abort_s = reinterpret_cast<volatile int*>(&sc->ok);  // CTA-local abort flag for the mbarrier waits

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    const int total_levels = 4 * p.n_layers;
    const int group = p.n_q / p.n_kv;

    // ---- prologue: barriers, first descriptor, its scales, the hidden state ----
    if (tid == 0) {
        for (int b = 0; b < 4; ++b) mbar_init(smem_u32(bars + b), 1);
        sc->ok = 0;
        sc->desc_ready = 0;
        mbar_init_fence();
    }
    if (tid < 4) {  // the shares do not change from layer to layer: two 64-bit divisions per level, once
        const LevelShape s = level_shape(tid, p);
        const int total_rb = (s.rows[0] + s.rows[1] + s.rows[2]) / kTileRows;
        sc->rb_lo[tid] = (int)((long long)total_rb * cta / grid);
        sc->rb_hi[tid] = (int)((long long)total_rb * (cta + 1) / grid);
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

    // bulk copies of this CTA's share of level L into weight buffer L & 1 (warp 0, all lanes)
    auto issue_level = [&](int L) {
        const int layer = L >> 2, level = L & 3;
        const LevelShape s = level_shape(level, p);
        const ChainLayerDev& dsc = desc_s[layer & 1];
        const int total_rb = (s.rows[0] + s.rows[1] + s.rows[2]) / kTileRows;
        const int lo = sc->rb_lo[level], hi = sc->rb_hi[level];
        const uint32_t rb_bytes = (uint32_t)(s.K / kTileCols) * kTileBytes;
        const uint32_t bar = smem_u32(bars + (L & 1));
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(hi - lo) * rb_bytes);
        __syncwarp();
        for (int i = lane; i < hi - lo; i += 32) {
            int row = (lo + i) * kTileRows, m = 0;
            if (row >= s.rows[0]) {  // which of the level's stacked matrices (no indexed array: it would live in local memory)
                row -= s.rows[0];
                m = 1;
                if (row >= s.rows[1]) { row -= s.rows[1]; m = 2; }
            }
            bulk_load(smem_u32(wbuf + (size_t)(L & 1) * p.buf_bytes) + (uint32_t)i * rb_bytes,
                      dsc.packed[s.first + m] + (size_t)(row / kTileRows) * rb_bytes, rb_bytes, bar);
        }
    };
    bool ok = true;
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
        const LevelShape s = level_shape(level, p);
        const int K = s.K, k_tiles = K / kTileCols;
        const int total_rb = (s.rows[0] + s.rows[1] + s.rows[2]) / kTileRows;
        const int rb_lo = sc->rb_lo[level], rb_hi = sc->rb_hi[level];
        const int n_rb = rb_hi - rb_lo;

        // ---- descriptor / scale prefetch for the next layer, weight prefetch for the next level ----
        if (level == 3 || level == 0) {  // level 3 needs the next layer's descriptor, level 0 this layer's scales
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            CSYNC();
            if (level == 3 && tid == 0) {
                __threadfence_block();
                *reinterpret_cast<volatile int*>(&sc->desc_ready) = layer + 1;  // the copy warp may go on to the next layer
            }
        }
        if (level == 0 && layer + 1 < p.n_layers && tid < (int)(sizeof(ChainLayerDev) / 16)) {
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(&desc_s[(layer + 1) & 1]) + 16u * tid),
                         "l"(reinterpret_cast<const uint8_t*>(p.layers + layer + 1) + 16 * tid)
                         : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (level == 3 && layer + 1 < p.n_layers && tid < 7) {
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(sw_s + 8 * ((layer + 1) & 1) + tid)),
                         "l"(desc_s[(layer + 1) & 1].s_w[tid])
                         : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }

        // ---- wait for the outputs of the previous level (grid barrier, bounded) ----
        if (L > 0) {
            if (tid == 0) {
                const unsigned target = (unsigned)grid * (unsigned)L;
                const unsigned long long t0 = globaltimer_ns();
                unsigned spins = 0;
                while (ld_acquire_u32(p.barrier) < target) {
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

        // ---- build this level's input vector (glue), RMSNorm, absmax int8 quantiser ----
        for (int i = tid; i < n_rb * 16; i += kChainThreads) acc_s[i] = 0;
        const __nv_bfloat16* gain = desc_s[layer & 1].gain[level];
        float xv[kMaxEpt], gv[kMaxEpt];
        // Element e of this thread is column 4 * (tid + (e / 4) * kChainThreads) + e % 4: four consecutive columns per
        // 16-byte load.  Every load of the stage is issued before anything is computed, so the L2 round trips overlap.
        float ra[kMaxEpt], rb[kMaxEpt];
#pragma unroll
        for (int q4 = 0; q4 < kMaxEpt / 4; ++q4) {
            const int i0 = 4 * (tid + q4 * kChainThreads);
            const bool in = i0 < K;  // K is a multiple of 4: a group of four is inside or outside as a whole
            float4 va = make_float4(0.0f, 0.0f, 0.0f, 0.0f), vb = va;
            if (in) {
                if (level == 0) {
                    if (layer > 0) va = ldcg_f32x4(p.dn + i0);
                } else if (level == 1) {
                    const int head = i0 / p.head_dim, j = i0 - head * p.head_dim;  // head_dim is a multiple of 4
                    va = ldcg_f32x4(p.q + i0);
                    vb = ldcg_f32x4(p.v + (head / group) * p.head_dim + j);
                } else if (level == 2) {
                    va = ldcg_f32x4(p.o + i0);
                } else {
                    va = ldcg_f32x4(p.g + i0);
                    vb = ldcg_f32x4(p.u + i0);
                }
            }
            ra[4 * q4] = va.x; ra[4 * q4 + 1] = va.y; ra[4 * q4 + 2] = va.z; ra[4 * q4 + 3] = va.w;
            rb[4 * q4] = vb.x; rb[4 * q4 + 1] = vb.y; rb[4 * q4 + 2] = vb.z; rb[4 * q4 + 3] = vb.w;
            if (gain != nullptr && in) {
                const uint2 gw = *reinterpret_cast<const uint2*>(gain + i0);
                gv[4 * q4] = __uint_as_float(gw.x << 16);
                gv[4 * q4 + 1] = __uint_as_float(gw.x & 0xffff0000u);
                gv[4 * q4 + 2] = __uint_as_float(gw.y << 16);
                gv[4 * q4 + 3] = __uint_as_float(gw.y & 0xffff0000u);
            } else {
                gv[4 * q4] = gv[4 * q4 + 1] = gv[4 * q4 + 2] = gv[4 * q4 + 3] = 1.0f;
            }
        }
        double sq = 0.0;
#pragma unroll
        for (int e = 0; e < kMaxEpt; ++e) {
            const int i = 4 * (tid + (e >> 2) * kChainThreads) + (e & 3);
            float x = 0.0f;
            if (i < K) {
                if (level == 0) {
                    x = __bfloat162float(h_s[i]);
                    if (layer > 0) {
                        x = bf16_round(__fadd_rn(x, ra[e]));
                        h_s[i] = __float2bfloat16_rn(x);
                    }
                } else if (level == 1) {
                    x = bf16_round(__fadd_rn(ra[e], rb[e]));
                } else if (level == 2) {
                    x = bf16_round(__fadd_rn(__bfloat162float(h_s[i]), ra[e]));
                    h_s[i] = __float2bfloat16_rn(x);
                } else {
                    const float r = fmaxf(ra[e], 0.0f);
                    x = bf16_round(__fmul_rn(__fmul_rn(r, r), rb[e]));
                }
            }
            xv[e] = x;
        }
        {   // sum of squares: error-free fp32 chains of eight, then fp64 (see sum_squares8)
            float lo8[8], hi8[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) { lo8[e] = xv[e]; hi8[e] = xv[8 + e]; }
            sq = sum_squares8(lo8);
            if (K > 8 * kChainThreads) sq += sum_squares8(hi8);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (lane == 0) sc->sq[warp] = sq;
        CSYNC();
        if (tid == 0) {
            double S = 0.0;
#pragma unroll
            for (int w = 0; w < kChainWarps; ++w) S += sc->sq[w];
            sc->r = (float)(1.0 / sqrt(S / (double)K + (double)p.eps));
        }
        CSYNC();
        const float r = sc->r;
        float amax = 0.0f;
#pragma unroll
        for (int e = 0; e < kMaxEpt; ++e) {
            xv[e] = __fmul_rn(__fmul_rn(xv[e], r), gv[e]);  // the normalised value
            amax = fmaxf(amax, fabsf(xv[e]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if (lane == 0) sc->mx[warp] = amax;
        CSYNC();
        float a = 1e-5f;
#pragma unroll
        for (int w = 0; w < kChainWarps; ++w) a = fmaxf(a, sc->mx[w]);
        const float sc_q = __fdiv_rn(127.0f, a), d = __fdiv_rn(a, 127.0f);
        int csum = 0;
#pragma unroll
        for (int q4 = 0; q4 < kMaxEpt / 4; ++q4) {
            const int i0 = 4 * (tid + q4 * kChainThreads);
            if (i0 < K) {
                const uint32_t word = pack_codes4(chain_round_code(__fmul_rn(xv[4 * q4], sc_q)), chain_round_code(__fmul_rn(xv[4 * q4 + 1], sc_q)),
                                                  chain_round_code(__fmul_rn(xv[4 * q4 + 2], sc_q)), chain_round_code(__fmul_rn(xv[4 * q4 + 3], sc_q)), csum);
                // lane-interleaved order inside each block of 256 columns: piece 4t+q -> byte 64q + 16t; four consecutive
                // columns stay together inside their 16-byte piece
                const int blk = i0 & ~255, rr = i0 & 255;
                *reinterpret_cast<uint32_t*>(xq_s + blk + 64 * ((rr >> 4) & 3) + 16 * (rr >> 6) + (rr & 15)) = word;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
        if (lane == 0) sc->sum[warp] = csum;
        CSYNC();
        int xsum = 0;
#pragma unroll
        for (int w = 0; w < kChainWarps; ++w) xsum += sc->sum[w];

        // ---- the level's weights: wait for the prefetched share, multiply ----
        mbar_wait(smem_u32(bars + (L & 1)), (uint32_t)(L >> 1) & 1u, abort_s);
        CSYNC();
        if (sc->ok) {  // the copy did not land in time: tell the other CTAs and leave
            if (tid == 0) atomicExch(p.abort_word, 1);
            ok = false;
            break;
        }
        const uint32_t buf_s = smem_u32(wbuf + (size_t)(L & 1) * p.buf_bytes);
        const uint32_t xq_a = smem_u32(xq_s) + 16u * t;
        for (int tix = warp; tix < n_rb * k_tiles; tix += kChainWarps) {
            const int rbl = tix / k_tiles, kt = tix - rbl * k_tiles;
            const uint4 w0v = lds128(buf_s + (uint32_t)tix * kTileBytes + 16u * lane);
            const uint4 w1v = lds128(buf_s + (uint32_t)tix * kTileBytes + 512u + 16u * lane);
            const uint32_t w0[4] = {w0v.x, w0v.y, w0v.z, w0v.w};
            const uint32_t w1[4] = {w1v.x, w1v.y, w1v.z, w1v.w};
            int acc[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
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
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                int sum = acc[hh][0] * 4 + acc[hh][1];  // accumulator j holds 4^j x its share: 64 x the sum
                sum = sum * 4 + acc[hh][2];
                sum = sum * 4 + acc[hh][3];
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                if (t == 0) atomicAdd(&acc_s[rbl * 16 + 8 * hh + g], sum >> 6);
            }
        }
        CSYNC();
        if (tid == 0) mbar_arrive(smem_u32(bars + 2 + (L & 1)));  // the buffer has been read: it may be refilled

        // ---- dequantising epilogue: this CTA's rows of the level's output ----
        for (int o = tid; o < n_rb * 16; o += kChainThreads) {
            int row = (rb_lo + (o >> 4)) * kTileRows + (o & 15), m = 0;
            if (row >= s.rows[0]) {  // which of the level's stacked matrices (no indexed array: it would live in local memory)
                row -= s.rows[0];
                m = 1;
                if (row >= s.rows[1]) { row -= s.rows[1]; m = 2; }
            }
            float* y;
            if (level == 0) y = m == 0 ? p.q : (m == 1 ? p.k : p.v);
            else if (level == 1) y = p.o;
            else if (level == 2) y = m == 0 ? p.g : p.u;
            else y = p.dn;
            const float s_w = sw_s[8 * (layer & 1) + s.first + m];
            y[row] = __fmul_rn(__fmul_rn((float)(acc_s[o] - xsum), s_w), d);
        }
        CSYNC();
        // release at GPU scope: the stores of every thread of the CTA (ordered before this by the barrier above) are
        // visible to whoever acquires the new count
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
    }

    // ---- after the last level: the final residual, written by CTA 0 ----
    if (warp < kChainWarps && ok && cta == 0) {
        if (tid == 0) {
            const unsigned target = (unsigned)grid * (unsigned)total_levels;
            const unsigned long long t0 = globaltimer_ns();
            unsigned spins = 0;
            while (ld_acquire_u32(p.barrier) < target) {
                if ((++spins & 255u) == 0u && (globaltimer_ns() - t0 > kWaitLimitNs || *reinterpret_cast<volatile int*>(p.abort_word))) {
                    atomicExch(p.abort_word, 1);
                    sc->ok = 1;
                    break;
                }
            }
        }
        CSYNC();
        if (!sc->ok)
            for (int i = tid; i < p.hidden; i += kChainThreads)
                p.h[i] = __float2bfloat16_rn(__fadd_rn(__bfloat162float(h_s[i]), ldcg_f32(p.dn + i)));
    }
    __syncthreads();
    if (!ok || sc->ok) abort_drain();  // bulk copies of this CTA may still be in flight
    if (tid == 0 && cta == 0 && *reinterpret_cast<volatile int*>(p.abort_word) != 0 && p.status_word != nullptr)
        atomicExch(p.status_word, BITLINEAR_ERR_TIMEOUT);
}

struct ChainLayout {
    size_t layers_off, out_off[7], sync_off, total;
};

ChainLayout chain_layout(int n_layers, int hidden, int ffn, int kv) {
    ChainLayout L;
    size_t off = 0;
    L.layers_off = off;
    off = align_up(off + (size_t)n_layers * sizeof(ChainLayerDev), 256);
    const int widths[7] = {hidden, kv, kv, hidden, ffn, ffn, hidden};  // q k v o g u dn
    for (int i = 0; i < 7; ++i) {
        L.out_off[i] = off;
        off = align_up(off + (size_t)widths[i] * sizeof(float), 256);
    }
    L.sync_off = off;
    off += 256;
    L.total = off;
    return L;
}

bool chain_dims_ok(int n_layers, int hidden, int ffn, int n_q, int n_kv, int hd) {
    if (n_layers <= 0 || n_q <= 0 || n_kv <= 0 || hd <= 0 || n_q % n_kv) return false;
    if (hidden != n_q * hd || (n_kv * hd) % kTileRows || hd % 4) return false;  // 16-byte loads never straddle a head
    return shape_ok(hidden, hidden) && shape_ok(ffn, hidden) && shape_ok(hidden, ffn) && hidden <= kMaxEpt * kChainThreads &&
           ffn <= kMaxEpt * kChainThreads;
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
    static int sm_count = 0, coop = 0;
    if (sm_count == 0) {
        int dev = 0, major = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            sm_count = 0;
            return BITLINEAR_ERR_CUDA;
        }
        if (major != 10) { sm_count = 0; return BITLINEAR_ERR_ARCH; }
    }
    if (!coop) return BITLINEAR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);
    if (!(flags & BITLINEAR_BATCH_REUSE_PLAN) &&
        cudaMemcpyAsync(base + L.layers_off, layers, (size_t)n_layers * sizeof(ChainLayerDev), cudaMemcpyHostToDevice, st) !=
            cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (cudaMemsetAsync(base + L.sync_off, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    ChainParams prm;
    prm.layers = reinterpret_cast<const ChainLayerDev*>(base + L.layers_off);
    prm.n_layers = n_layers; prm.hidden = hidden; prm.ffn = ffn; prm.n_q = n_q_heads; prm.n_kv = n_kv_heads;
    prm.head_dim = head_dim; prm.eps = rms_eps;
    prm.h = static_cast<__nv_bfloat16*>(h_bf16);
    float* outs[7];
    for (int i = 0; i < 7; ++i) outs[i] = reinterpret_cast<float*>(base + L.out_off[i]);
    prm.q = outs[0]; prm.k = outs[1]; prm.v = outs[2]; prm.o = outs[3]; prm.g = outs[4]; prm.u = outs[5]; prm.dn = outs[6];
    prm.barrier = reinterpret_cast<unsigned*>(base + L.sync_off);
    prm.abort_word = reinterpret_cast<int*>(base + L.sync_off + 64);
    prm.status_word = device_status_word();
    // the largest per-CTA share of a level, in bytes of packed weights
    const int grid = sm_count;
    auto share = [&](int rows, int K) { return (size_t)((rows / kTileRows + grid - 1) / grid) * (K / kTileCols) * kTileBytes; };
    size_t buf = share(hidden + 2 * kv, hidden);
    buf = std::max(buf, share(hidden, hidden));
    buf = std::max(buf, share(2 * ffn, hidden));
    buf = std::max(buf, share(hidden, ffn));
    prm.buf_bytes = (int)buf;
    const int kmax = hidden > ffn ? hidden : ffn;
    const size_t max_rb = buf / ((size_t)(hidden / kTileCols) * kTileBytes);
    const size_t smem = 2 * buf + kmax + (size_t)hidden * 2 + max_rb * 64 + 2 * sizeof(ChainLayerDev) + 64 + 32 +
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
