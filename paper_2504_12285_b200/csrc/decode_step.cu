// The rest of a decode step around the BitLinear layers (paper Section 2: rotary position embeddings; a Transformer
// decoder, i.e. causal attention - with grouped queries in the 2B configuration; a vocabulary of 128,256 tokens, hence
// a bf16 embedding table and an output head of that many rows, which is larger than all packed BitLinear weights
// together).  None of these is a BitLinear; they are here so that a whole decoded token can be timed.
//
//   rope_kv_kernel            : rotates q and k (pairs i, i + head_dim/2; angle = position * base^(-2i/head_dim), formed
//                               in fp64 because positions reach the thousands), writes q as bf16 and appends k, v to
//                               the bf16 cache of the token's sequence.
//   attn_decode_partial_kernel: one CTA per (token, KV head, slice of the cache); 64-row tiles of keys and values arrive
//                               by tensor-map copies issued by a producer warp, the query heads of the group are the
//                               8-column side of a tensor-core operand (mma.sync, bf16 inputs, fp32 accumulation),
//                               softmax in fp32; partial (max, sum, weighted values) per slice.
//   attn_decode_combine_kernel: merges the slices of a (token, query head) and writes bf16.
//   lm_head_mma_kernel        : logits = x . E^T for up to 16 tokens on the tensor cores (tokens = rows of the A operand),
//                               the table streamed once with 128-bit loads (HBM-bound: 657 MB for 128,256 x 2560).
//   embed_kernel              : row gather.
// All of them but the output head and the gather are launched as programmatic dependents of the launch in front of
// them and read nothing before griddepcontrol.wait.
#include "common.cuh"
#include "sm100_sync.cuh"
#include "tensor_map.cuh"

#include <algorithm>
#include <mutex>
#include <type_traits>

namespace bitlinear {

namespace {

__device__ __forceinline__ float bf16_lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---------------------------------------------------------------------------------------------- RoPE + cache append

// (cos, sin) of position * base^(-2i / head_dim), formed in fp64 and rounded once: the one place the angle is computed,
// so the table built from it and the kernel that rotates without a table give the same bits
__device__ __forceinline__ float2 rope_cos_sin(int pos, int i, int hd, double log2_base) {
    const double angle = (double)pos * exp2(-2.0 * (double)i / (double)hd * log2_base);
    double sd, cd;
    sincos(angle, &sd, &cd);
    return make_float2((float)cd, (float)sd);
}

// table[pos][i] = (cos, sin) for every cache position and rotation pair
__global__ void __launch_bounds__(256) rope_table_kernel(float2* __restrict__ table, int t_max, int hd, double log2_base) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int half = hd / 2;
    if (idx >= (long long)t_max * half) return;
    table[idx] = rope_cos_sin((int)(idx / half), (int)(idx % half), hd, log2_base);
}

__global__ void __launch_bounds__(256) rope_kv_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                                      const float* __restrict__ v, const int* __restrict__ positions,
                                                      const int* __restrict__ seq_ids, int M, int n_q, int n_kv, int hd, int n_seq,
                                                      double log2_base, __nv_bfloat16* __restrict__ q_out,
                                                      __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                                                      int t_max) {
    // a programmatic dependent of the launch before it (the q/k/v projections) and the primary of the attention launch
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int half = hd / 2;
    const int pairs_per_tok = (n_q + n_kv) * half;
    const int vals_per_tok = n_kv * hd;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n_rot = (long long)M * pairs_per_tok;
    if (idx < n_rot) {
        const int m = (int)(idx / pairs_per_tok), r = (int)(idx - (long long)m * pairs_per_tok);
        const int head = r / half, i = r - head * half;
        const int pos = positions[m];
        const float2 cs = rope_cos_sin(pos, i, hd, log2_base);
        const float c = cs.x, s = cs.y;
        const bool is_q = head < n_q;
        const float* src = is_q ? q + (size_t)m * n_q * hd + (size_t)head * hd : k + (size_t)m * n_kv * hd + (size_t)(head - n_q) * hd;
        const float lo = src[i], hi = src[i + half];
        const float o_lo = __fsub_rn(__fmul_rn(lo, c), __fmul_rn(hi, s));
        const float o_hi = __fadd_rn(__fmul_rn(hi, c), __fmul_rn(lo, s));
        const int seq = seq_ids ? seq_ids[m] : 0;
        if (!is_q && (pos < 0 || pos >= t_max || seq < 0 || seq >= n_seq)) return;  // a row outside the cache is not stored
        __nv_bfloat16* dst;
        if (is_q) dst = q_out + (size_t)m * n_q * hd + (size_t)head * hd;
        else dst = k_cache + (((size_t)seq * n_kv + (size_t)(head - n_q)) * t_max + pos) * hd;
        dst[i] = __float2bfloat16_rn(o_lo);
        dst[i + half] = __float2bfloat16_rn(o_hi);
    } else if (idx < n_rot + (long long)M * vals_per_tok) {
        const long long j = idx - n_rot;
        const int m = (int)(j / vals_per_tok), e = (int)(j - (long long)m * vals_per_tok);
        const int seq = seq_ids ? seq_ids[m] : 0;
        if (positions[m] < 0 || positions[m] >= t_max || seq < 0 || seq >= n_seq) return;
        v_cache[(((size_t)seq * n_kv + (size_t)(e / hd)) * t_max + positions[m]) * hd + (e % hd)] =
            __float2bfloat16_rn(v[(size_t)m * vals_per_tok + e]);
    }
}

// ---------------------------------------------------------------------------------------------- decode attention

constexpr int kAttnKeys = 64;       // cache rows per tile
constexpr int kAttnMaxStages = 3;   // tiles in flight per CTA (1 when every slice is a single tile)
constexpr int kAttnMaxSplits = 64;  // partial results per (token, query head)

// partial result of one slice of the cache for one (token, query head): weighted values, running maximum, sum of weights
template <int HD>
struct __align__(16) AttnPartial {
    float o[HD];
    float m, l, pad[2];
};

template <int HD>
constexpr size_t attn_smem_bytes(int stages) {
    return 1024 /*alignment slack*/ + (size_t)stages * 2 * kAttnKeys * HD * 2 + 16 * kAttnMaxStages + 8;
}

// How the 64-row tiles of a token's live cache rows are dealt to the slices: `per` tiles each, `live` slices in use.
struct AttnSlices {
    int per, live;
};
__host__ __device__ inline AttnSlices attn_slices(int len, int splits) {
    const int tiles = (len + kAttnKeys - 1) / kAttnKeys;
    const int per = tiles > 0 ? (tiles + splits - 1) / splits : 1;
    return {per, (tiles + per - 1) / per};
}

// (cache rows are read once per call: marked evict-first in L2, so that a context longer than L2 does not push out what
// is read again - the partial results, the projections)
__device__ __forceinline__ void tma_tile_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
// four 8 x 8 matrices of 16-bit elements, row addresses from lanes 8i .. 8i+7 for matrix i
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// d += a * b, 16 x 8 x 16, bf16 operands, fp32 accumulation
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transpose of an 8 x 8 matrix of 16-bit elements held one row pair per lane (the layout ldmatrix delivers)
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Cache rows token m attends to.  Plain calls clamp the given length to the cache; a call that appends the token's own
// row (row length - 1) takes a length outside 1 .. t_max as "no token" (nothing stored, a zero result).
__device__ __forceinline__ int attn_len(const int* __restrict__ lengths, int seq, int m, int n_seq, int t_max, bool own_row) {
    if (seq < 0 || seq >= n_seq) return 0;
    const int raw = lengths[m];
    if (own_row) return (raw >= 1 && raw <= t_max) ? raw : 0;
    return min(max(raw, 0), t_max);
}

// One CTA per (slice of the cache, KV head, token): four consumer warps and one producer warp.  A slice is a run of
// 64-row tiles; each tile's key and value rows of this KV head (64 x HD bf16 each) arrive in shared memory by
// tensor-map copies of 64 rows x 128 bytes (128-byte swizzle; a head's rows are contiguous in the cache, so a tile is
// 64 * HD * 2 contiguous bytes of HBM) issued by the producer into a ring of `stages` tiles
// (full / empty barriers per stage), so every query head of the group reads the cache from HBM once.
// Consumer warp w takes keys 16w .. 16w+15 of every tile and works on the transposed problem, which wastes the least
// of the 16 x 8 x 16 tensor-core shape on a group of at most 8 heads:
//   S^T (16 keys x 8 heads) = K (16 x HD) Q^T   - K fragments by ldmatrix, Q^T from registers; bf16 products are exact,
//                                                 accumulation in fp32;
//   a running softmax per head in fp32 (the keys of a head sit in one accumulator column);
//   O^T (HD x 8 heads) += V^T (HD x 16 keys) P  - V^T fragments by ldmatrix.trans; P is the exponentiated S^T,
//                                                 split into two bf16 parts (P = P_hi + P_lo, relative error 2^-17)
//                                                 so that the bf16 operand costs no accuracy, and transposed into
//                                                 the B-operand layout by movmatrix.
// The four warps' results are merged in shared memory at the end.  Slices past the token's length return at once and
// are not read by the combine kernel.  Rows of a tile past the token's length are copied (they are inside the cache,
// or zero-filled past its end); their scores are discarded by a select and their value rows are overwritten with zeros
// before use, so whatever bits they hold never enter a result.
//
// With OWN (the token's own row is part of the call) the kernel also does the work of the rotary-embedding launch: q, k
// and v arrive as fp32 projections; every consumer warp rotates the group's query heads itself (cos, sin from a
// table, the same fp32 operations in the same order as rope_kv_kernel, hence the same bits); the one warp whose keys
// include row length - 1 rotates k, rounds k and v to bf16, stores them to the cache in global memory and, once the
// tile has landed, over the row's stale copy in shared memory.  No other CTA reads that row: it lies in one slice of
// one (token, KV head), and the tokens of such a call belong to different sequences.
struct AttnOwnRow {
    const float* q;        // [M][n_q * HD]   fp32, not rotated
    const float* k;        // [M][n_kv * HD]
    const float* v;        // [M][n_kv * HD]
    const float2* table;   // [t_max][HD / 2] (cos, sin)
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
};

template <int HD, bool OWN>
__global__ void __launch_bounds__(160) attn_decode_partial_kernel(const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_v,
                                                                  const __nv_bfloat16* __restrict__ q, const AttnOwnRow own,
                                                                  const int* __restrict__ lengths,
                                                                  const int* __restrict__ seq_ids, int n_q, int n_kv, int n_seq, int t_max,
                                                                  int splits, int stages, float scale,
                                                                  AttnPartial<HD>* __restrict__ part, int* __restrict__ status_word) {
    constexpr int HALVES = HD / 64;                   // 128-byte column blocks of a row
    constexpr uint32_t kHalfBytes = kAttnKeys * 128;  // one block of a tile: 64 rows x 128 bytes
    constexpr uint32_t kTileBytes = HALVES * kHalfBytes;
    constexpr int KS = HD / 16;    // k-steps of K Q^T, and 16-row tiles of O^T
    constexpr int OPAD = HD + 4;   // row stride of the merge buffer (floats)
    extern __shared__ uint8_t attn_smem_raw[];
    const int split = blockIdx.x, kvh = blockIdx.y, m = blockIdx.z;
    const int group = n_q / n_kv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, qd = lane & 3;  // fragment coordinates of this lane
    uint8_t* smem = attn_smem_raw + ((1024u - (smem_u32(attn_smem_raw) & 1023u)) & 1023u);
    const uint32_t ring_s = smem_u32(smem);  // [stage][K, V][block][64 rows][128 bytes, swizzled]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)stages * 2 * kTileBytes);  // full[3], empty[3]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kAttnMaxStages);
    const uint32_t full_s = smem_u32(bars), empty_s = full_s + 8u * kAttnMaxStages;
    // what needs no global data comes first: this launch is a programmatic dependent and may begin while the launch
    // before it (rotary embedding + cache append, or whatever wrote the lengths) is still running
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
        *abort_flag = 0;
        for (int st = 0; st < stages; ++st) {
            mbar_init(full_s + 8u * st, 1);
            mbar_init(empty_s + 8u * st, 4);  // one arrival per consumer warp
        }
        mbar_init_fence();
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");  // nothing is read from global memory before this
    const int seq = seq_ids ? seq_ids[m] : 0;
    const int len = attn_len(lengths, seq, m, n_seq, t_max, OWN);
    const AttnSlices sl = attn_slices(len, splits);
    if (split >= sl.live) return;  // the whole CTA: nothing of this slice is live
    const int tile0 = split * sl.per;
    const int n_tiles = min(sl.per, (len + kAttnKeys - 1) / kAttnKeys - tile0);
    // the merge kernel may be scheduled now; it waits for this whole grid before it reads a partial result
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();  // barriers initialised, abort flag cleared

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};  // heads 2qd, 2qd+1 over this warp's keys
    float o[KS][4];  // O^T: rows 16mt + g (+8), columns heads 2qd, 2qd+1
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.0f;

    if (warp == 4) {
        // ---- producer: one lane feeds the ring
        if (lane == 0) {
            const int row0 = (seq * n_kv + kvh) * t_max + tile0 * kAttnKeys;  // this head's rows are contiguous
            const uint64_t once = l2_evict_first_policy();
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t st = (uint32_t)(i % stages), dst = ring_s + st * 2u * kTileBytes, bar = full_s + 8u * st;
                if (i >= stages && !mbar_wait(empty_s + 8u * st, (uint32_t)(i / stages - 1) & 1u, abort_flag)) break;
                mbar_expect_tx(bar, 2u * kTileBytes);
#pragma unroll
                for (int hf = 0; hf < HALVES; ++hf) {
                    tma_tile_2d(dst + hf * kHalfBytes, &map_k, hf * 64, row0 + i * kAttnKeys, bar, once);
                    tma_tile_2d(dst + kTileBytes + hf * kHalfBytes, &map_v, hf * 64, row0 + i * kAttnKeys, bar, once);
                }
            }
        }
    } else {
        // ---- consumers
        // Q^T as the B operand: column g = head kvh * group + g (zero columns past the group), two registers per k-step
        uint32_t qb[KS][2];
        const int kb = warp * 16;  // this warp's keys of a tile
        // OWN: the token's own row is row `pos`, in tile `own_tile` of this slice if this CTA has it at all, and among
        // this warp's keys if own_warp; its new key and value, as bf16 pairs, for dims 2 lane (+ HD / 2) and 4 lane ...
        const int pos = len - 1;
        const int own_tile = OWN ? pos / kAttnKeys - tile0 : -1;
        const bool own_warp = OWN && own_tile >= 0 && own_tile < n_tiles && (pos % kAttnKeys) / 16 == warp;
        const bool k_lane = 2 * lane < HD / 2, v_lane = 4 * lane < HD;
        uint32_t k_lo = 0u, k_hi = 0u, v_a = 0u, v_b = 0u;
        if constexpr (!OWN) {
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)m * n_q + (size_t)kvh * group + min(g, group - 1)) * HD);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qb[ks][0] = g < group ? qrow[8 * ks + qd] : 0u;
                qb[ks][1] = g < group ? qrow[8 * ks + 4 + qd] : 0u;
            }
        } else {
            // the rotation pairs dim i with dim i + HD / 2: k-step ks with k-step ks + KS / 2, same place in the fragment
            const float* qrow = own.q + ((size_t)m * n_q + (size_t)kvh * group + min(g, group - 1)) * HD;
            const float2* trow = own.table + (size_t)pos * (HD / 2);
#pragma unroll
            for (int ks = 0; ks < KS / 2; ++ks) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int i = 16 * ks + 8 * h + 2 * qd;
                    const float2 lo = *reinterpret_cast<const float2*>(qrow + i), hi = *reinterpret_cast<const float2*>(qrow + i + HD / 2);
                    const float4 cs = *reinterpret_cast<const float4*>(trow + i);  // cos, sin of pair i; cos, sin of pair i + 1
                    const float lo0 = __fsub_rn(__fmul_rn(lo.x, cs.x), __fmul_rn(hi.x, cs.y));
                    const float hi0 = __fadd_rn(__fmul_rn(hi.x, cs.x), __fmul_rn(lo.x, cs.y));
                    const float lo1 = __fsub_rn(__fmul_rn(lo.y, cs.z), __fmul_rn(hi.y, cs.w));
                    const float hi1 = __fadd_rn(__fmul_rn(hi.y, cs.z), __fmul_rn(lo.y, cs.w));
                    qb[ks][h] = g < group ? pack_bf16(lo0, lo1) : 0u;
                    qb[ks + KS / 2][h] = g < group ? pack_bf16(hi0, hi1) : 0u;
                }
            }
            if (own_warp) {
                const size_t src = ((size_t)m * n_kv + kvh) * HD, dst = (((size_t)seq * n_kv + kvh) * t_max + pos) * HD;
                if (k_lane) {
                    const int i = 2 * lane;
                    const float2 lo = *reinterpret_cast<const float2*>(own.k + src + i);
                    const float2 hi = *reinterpret_cast<const float2*>(own.k + src + i + HD / 2);
                    const float4 cs = *reinterpret_cast<const float4*>(trow + i);
                    k_lo = pack_bf16(__fsub_rn(__fmul_rn(lo.x, cs.x), __fmul_rn(hi.x, cs.y)),
                                     __fsub_rn(__fmul_rn(lo.y, cs.z), __fmul_rn(hi.y, cs.w)));
                    k_hi = pack_bf16(__fadd_rn(__fmul_rn(hi.x, cs.x), __fmul_rn(lo.x, cs.y)),
                                     __fadd_rn(__fmul_rn(hi.y, cs.z), __fmul_rn(lo.y, cs.w)));
                    *reinterpret_cast<uint32_t*>(own.k_cache + dst + i) = k_lo;
                    *reinterpret_cast<uint32_t*>(own.k_cache + dst + i + HD / 2) = k_hi;
                }
                if (v_lane) {
                    const float4 t = *reinterpret_cast<const float4*>(own.v + src + 4 * lane);
                    v_a = pack_bf16(t.x, t.y);
                    v_b = pack_bf16(t.z, t.w);
                    *reinterpret_cast<uint2*>(own.v_cache + dst + 4 * lane) = make_uint2(v_a, v_b);
                }
            }
        }
        const int mi = lane >> 3, mr = lane & 7;  // the matrix and row this lane addresses for ldmatrix
        for (int i = 0; i < n_tiles; ++i) {
            const uint32_t st = (uint32_t)(i % stages);
            if (!mbar_wait(full_s + 8u * st, (uint32_t)(i / stages) & 1u, abort_flag)) break;
            const int n = min(kAttnKeys, len - (tile0 + i) * kAttnKeys);  // live rows of the tile, >= 1
            if (kb < n) {
                const uint32_t kbase = ring_s + st * 2u * kTileBytes, vbase = kbase + kTileBytes;
                if (OWN && own_warp && i == own_tile) {
                    // the copy of the tile was read from the cache before (or while) the row was stored: put the new
                    // row over it.  Element d of row r sits in block d / 64 at byte 128 r + 16 ((d % 64) / 8 ^ r % 8) + 2 (d % 8).
                    const uint32_t r = (uint32_t)(pos % kAttnKeys);
                    auto at = [&](uint32_t base, int d) {
                        return base + (uint32_t)(d >> 6) * kHalfBytes + r * 128u + (((((uint32_t)d & 63u) >> 3) ^ (r & 7u)) << 4) + ((uint32_t)d & 7u) * 2u;
                    };
                    if (k_lane) {
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(at(kbase, 2 * lane)), "r"(k_lo) : "memory");
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(at(kbase, 2 * lane + HD / 2)), "r"(k_hi) : "memory");
                    }
                    if (v_lane) asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(at(vbase, 4 * lane)), "r"(v_a), "r"(v_b) : "memory");
                    __syncwarp();
                }
                if (n < kb + 16) {  // the ragged end: zero this warp's dead value rows
                    for (int idx = lane; idx < (kb + 16 - n) * HALVES * 8; idx += 32) {
                        const int row = n + idx / (HALVES * 8), c = idx % (HALVES * 8);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vbase + (c >> 3) * kHalfBytes + row * 128 + (c & 7) * 16),
                                     "r"(0u)
                                     : "memory");
                    }
                    __syncwarp();
                }
                // this lane's row of the four 8 x 8 blocks a ldmatrix.x4 fetches: keys kb + 8 (mi & 1) + mr, 16-byte chunk
                // (mi >> 1) of the pair of chunks in turn - the same addressing for K (plain) and V (transposed)
                const uint32_t row_off = (uint32_t)(kb + 8 * (mi & 1) + mr) * 128u;
                // S^T = K Q^T, two accumulators to halve the dependent chain
                float s0[4] = {0.0f, 0.0f, 0.0f, 0.0f}, s1[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int chunk = ((2 * ks) & 7) + (mi >> 1);
                    uint32_t a[4];  // a0: keys 0-7, dims 0-7 of the step; a1: keys 8-15; a2, a3: dims 8-15
                    ldsm_x4(kbase + (ks >> 2) * kHalfBytes + row_off + ((chunk ^ mr) << 4), a);
                    if (ks & 1) mma_bf16(s1, a, qb[ks][0], qb[ks][1]);
                    else mma_bf16(s0, a, qb[ks][0], qb[ks][1]);
                }
                // s[0], s[1]: key kb + g, heads 2qd, 2qd+1;  s[2], s[3]: key kb + g + 8
                const bool live_lo = kb + g < n, live_hi = kb + g + 8 < n;
                float sv[4];
                sv[0] = live_lo ? (s0[0] + s1[0]) * scale : -INFINITY;  // a dead row may hold anything: selected away
                sv[1] = live_lo ? (s0[1] + s1[1]) * scale : -INFINITY;
                sv[2] = live_hi ? (s0[2] + s1[2]) * scale : -INFINITY;
                sv[3] = live_hi ? (s0[3] + s1[3]) * scale : -INFINITY;
                float mt0 = fmaxf(sv[0], sv[2]), mt1 = fmaxf(sv[1], sv[3]);
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    mt0 = fmaxf(mt0, __shfl_xor_sync(0xffffffffu, mt0, off));
                    mt1 = fmaxf(mt1, __shfl_xor_sync(0xffffffffu, mt1, off));
                }
                const float mn0 = fmaxf(m_run[0], mt0), mn1 = fmaxf(m_run[1], mt1);  // finite: key kb is live
                const float corr0 = expf(m_run[0] - mn0), corr1 = expf(m_run[1] - mn1);  // expf(-inf) = 0 the first time
                float pv[4];
                pv[0] = expf(sv[0] - mn0);  // 0 for a dead key
                pv[1] = expf(sv[1] - mn1);
                pv[2] = expf(sv[2] - mn0);
                pv[3] = expf(sv[3] - mn1);
                float lt0 = pv[0] + pv[2], lt1 = pv[1] + pv[3];
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    lt0 += __shfl_xor_sync(0xffffffffu, lt0, off);
                    lt1 += __shfl_xor_sync(0xffffffffu, lt1, off);
                }
                l_run[0] = fmaf(l_run[0], corr0, lt0);
                l_run[1] = fmaf(l_run[1], corr1, lt1);
                m_run[0] = mn0;
                m_run[1] = mn1;
                // P (keys x heads) as the B operand: the accumulator holds it one row pair per lane, the operand wants
                // it one column pair per lane - an 8 x 8 transpose per block of eight keys
                float ph[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) ph[e] = __bfloat162float(__float2bfloat16_rn(pv[e]));
                const uint32_t b0h = movmatrix_t(pack_bf16(ph[0], ph[1])), b1h = movmatrix_t(pack_bf16(ph[2], ph[3]));
                const uint32_t b0l = movmatrix_t(pack_bf16(pv[0] - ph[0], pv[1] - ph[1]));
                const uint32_t b1l = movmatrix_t(pack_bf16(pv[2] - ph[2], pv[3] - ph[3]));
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    o[mt][0] *= corr0;
                    o[mt][1] *= corr1;
                    o[mt][2] *= corr0;
                    o[mt][3] *= corr1;
                }
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {  // dims 16mt .. 16mt+15
                    const int chunk = ((2 * mt) & 7) + (mi >> 1);
                    uint32_t a[4];  // transposed on load: a0: dims 0-7 x keys 0-7; a1: dims 0-7 x keys 8-15; a2, a3: dims 8-15
                    ldsm_x4_t(vbase + (mt >> 2) * kHalfBytes + row_off + ((chunk ^ mr) << 4), a);
                    // the operand order is (dims 0-7, keys 0-7), (dims 8-15, keys 0-7), (dims 0-7, keys 8-15), (dims 8-15, keys 8-15)
                    const uint32_t av[4] = {a[0], a[2], a[1], a[3]};
                    mma_bf16(o[mt], av, b0h, b1h);
                    mma_bf16(o[mt], av, b0l, b1l);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_s + 8u * st);  // this warp is done with the stage
        }
    }
    __syncthreads();  // every copy that was issued has landed and been consumed - or the CTA is giving up
    if (*abort_flag) {
        if (threadIdx.x == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
        abort_drain();
        return;
    }
    // merge the four consumer warps (the ring is free)
    float* om = reinterpret_cast<float*>(smem);  // [warp][head][OPAD]
    float* mm = om + 4 * 8 * OPAD;               // [warp][head]
    float* ll = mm + 32;
    if (warp < 4) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int head = 2 * qd + e;
            if (head < group) {
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    om[(warp * 8 + head) * OPAD + 16 * mt + g] = o[mt][e];
                    om[(warp * 8 + head) * OPAD + 16 * mt + g + 8] = o[mt][2 + e];
                }
                if (g == 0) {
                    mm[warp * 8 + head] = m_run[e];
                    ll[warp * 8 + head] = l_run[e];
                }
            }
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < group * HD; idx += blockDim.x) {
        const int row = idx / HD, d = idx - row * HD;
        float m_all = mm[row];
#pragma unroll
        for (int w = 1; w < 4; ++w) m_all = fmaxf(m_all, mm[w * 8 + row]);  // finite: warp 0 always has a live key
        float l = 0.0f, acc = 0.0f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float f = expf(mm[w * 8 + row] - m_all);  // 0 for a warp that saw no key
            l = fmaf(ll[w * 8 + row], f, l);
            acc = fmaf(om[(w * 8 + row) * OPAD + d], f, acc);
        }
        AttnPartial<HD>& dst = part[((size_t)m * n_q + (size_t)kvh * group + row) * splits + split];
        dst.o[d] = acc;
        if (d == 0) { dst.m = m_all; dst.l = l; }
    }
}

// Merges the live slices (at most 64) of a (token, query head) and writes bf16; a token of length 0 gets zeros.  Four
// warps deal the slices among themselves, every load of a warp independent of the others, and meet in shared memory.
template <int HD>
__global__ void __launch_bounds__(128) attn_decode_combine_kernel(const AttnPartial<HD>* __restrict__ part, const int* __restrict__ lengths,
                                                                  const int* __restrict__ seq_ids, int n_q, int n_seq, int t_max, int splits,
                                                                  int own_row, __nv_bfloat16* __restrict__ out) {
    constexpr int CPL = HD / 32;
    __shared__ float red[4][HD];
    const size_t mh = blockIdx.x;  // token * n_q + head
    const int m = (int)(mh / n_q);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the o projection may start fetching its weights
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the partial results come from the launch before this one
    const AttnPartial<HD>* p = part + mh * splits;
    // every load of the kernel is issued before the first result is needed, the token's length included: sixteen
    // slots per warp and the maxima and sums of all slots, live or not (a slot that no slice wrote holds whatever the
    // workspace held; it is discarded by a select, never multiplied)
    float v[kAttnMaxSplits / 4][CPL];
#pragma unroll
    for (int i = 0; i < kAttnMaxSplits / 4; ++i) {
        const float* po = p[min(warp + 4 * i, splits - 1)].o + lane * CPL;
        if constexpr (CPL == 4) {
            const float4 t = *reinterpret_cast<const float4*>(po);
            v[i][0] = t.x, v[i][1] = t.y, v[i][2] = t.z, v[i][3] = t.w;
        } else {
            const float2 t = *reinterpret_cast<const float2*>(po);
            v[i][0] = t.x, v[i][1] = t.y;
        }
    }
    const float2 ml0 = *reinterpret_cast<const float2*>(&p[min(lane, splits - 1)].m);
    const float2 ml1 = *reinterpret_cast<const float2*>(&p[min(lane + 32, splits - 1)].m);
    const int len = attn_len(lengths, seq_ids ? seq_ids[m] : 0, m, n_seq, t_max, own_row != 0);
    const int live = attn_slices(len, splits).live;  // <= splits <= 64
    if (live == 0) {  // block-uniform
        for (int d = threadIdx.x; d < HD; d += blockDim.x) out[mh * HD + d] = __float2bfloat16_rn(0.0f);
        return;
    }
    const float m0 = lane < live ? ml0.x : -INFINITY, m1 = lane + 32 < live ? ml1.x : -INFINITY;
    const float l0 = lane < live ? ml0.y : 0.0f, l1 = lane + 32 < live ? ml1.y : 0.0f;
    float m_all = fmaxf(m0, m1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, off));
    const float f0 = lane < live ? expf(m0 - m_all) : 0.0f, f1 = lane + 32 < live ? expf(m1 - m_all) : 0.0f;
    float l = fmaf(l0, f0, l1 * f1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    float acc[CPL];
#pragma unroll
    for (int e = 0; e < CPL; ++e) acc[e] = 0.0f;
#pragma unroll
    for (int i = 0; i < kAttnMaxSplits / 4; ++i) {
        const int s = warp + 4 * i;  // warp-uniform
        const float f = __shfl_sync(0xffffffffu, s < 32 ? f0 : f1, s & 31);
#pragma unroll
        for (int e = 0; e < CPL; ++e) acc[e] = s < live ? fmaf(v[i][e], f, acc[e]) : acc[e];
    }
#pragma unroll
    for (int e = 0; e < CPL; ++e) red[warp][lane * CPL + e] = acc[e];
    __syncthreads();
    for (int d = threadIdx.x; d < HD; d += blockDim.x) {
        const float o = (red[0][d] + red[1][d]) + (red[2][d] + red[3][d]);
        out[mh * HD + d] = __float2bfloat16_rn(l > 0.0f ? o / l : 0.0f);
    }
}

// ---------------------------------------------------------------------------------------------- output head, embedding

// The output head for 1 .. 16 tokens on the tensor cores: the tokens are the 16 rows of the A operand (zero rows past M),
// eight vocabulary rows are the columns of B.  A lane loads 16 bytes (eight consecutive k) of its vocabulary row straight
// from global memory and uses them as the B registers of two mma.sync steps; since a dot product does not care about
// the order of k, the k-slots of a step are simply those eight values of the four lanes that share a column, and the
// A operand (x, staged in shared memory) is read with the same assignment.  The table is streamed once.
__global__ void __launch_bounds__(512) lm_head_mma_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ table,
                                                          int M, int V, int K, int x_stride, float* __restrict__ logits) {
    extern __shared__ __align__(16) uint8_t xs_raw[];  // [16][x_stride bytes]: rows 64 bytes apart modulo 128
    const int n_vec = K / 8, pad_vec = (K + 31) / 32 * 4;  // 16-byte chunks of a row, and up to the next 32 columns
    for (int i = threadIdx.x; i < 16 * pad_vec; i += blockDim.x) {
        const int m = i / pad_vec, c = i - m * pad_vec;
        *reinterpret_cast<uint4*>(xs_raw + (size_t)m * x_stride + c * 16) =
            (m < M && c < n_vec) ? reinterpret_cast<const uint4*>(x)[(size_t)m * n_vec + c] : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, sq = lane & 3;
    const int warps = gridDim.x * (blockDim.x >> 5);
    const uint8_t* xa = xs_raw + (size_t)g * x_stride + sq * 16;
    const uint8_t* xb = xa + (size_t)8 * x_stride;
    const int k_blocks = K / 32;  // whole 32-k blocks; K % 32 is handled by the tail below
    // a warp takes sixteen vocabulary rows per pass - two B operands for every A fragment it reads from shared memory, which
    // halves the shared-memory traffic per table byte (with sixteen tokens that traffic is what bounds the kernel)
    for (int v0 = 16 * (blockIdx.x * (blockDim.x >> 5) + warp); v0 < V; v0 += 16 * warps) {
        const uint4* row0 = reinterpret_cast<const uint4*>(table + (size_t)min(v0 + g, V - 1) * K) + sq;
        const uint4* row1 = reinterpret_cast<const uint4*>(table + (size_t)min(v0 + 8 + g, V - 1) * K) + sq;
        float c[2][4] = {{0.0f, 0.0f, 0.0f, 0.0f}, {0.0f, 0.0f, 0.0f, 0.0f}};
        auto mma2 = [&](float (&d)[4], const uint4& a, const uint4& a8, const uint4& bq) {
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                         : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                         : "r"(a.x), "r"(a8.x), "r"(a.y), "r"(a8.y), "r"(bq.x), "r"(bq.y));
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                         : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                         : "r"(a.z), "r"(a8.z), "r"(a.w), "r"(a8.w), "r"(bq.z), "r"(bq.w));
        };
        auto step = [&](const uint4& b0, const uint4& b1, int kb) {
            const uint4 a = *reinterpret_cast<const uint4*>(xa + kb * 64);
            const uint4 a8 = *reinterpret_cast<const uint4*>(xb + kb * 64);
            mma2(c[0], a, a8, b0);
            mma2(c[1], a, a8, b1);
        };
        int kb = 0;
        for (; kb + 4 <= k_blocks; kb += 4) {  // eight loads in flight per lane
            uint4 b0[4], b1[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                b0[u] = __ldcs(row0 + (kb + u) * 4);
                b1[u] = __ldcs(row1 + (kb + u) * 4);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) step(b0[u], b1[u], kb + u);
        }
        for (; kb < k_blocks; ++kb) step(__ldcs(row0 + kb * 4), __ldcs(row1 + kb * 4), kb);
        if (K % 32) {  // 8, 16 or 24 columns left: the lanes whose chunk lies past the end contribute zeros
            const bool in = sq * 8 < K % 32;
            step(in ? __ldcs(row0 + kb * 4) : make_uint4(0, 0, 0, 0), in ? __ldcs(row1 + kb * 4) : make_uint4(0, 0, 0, 0), kb);
        }  // (the staged x row is zero-padded up to the next 32 columns)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int v = v0 + 8 * h + 2 * sq;
            if (g < M) {
                if (v < V) logits[(size_t)g * V + v] = c[h][0];
                if (v + 1 < V) logits[(size_t)g * V + v + 1] = c[h][1];
            }
            if (g + 8 < M) {
                if (v < V) logits[(size_t)(g + 8) * V + v] = c[h][2];
                if (v + 1 < V) logits[(size_t)(g + 8) * V + v + 1] = c[h][3];
            }
        }
    }
}

__global__ void __launch_bounds__(256) embed_kernel(const int* __restrict__ ids, const __nv_bfloat16* __restrict__ table, int M,
                                                    int V, int K, __nv_bfloat16* __restrict__ out) {
    const int n_vec = K / 8;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)M * n_vec) return;
    const int m = (int)(i / n_vec), c = (int)(i - (long long)m * n_vec);
    int id = ids[m];
    id = id < 0 ? 0 : (id >= V ? V - 1 : id);  // out-of-range ids are clamped, never followed out of the table
    reinterpret_cast<uint4*>(out)[i] = reinterpret_cast<const uint4*>(table)[(size_t)id * n_vec + c];
}

// partial results reserved per (token, query head): one per tile of the cache, 64 at most
int attn_splits_max(int t_max) { return std::min(kAttnMaxSplits, (t_max + kAttnKeys - 1) / kAttnKeys); }

// Launch shape: slices per (token, KV head) and tiles in flight per CTA.  When one CTA per tile fits on the GPU at once
// (a ring of one tile, six CTAs per SM) every tile gets its own CTA.  Otherwise CTAs carry a two-tile ring (three per
// SM) and the slice count is the one that fills whole waves of resident CTAs best.
struct AttnPlan {
    int splits, stages;
};
AttnPlan attn_plan(int M, int n_kv, int t_max, int sm_count) {
    const long long pairs = (long long)M * n_kv;
    const int tiles = (t_max + kAttnKeys - 1) / kAttnKeys, cap = std::min(kAttnMaxSplits, tiles);
    if (tiles <= kAttnMaxSplits && pairs * tiles <= 6ll * sm_count) return {tiles, 1};
    // the fewest waves of resident CTAs that are at least 85 % full (long slices: a CTA's start-up and its merge are paid
    // once per slice), else the fullest
    const long long slots = 3ll * sm_count;
    int best = 1;
    double best_util = 0.0;
    for (int w = 1; w <= 4; ++w) {
        const int s = (int)std::min<long long>(cap, w * slots / pairs);
        if (s < 1) continue;
        const long long ctas = pairs * s, waves = (ctas + slots - 1) / slots;
        const double util = (double)ctas / (double)(waves * slots);
        if (util > best_util + 1e-9) best = s, best_util = util;
        if (util >= 0.85) break;
    }
    return {best, std::min(2, (tiles + best - 1) / best)};
}

// rows = the cache rows of every (sequence, KV head), columns = hd; box = 64 rows x 64 columns (128 bytes), 128-byte swizzle
bool make_cache_map(CUtensorMap* map, const void* cache, int n_seq, int t_max, int n_kv, int hd) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)hd, (cuuint64_t)n_seq * n_kv * t_max};
    const cuuint64_t strides[1] = {(cuuint64_t)hd * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kAttnKeys};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(cache), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// the attention kernels need more than the default dynamic shared memory: opted in once per device
template <int HD>
bool attn_opt_in() {
    static std::mutex mu;
    static bool done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return false;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!done[dev]) {
        if (cudaFuncSetAttribute(attn_decode_partial_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)attn_smem_bytes<HD>(kAttnMaxStages)) != cudaSuccess ||
            cudaFuncSetAttribute(attn_decode_partial_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)attn_smem_bytes<HD>(kAttnMaxStages)) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        done[dev] = true;
    }
    return true;
}

bool attn_dims_ok(int M, int n_q, int n_kv, int hd, int t_max) {
    return M >= 0 && M <= 65535 && n_q > 0 && n_kv > 0 && n_q % n_kv == 0 && n_q / n_kv <= 8 && (hd == 64 || hd == 128) && t_max > 0 && t_max <= (1 << 22);
}

// the two launches of decode attention (slices, merge); arguments already checked for shape and null
int attn_launch(const __nv_bfloat16* q_bf16, const AttnOwnRow& own, bool own_row, const void* k_cache, const void* v_cache,
                const int32_t* lengths, const int32_t* seq_ids, int M, int n_q_heads, int n_kv_heads, int head_dim, int n_seq, int t_max,
                void* out_bf16, void* ws, size_t ws_bytes, void* stream) {
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out_bf16)) return BITLINEAR_ERR_ALIGN;
    if (!ws || !aligned16(ws) ||
        ws_bytes < (size_t)M * n_q_heads * attn_splits_max(t_max) * (sizeof(float) * (4 + head_dim)))
        return BITLINEAR_ERR_WORKSPACE;
    int sm_count = 0;
    if (const int rc = device_sm_count(&sm_count)) return rc;
    CUtensorMap map_k, map_v;
    if (!make_cache_map(&map_k, k_cache, n_seq, t_max, n_kv_heads, head_dim) ||
        !make_cache_map(&map_v, v_cache, n_seq, t_max, n_kv_heads, head_dim))
        return BITLINEAR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const AttnPlan plan = attn_plan(M, n_kv_heads, t_max, sm_count);
    const float scale = 1.0f / sqrtf((float)head_dim);
    int* status = device_status_word();
    // both kernels are programmatic dependents of the launch before them: they may be scheduled while it drains, and
    // call griddepcontrol.wait before reading anything
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    auto launch = [&](auto hd_tag, auto own_tag) {
        constexpr int HD = decltype(hd_tag)::value;
        constexpr bool OWN = decltype(own_tag)::value;
        if (!attn_opt_in<HD>()) return (int)BITLINEAR_ERR_CUDA;
        auto* part = static_cast<AttnPartial<HD>*>(ws);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)plan.splits, (unsigned)n_kv_heads, (unsigned)M);
        cfg.blockDim = dim3(160);
        cfg.dynamicSmemBytes = attn_smem_bytes<HD>(plan.stages);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, attn_decode_partial_kernel<HD, OWN>, map_k, map_v, q_bf16, own, lengths, seq_ids, n_q_heads,
                               n_kv_heads, n_seq, t_max, plan.splits, plan.stages, scale, part, status) != cudaSuccess) {
            cudaGetLastError();
            return (int)BITLINEAR_ERR_CUDA;
        }
        cfg.gridDim = dim3((unsigned)(M * n_q_heads));
        cfg.blockDim = dim3(128);
        cfg.dynamicSmemBytes = 0;
        if (cudaLaunchKernelEx(&cfg, attn_decode_combine_kernel<HD>, (const AttnPartial<HD>*)part, lengths, seq_ids, n_q_heads, n_seq,
                               t_max, plan.splits, (int)OWN, static_cast<__nv_bfloat16*>(out_bf16)) != cudaSuccess) {
            cudaGetLastError();
            return (int)BITLINEAR_ERR_CUDA;
        }
        return (int)BITLINEAR_OK;
    };
    using T = std::true_type;
    using F = std::false_type;
    if (head_dim == 128) return own_row ? launch(std::integral_constant<int, 128>{}, T{}) : launch(std::integral_constant<int, 128>{}, F{});
    return own_row ? launch(std::integral_constant<int, 64>{}, T{}) : launch(std::integral_constant<int, 64>{}, F{});
}

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

int bitlinear_rope_kv(const float* q, const float* k, const float* v, const int32_t* positions, const int32_t* seq_ids, int M,
                      int n_q_heads, int n_kv_heads, int head_dim, float rope_base, void* q_out_bf16, void* k_cache_bf16,
                      void* v_cache_bf16, int n_seq, int t_max, void* stream) {
    if (M < 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || head_dim % 8 || n_seq <= 0 || t_max <= 0 || !(rope_base > 1.0f))
        return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q || !k || !v || !positions || !q_out_bf16 || !k_cache_bf16 || !v_cache_bf16) return BITLINEAR_ERR_NULL;
    const long long work = (long long)M * ((n_q_heads + n_kv_heads) * (head_dim / 2) + n_kv_heads * head_dim);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((work + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, rope_kv_kernel, q, k, v, positions, seq_ids, M, n_q_heads, n_kv_heads, head_dim, n_seq,
                           log2((double)rope_base), static_cast<__nv_bfloat16*>(q_out_bf16), static_cast<__nv_bfloat16*>(k_cache_bf16),
                           static_cast<__nv_bfloat16*>(v_cache_bf16), t_max) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

size_t bitlinear_attention_workspace_bytes(int M, int n_q_heads, int n_kv_heads, int head_dim, int t_max) {
    if (!attn_dims_ok(M, n_q_heads, n_kv_heads, head_dim, t_max)) return 0;
    return (size_t)(M > 0 ? M : 1) * n_q_heads * attn_splits_max(t_max) * (sizeof(float) * (4 + head_dim));
}

int bitlinear_attention_decode(const void* q_bf16, const void* k_cache_bf16, const void* v_cache_bf16, const int32_t* lengths,
                               const int32_t* seq_ids, int M, int n_q_heads, int n_kv_heads, int head_dim, int n_seq, int t_max,
                               void* out_bf16, void* ws, size_t ws_bytes, void* stream) {
    if (!attn_dims_ok(M, n_q_heads, n_kv_heads, head_dim, t_max) || n_seq <= 0 || (long long)n_seq * n_kv_heads * t_max > (1ll << 30))
        return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q_bf16 || !k_cache_bf16 || !v_cache_bf16 || !lengths || !out_bf16) return BITLINEAR_ERR_NULL;
    if (!aligned16(q_bf16)) return BITLINEAR_ERR_ALIGN;
    return attn_launch(static_cast<const __nv_bfloat16*>(q_bf16), AttnOwnRow{}, false, k_cache_bf16, v_cache_bf16, lengths, seq_ids, M,
                       n_q_heads, n_kv_heads, head_dim, n_seq, t_max, out_bf16, ws, ws_bytes, stream);
}

int bitlinear_rope_table(float rope_base, int head_dim, int t_max, float* table_out, void* stream) {
    if ((head_dim != 64 && head_dim != 128) || t_max <= 0 || t_max > (1 << 22) || !(rope_base > 1.0f)) return BITLINEAR_ERR_SHAPE;
    if (!table_out) return BITLINEAR_ERR_NULL;
    if (!aligned16(table_out)) return BITLINEAR_ERR_ALIGN;
    const long long work = (long long)t_max * (head_dim / 2);
    rope_table_kernel<<<(unsigned)((work + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<float2*>(table_out), t_max, head_dim, log2((double)rope_base));
    if (cudaGetLastError() != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return BITLINEAR_OK;
}

int bitlinear_attention_decode_append(const float* q, const float* k, const float* v, const float* rope_table, void* k_cache_bf16,
                                      void* v_cache_bf16, const int32_t* lengths, const int32_t* seq_ids, int M, int n_q_heads,
                                      int n_kv_heads, int head_dim, int n_seq, int t_max, void* out_bf16, void* ws, size_t ws_bytes,
                                      void* stream) {
    if (!attn_dims_ok(M, n_q_heads, n_kv_heads, head_dim, t_max) || n_seq <= 0 || (long long)n_seq * n_kv_heads * t_max > (1ll << 30))
        return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q || !k || !v || !rope_table || !k_cache_bf16 || !v_cache_bf16 || !lengths || !out_bf16) return BITLINEAR_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(rope_table)) return BITLINEAR_ERR_ALIGN;
    const AttnOwnRow own = {q, k, v, reinterpret_cast<const float2*>(rope_table), static_cast<__nv_bfloat16*>(k_cache_bf16),
                            static_cast<__nv_bfloat16*>(v_cache_bf16)};
    return attn_launch(nullptr, own, true, k_cache_bf16, v_cache_bf16, lengths, seq_ids, M, n_q_heads, n_kv_heads, head_dim, n_seq,
                       t_max, out_bf16, ws, ws_bytes, stream);
}

int bitlinear_lm_head(const void* x_bf16, const void* table_bf16, int M, int V, int K, float* logits, void* stream) {
    if (M < 0 || M > 16 || V <= 0 || K <= 0 || K % 8) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!x_bf16 || !table_bf16 || !logits) return BITLINEAR_ERR_NULL;
    if (!aligned16(x_bf16) || !aligned16(table_bf16)) return BITLINEAR_ERR_ALIGN;
    int sm_count = 0;
    if (const int rc = device_sm_count(&sm_count)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16 *xp = static_cast<const __nv_bfloat16*>(x_bf16), *tp = static_cast<const __nv_bfloat16*>(table_bf16);
    // rows of the staged x: K rounded up to 32 columns (zero-filled), 64 bytes apart modulo 128 so that the two rows a
    // quarter-warp reads together fall into different halves of the banks
    const int x_stride = ((K + 31) / 32 * 64 + 127) / 128 * 128 + 64;
    const size_t smem = (size_t)16 * x_stride;
    if (cudaFuncSetAttribute(lm_head_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_SHAPE;  // K too large for the staged activations
    }
    lm_head_mma_kernel<<<(unsigned)(sm_count * 2), 512, smem, st>>>(xp, tp, M, V, K, x_stride, logits);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

int bitlinear_embed(const int32_t* ids, const void* table_bf16, int M, int V, int K, void* out_bf16, void* stream) {
    if (M < 0 || V <= 0 || K <= 0 || K % 8) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!ids || !table_bf16 || !out_bf16) return BITLINEAR_ERR_NULL;
    if (!aligned16(table_bf16) || !aligned16(out_bf16)) return BITLINEAR_ERR_ALIGN;
    const long long work = (long long)M * (K / 8);
    embed_kernel<<<(unsigned)((work + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        ids, static_cast<const __nv_bfloat16*>(table_bf16), M, V, K, static_cast<__nv_bfloat16*>(out_bf16));
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

}  // extern "C"
