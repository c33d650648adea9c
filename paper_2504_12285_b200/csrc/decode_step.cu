// The rest of a decode step around the BitLinear layers (paper Section 2: rotary position embeddings; a Transformer
// decoder, i.e. causal attention - with grouped queries in the 2B configuration; a vocabulary of 128,256 tokens, hence
// a bf16 embedding table and an output head of that many rows, which is larger than all packed BitLinear weights
// together).  None of these is a BitLinear; they are here so that a whole decoded token can be timed.
//
//   rope_kv_kernel            : rotates q and k (pairs i, i + head_dim/2; angle = position * base^(-2i/head_dim), formed
//                               in fp64 because positions reach the thousands), writes q as bf16 and appends k, v to
//                               the bf16 cache of the token's sequence.
//   attn_decode_partial_kernel: one CTA per (token, KV head, slice of 64 cache positions), one warp per query head of the
//                               group; the slice is bulk-copied into shared memory once and scored by all heads;
//                               softmax in fp32; partial (max, sum, weighted values) per slice.
//   attn_decode_combine_kernel: merges the slices of a (token, query head) and writes bf16.
//   lm_head_kernel            : logits = x . E^T for up to 16 tokens, one warp per vocabulary row, the table streamed
//                               once with 128-bit loads (HBM-bound: 657 MB for 128,256 x 2560).
//   embed_kernel              : row gather.
#include "common.cuh"
#include "sm100_sync.cuh"

#include <type_traits>

namespace bitlinear {

namespace {

__device__ __forceinline__ float bf16_lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---------------------------------------------------------------------------------------------- RoPE + cache append

__global__ void __launch_bounds__(256) rope_kv_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                                      const float* __restrict__ v, const int* __restrict__ positions,
                                                      const int* __restrict__ seq_ids, int M, int n_q, int n_kv, int hd,
                                                      double log2_base, __nv_bfloat16* __restrict__ q_out,
                                                      __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                                                      int t_max) {
    const int half = hd / 2;
    const int pairs_per_tok = (n_q + n_kv) * half;
    const int vals_per_tok = n_kv * hd;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n_rot = (long long)M * pairs_per_tok;
    if (idx < n_rot) {
        const int m = (int)(idx / pairs_per_tok), r = (int)(idx - (long long)m * pairs_per_tok);
        const int head = r / half, i = r - head * half;
        const int pos = positions[m];
        const double angle = (double)pos * exp2(-2.0 * (double)i / (double)hd * log2_base);
        double sd, cd;
        sincos(angle, &sd, &cd);
        const float c = (float)cd, s = (float)sd;
        const bool is_q = head < n_q;
        const float* src = is_q ? q + (size_t)m * n_q * hd + (size_t)head * hd : k + (size_t)m * n_kv * hd + (size_t)(head - n_q) * hd;
        const float lo = src[i], hi = src[i + half];
        const float o_lo = __fsub_rn(__fmul_rn(lo, c), __fmul_rn(hi, s));
        const float o_hi = __fadd_rn(__fmul_rn(hi, c), __fmul_rn(lo, s));
        if (!is_q && (pos < 0 || pos >= t_max)) return;  // a position outside the cache is not stored
        __nv_bfloat16* dst;
        if (is_q) dst = q_out + (size_t)m * n_q * hd + (size_t)head * hd;
        else dst = k_cache + ((size_t)(seq_ids ? seq_ids[m] : 0) * t_max + pos) * vals_per_tok + (size_t)(head - n_q) * hd;
        dst[i] = __float2bfloat16_rn(o_lo);
        dst[i + half] = __float2bfloat16_rn(o_hi);
    } else if (idx < n_rot + (long long)M * vals_per_tok) {
        const long long j = idx - n_rot;
        const int m = (int)(j / vals_per_tok), e = (int)(j - (long long)m * vals_per_tok);
        if (positions[m] < 0 || positions[m] >= t_max) return;
        v_cache[((size_t)(seq_ids ? seq_ids[m] : 0) * t_max + positions[m]) * vals_per_tok + e] =
            __float2bfloat16_rn(v[(size_t)m * vals_per_tok + e]);
    }
}

// ---------------------------------------------------------------------------------------------- decode attention

constexpr int kAttnKeys = 64;  // cache positions per CTA

// partial result of one slice of the cache for one (token, query head): weighted values, running maximum, sum of weights
template <int HD>
struct __align__(16) AttnPartial {
    float o[HD];
    float m, l, pad[2];
};

template <int HD>
constexpr size_t attn_smem_bytes(int group) {
    return (size_t)2 * kAttnKeys * HD * 2 + (size_t)group * (HD + kAttnKeys) * sizeof(float) + 16;
}

// One CTA per (slice of 64 cache positions, KV head, token); one warp per query head of the group.  The slice's key and
// value rows of this KV head (HD bf16 each, contiguous) are brought into shared memory by one bulk copy per row, all in
// flight at once, so that a CTA pays one round trip to HBM; then every warp scores the 64 keys against its query
// (one key per lane, the 16-byte chunks of a row visited in a lane-rotated order so that the lanes of a quarter-warp
// hit distinct banks), takes the softmax weights of the slice and accumulates the values (one lane per HD/32
// coordinates).  Slices past the token's length return at once and are not read by the combine kernel.
template <int HD>
__global__ void __launch_bounds__(256) attn_decode_partial_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_cache,
                                                                  const __nv_bfloat16* __restrict__ v_cache, const int* __restrict__ lengths,
                                                                  const int* __restrict__ seq_ids, int n_q, int n_kv, int t_max,
                                                                  int splits, float scale, AttnPartial<HD>* __restrict__ part,
                                                                  int* __restrict__ status_word) {
    constexpr int NCH = HD / 8;   // 16-byte chunks per row
    constexpr int CPL = HD / 32;  // value coordinates per lane
    extern __shared__ __align__(16) uint8_t attn_smem[];
    const int split = blockIdx.x, g = blockIdx.y, m = blockIdx.z;
    const int group = n_q / n_kv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = g * group + warp;  // this warp's query head
    const int len = min(max(lengths[m], 0), t_max);
    const int t0 = split * kAttnKeys;
    if (t0 >= len) return;  // the whole CTA: nothing of this slice is live
    const int n = min(kAttnKeys, len - t0);

    uint4* k_s = reinterpret_cast<uint4*>(attn_smem);                                  // [64][NCH]
    uint4* v_s = k_s + kAttnKeys * NCH;                                                // [64][NCH]
    float* q_s = reinterpret_cast<float*>(v_s + kAttnKeys * NCH) + warp * HD;          // two planes [NCH][4] per head
    float* p_s = reinterpret_cast<float*>(v_s + kAttnKeys * NCH) + group * HD + warp * kAttnKeys;
    uint64_t* bar = reinterpret_cast<uint64_t*>(reinterpret_cast<float*>(v_s + kAttnKeys * NCH) + group * (HD + kAttnKeys));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar + 1);
    const uint32_t bar_s = smem_u32(bar);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar_s, 1);
        mbar_init_fence();
    }
    __syncthreads();
    if (warp == 0) {
        if (lane == 0) mbar_expect_tx(bar_s, (uint32_t)n * HD * 2u * 2u);
        __syncwarp();
        const size_t row0 = ((size_t)(seq_ids ? seq_ids[m] : 0) * t_max + t0) * ((size_t)n_kv * HD) + (size_t)g * HD;
        for (int r = lane; r < n; r += 32) {
            const size_t off = row0 + (size_t)r * n_kv * HD;
            bulk_load(smem_u32(k_s + r * NCH), k_cache + off, HD * 2, bar_s);
            bulk_load(smem_u32(v_s + r * NCH), v_cache + off, HD * 2, bar_s);
        }
    }
    // the query as fp32 in two planes: plane 0 holds coordinates 8j .. 8j+3 of chunk j, plane 1 coordinates 8j+4 .. 8j+7,
    // so that lanes reading eight different chunks with 16-byte loads cover all 32 banks once
    {
        const __nv_bfloat16* qh = q + ((size_t)m * n_q + h) * HD;
        for (int c = lane; c < HD; c += 32) q_s[(c >> 2 & 1) * (HD / 2) + (c >> 3) * 4 + (c & 3)] = __bfloat162float(qh[c]);
    }
    __syncwarp();
    const bool ok = mbar_wait(bar_s, 0, abort_flag);
    if (!ok) {
        if (lane == 0 && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
        abort_drain();
        return;
    }

    // scores of keys lane and lane + 32
    float s[kAttnKeys / 32];
#pragma unroll
    for (int pass = 0; pass < kAttnKeys / 32; ++pass) {
        const int t = pass * 32 + lane;
        float dot = 0.0f;
        if (t < n) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int j = (c + lane) & (NCH - 1);
                const uint4 u = k_s[t * NCH + j];
                const float4 qa = *reinterpret_cast<const float4*>(q_s + j * 4);
                const float4 qb = *reinterpret_cast<const float4*>(q_s + HD / 2 + j * 4);
                dot = fmaf(qa.x, bf16_lo_f(u.x), dot);
                dot = fmaf(qa.y, bf16_hi_f(u.x), dot);
                dot = fmaf(qa.z, bf16_lo_f(u.y), dot);
                dot = fmaf(qa.w, bf16_hi_f(u.y), dot);
                dot = fmaf(qb.x, bf16_lo_f(u.z), dot);
                dot = fmaf(qb.y, bf16_hi_f(u.z), dot);
                dot = fmaf(qb.z, bf16_lo_f(u.w), dot);
                dot = fmaf(qb.w, bf16_hi_f(u.w), dot);
            }
        }
        s[pass] = t < n ? dot * scale : -INFINITY;
    }
    float mx = s[0];
#pragma unroll
    for (int pass = 1; pass < kAttnKeys / 32; ++pass) mx = fmaxf(mx, s[pass]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));  // finite: key t0 is live
    float l = 0.0f;
#pragma unroll
    for (int pass = 0; pass < kAttnKeys / 32; ++pass) {
        const float p = expf(s[pass] - mx);  // expf(-inf) = 0 for the keys past the end
        p_s[pass * 32 + lane] = p;
        l += p;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    __syncwarp();

    // weighted values: this lane's CPL coordinates over the n live keys, two independent chains
    float o0[CPL], o1[CPL];
#pragma unroll
    for (int e = 0; e < CPL; ++e) o0[e] = o1[e] = 0.0f;
    const uint16_t* v16 = reinterpret_cast<const uint16_t*>(v_s) + lane * CPL;
    auto add_key = [&](int t, float (&o)[CPL]) {
        const float p = p_s[t];
        if constexpr (CPL == 4) {
            const uint2 u = *reinterpret_cast<const uint2*>(v16 + t * HD);
            o[0] = fmaf(p, bf16_lo_f(u.x), o[0]);
            o[1] = fmaf(p, bf16_hi_f(u.x), o[1]);
            o[2] = fmaf(p, bf16_lo_f(u.y), o[2]);
            o[3] = fmaf(p, bf16_hi_f(u.y), o[3]);
        } else {
            const uint32_t u = *reinterpret_cast<const uint32_t*>(v16 + t * HD);
            o[0] = fmaf(p, bf16_lo_f(u), o[0]);
            o[1] = fmaf(p, bf16_hi_f(u), o[1]);
        }
    };
    int t = 0;
    for (; t + 2 <= n; t += 2) {
        add_key(t, o0);
        add_key(t + 1, o1);
    }
    if (t < n) add_key(t, o0);

    AttnPartial<HD>& dst = part[((size_t)m * n_q + h) * splits + split];
    if constexpr (CPL == 4) {
        *reinterpret_cast<float4*>(dst.o + lane * 4) = make_float4(o0[0] + o1[0], o0[1] + o1[1], o0[2] + o1[2], o0[3] + o1[3]);
    } else {
        *reinterpret_cast<float2*>(dst.o + lane * 2) = make_float2(o0[0] + o1[0], o0[1] + o1[1]);
    }
    if (lane == 0) { dst.m = mx; dst.l = l; }
}

// Merges the live slices of a (token, query head) and writes bf16; a token of length 0 gets zeros.
template <int HD>
__global__ void __launch_bounds__(HD) attn_decode_combine_kernel(const AttnPartial<HD>* __restrict__ part, const int* __restrict__ lengths,
                                                                 int n_q, int t_max, int splits, __nv_bfloat16* __restrict__ out) {
    const size_t mh = blockIdx.x;  // token * n_q + head
    const int len = min(max(lengths[mh / n_q], 0), t_max);
    const int live = (len + kAttnKeys - 1) / kAttnKeys;
    const AttnPartial<HD>* p = part + mh * splits;
    float m_all = -INFINITY;
    for (int s = 0; s < live; ++s) m_all = fmaxf(m_all, p[s].m);
    float l = 0.0f, o = 0.0f;
    for (int s = 0; s < live; ++s) {
        const float f = expf(p[s].m - m_all);
        l = fmaf(p[s].l, f, l);
        o = fmaf(p[s].o[threadIdx.x], f, o);
    }
    out[mh * HD + threadIdx.x] = __float2bfloat16_rn(l > 0.0f ? o / l : 0.0f);
}

// ---------------------------------------------------------------------------------------------- output head, embedding

template <int MT>
__global__ void __launch_bounds__(256) lm_head_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ table,
                                                      int M, int V, int K, float* __restrict__ logits) {
    extern __shared__ __align__(16) uint8_t xs_raw[];
    uint4* xs = reinterpret_cast<uint4*>(xs_raw);  // [MT][K] bf16
    const int n_vec = K / 8;
    for (int i = threadIdx.x; i < MT * n_vec; i += blockDim.x) {
        const int m = i / n_vec;
        xs[i] = m < M ? reinterpret_cast<const uint4*>(x)[(size_t)m * n_vec + (i - m * n_vec)] : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int v = blockIdx.x * (blockDim.x >> 5) + warp; v < V; v += warps) {
        const uint4* row = reinterpret_cast<const uint4*>(table + (size_t)v * K);
        float acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0.0f;
#pragma unroll 4
        for (int c = lane; c < n_vec; c += 32) {
            const uint4 u = __ldcs(row + c);  // streamed once
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
            float e[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) { e[2 * j] = bf16_lo_f(w[j]); e[2 * j + 1] = bf16_hi_f(w[j]); }
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint4 xu = xs[m * n_vec + c];
                const uint32_t xw[4] = {xu.x, xu.y, xu.z, xu.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[m] = fmaf(bf16_lo_f(xw[j]), e[2 * j], acc[m]);
                    acc[m] = fmaf(bf16_hi_f(xw[j]), e[2 * j + 1], acc[m]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float a = acc[m];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            if (lane == 0 && m < M) logits[(size_t)m * V + v] = a;
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

int attn_splits(int t_max) { return (t_max + kAttnKeys - 1) / kAttnKeys; }

bool attn_dims_ok(int M, int n_q, int n_kv, int hd, int t_max) {
    return M >= 0 && n_q > 0 && n_kv > 0 && n_q % n_kv == 0 && n_q / n_kv <= 8 && (hd == 64 || hd == 128) && t_max > 0 && t_max <= (1 << 22);
}

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

int bitlinear_rope_kv(const float* q, const float* k, const float* v, const int32_t* positions, const int32_t* seq_ids, int M,
                      int n_q_heads, int n_kv_heads, int head_dim, float rope_base, void* q_out_bf16, void* k_cache_bf16,
                      void* v_cache_bf16, int t_max, void* stream) {
    if (M < 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || head_dim % 8 || t_max <= 0 || !(rope_base > 1.0f))
        return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q || !k || !v || !positions || !q_out_bf16 || !k_cache_bf16 || !v_cache_bf16) return BITLINEAR_ERR_NULL;
    const long long work = (long long)M * ((n_q_heads + n_kv_heads) * (head_dim / 2) + n_kv_heads * head_dim);
    rope_kv_kernel<<<(unsigned)((work + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        q, k, v, positions, seq_ids, M, n_q_heads, n_kv_heads, head_dim, log2((double)rope_base),
        static_cast<__nv_bfloat16*>(q_out_bf16), static_cast<__nv_bfloat16*>(k_cache_bf16), static_cast<__nv_bfloat16*>(v_cache_bf16),
        t_max);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

size_t bitlinear_attention_workspace_bytes(int M, int n_q_heads, int n_kv_heads, int head_dim, int t_max) {
    if (!attn_dims_ok(M, n_q_heads, n_kv_heads, head_dim, t_max)) return 0;
    return (size_t)(M > 0 ? M : 1) * n_q_heads * attn_splits(t_max) * (sizeof(float) * (4 + head_dim));
}

int bitlinear_attention_decode(const void* q_bf16, const void* k_cache_bf16, const void* v_cache_bf16, const int32_t* lengths,
                               const int32_t* seq_ids, int M, int n_q_heads, int n_kv_heads, int head_dim, int t_max,
                               void* out_bf16, void* ws, size_t ws_bytes, void* stream) {
    if (!attn_dims_ok(M, n_q_heads, n_kv_heads, head_dim, t_max)) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q_bf16 || !k_cache_bf16 || !v_cache_bf16 || !lengths || !out_bf16) return BITLINEAR_ERR_NULL;
    if (!aligned16(q_bf16) || !aligned16(k_cache_bf16) || !aligned16(v_cache_bf16) || !aligned16(out_bf16)) return BITLINEAR_ERR_ALIGN;
    if (!ws || !aligned16(ws) || ws_bytes < bitlinear_attention_workspace_bytes(M, n_q_heads, n_kv_heads, head_dim, t_max))
        return BITLINEAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int splits = attn_splits(t_max), group = n_q_heads / n_kv_heads;
    const float scale = 1.0f / sqrtf((float)head_dim);
    const dim3 grid((unsigned)splits, (unsigned)n_kv_heads, (unsigned)M);
    const __nv_bfloat16 *qp = static_cast<const __nv_bfloat16*>(q_bf16), *kp = static_cast<const __nv_bfloat16*>(k_cache_bf16),
                        *vp = static_cast<const __nv_bfloat16*>(v_cache_bf16);
    int* status = device_status_word();
    auto launch = [&](auto hd_tag) {
        constexpr int HD = decltype(hd_tag)::value;
        auto* part = static_cast<AttnPartial<HD>*>(ws);
        attn_decode_partial_kernel<HD><<<grid, 32 * group, attn_smem_bytes<HD>(group), st>>>(qp, kp, vp, lengths, seq_ids, n_q_heads, n_kv_heads,
                                                                                          t_max, splits, scale, part, status);
        attn_decode_combine_kernel<HD><<<(unsigned)(M * n_q_heads), HD, 0, st>>>(part, lengths, n_q_heads, t_max, splits,
                                                                               static_cast<__nv_bfloat16*>(out_bf16));
    };
    if (head_dim == 128) launch(std::integral_constant<int, 128>{});
    else launch(std::integral_constant<int, 64>{});
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
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
    const unsigned grid = (unsigned)(sm_count * 4);
    auto launch = [&](auto kernel, int mt) {
        const size_t smem = (size_t)mt * K * 2;
        if (smem > 48 * 1024 && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return (int)BITLINEAR_ERR_SHAPE;
        }
        kernel<<<grid, 256, smem, st>>>(xp, tp, M, V, K, logits);
        return cudaGetLastError() == cudaSuccess ? (int)BITLINEAR_OK : (int)BITLINEAR_ERR_CUDA;
    };
    if (M == 1) return launch(lm_head_kernel<1>, 1);
    if (M <= 2) return launch(lm_head_kernel<2>, 2);
    if (M <= 4) return launch(lm_head_kernel<4>, 4);
    if (M <= 8) return launch(lm_head_kernel<8>, 8);
    return launch(lm_head_kernel<16>, 16);
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
