// Element-wise glue between the BitLinear matmuls of a decoder layer (paper Section 2: squared-ReLU feed-forward
// activation; residual connections of the Transformer).  Attention itself is not a BitLinear and is not part of this
// library: the chained decode benchmark uses a fixed stand-in that only mixes the q and v projections.
// Every operation is fp32 with one rounding per arithmetic step, then one round-to-nearest-even cast to bf16.
#include "common.cuh"

namespace bitlinear {

namespace {

__global__ void __launch_bounds__(256) relu2_mul_kernel(const float* __restrict__ gate, const float* __restrict__ up,
                                                        __nv_bfloat16* __restrict__ u, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float r = fmaxf(gate[i], 0.0f);
    u[i] = __float2bfloat16_rn(__fmul_rn(__fmul_rn(r, r), up[i]));
}

__global__ void __launch_bounds__(256) residual_add_kernel(__nv_bfloat16* __restrict__ h, const float* __restrict__ y,
                                                           size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    h[i] = __float2bfloat16_rn(__fadd_rn(__bfloat162float(h[i]), y[i]));
}

__global__ void __launch_bounds__(256) attn_standin_kernel(const float* __restrict__ q, const float* __restrict__ v,
                                                           __nv_bfloat16* __restrict__ o_in, int M, int n_q, int n_kv,
                                                           int head_dim) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t width = (size_t)n_q * head_dim;
    if (i >= (size_t)M * width) return;
    const size_t m = i / width;
    const int c = (int)(i - m * width), head = c / head_dim, j = c - head * head_dim;
    const int kv = head / (n_q / n_kv);
    o_in[i] = __float2bfloat16_rn(__fadd_rn(q[i], v[m * (size_t)n_kv * head_dim + (size_t)kv * head_dim + j]));
}

inline unsigned blocks_for(size_t n) { return (unsigned)((n + 255) / 256); }

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

int bitlinear_glue_relu2_mul(const float* gate, const float* up, void* u_bf16, int M, int F, void* stream) {
    if (M < 0 || F <= 0) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!gate || !up || !u_bf16) return BITLINEAR_ERR_NULL;
    const size_t n = (size_t)M * F;
    relu2_mul_kernel<<<blocks_for(n), 256, 0, static_cast<cudaStream_t>(stream)>>>(gate, up, static_cast<__nv_bfloat16*>(u_bf16), n);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

int bitlinear_glue_residual_add(void* h_bf16, const float* y, int M, int N, void* stream) {
    if (M < 0 || N <= 0) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!h_bf16 || !y) return BITLINEAR_ERR_NULL;
    const size_t n = (size_t)M * N;
    residual_add_kernel<<<blocks_for(n), 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<__nv_bfloat16*>(h_bf16), y, n);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

int bitlinear_glue_attn_standin(const float* q, const float* v, void* o_in_bf16, int M, int n_q_heads, int n_kv_heads,
                                int head_dim, void* stream) {
    if (M < 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || n_q_heads % n_kv_heads) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!q || !v || !o_in_bf16) return BITLINEAR_ERR_NULL;
    const size_t n = (size_t)M * n_q_heads * head_dim;
    attn_standin_kernel<<<blocks_for(n), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        q, v, static_cast<__nv_bfloat16*>(o_in_bf16), M, n_q_heads, n_kv_heads, head_dim);
    return cudaGetLastError() == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA;
}

}  // extern "C"
