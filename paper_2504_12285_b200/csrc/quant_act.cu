// Stand-alone launch of the fused RMSNorm + absmax int8 quantiser: one CTA per token.
#include "quant_row.cuh"

namespace bitlinear {

namespace {

template <int VPT>
__global__ void __launch_bounds__(kQuantThreads) quant_act_kernel(const __nv_bfloat16* __restrict__ x,
                                                                  const __nv_bfloat16* __restrict__ gain, float eps,
                                                                  int K, int8_t* __restrict__ xq,
                                                                  float* __restrict__ d_out,
                                                                  int32_t* __restrict__ xsum_out) {
    __shared__ RowReduceSmem sm;
    const size_t row = blockIdx.x;
    quant_row<VPT>(x + row * K, gain, eps, K, xq + row * K, d_out + row, xsum_out ? xsum_out + row : nullptr, sm);
}

// Many tokens: one warp per token, eight tokens per CTA.
__global__ void __launch_bounds__(kQuantThreads) quant_act_warp_kernel(const __nv_bfloat16* __restrict__ x,
                                                                       const __nv_bfloat16* __restrict__ gain, float eps,
                                                                       int M, int K, int8_t* __restrict__ xq,
                                                                       float* __restrict__ d_out,
                                                                       int32_t* __restrict__ xsum_out) {
    const size_t row = (size_t)blockIdx.x * kQuantWarps + (threadIdx.x >> 5);
    if (row >= (size_t)M) return;
    quant_row_warp<0>(x + row * K, gain, eps, K, xq + row * K, d_out + row, xsum_out ? xsum_out + row : nullptr);
}

// The same two launch shapes with an element-wise step in front of the quantiser (see RowOp in quant_row.cuh).
template <int VPT>
__global__ void __launch_bounds__(kQuantThreads) quant_act_step_kernel(const RowOp op, const void* __restrict__ x,
                                                                       const __nv_bfloat16* __restrict__ gain, float eps, int K,
                                                                       int8_t* __restrict__ xq, float* __restrict__ d_out,
                                                                       int32_t* __restrict__ xsum_out) {
    __shared__ RowReduceSmem sm;
    const int row = blockIdx.x;
    with_row_source(op, x, row, K, [&](auto src) {
        quant_row_src<VPT, 0>(src, gain, eps, K, xq + (size_t)row * K, d_out + row, xsum_out ? xsum_out + row : nullptr, sm);
    });
}

__global__ void __launch_bounds__(kQuantThreads) quant_act_step_warp_kernel(const RowOp op, const void* __restrict__ x,
                                                                            const __nv_bfloat16* __restrict__ gain, float eps,
                                                                            int M, int K, int8_t* __restrict__ xq,
                                                                            float* __restrict__ d_out,
                                                                            int32_t* __restrict__ xsum_out) {
    const int row = blockIdx.x * kQuantWarps + (threadIdx.x >> 5);
    if (row >= M) return;
    with_row_source(op, x, row, K, [&](auto src) {
        quant_row_warp_src<0>(src, gain, eps, K, xq + (size_t)row * K, d_out + row, xsum_out ? xsum_out + row : nullptr);
    });
}

}  // namespace

cudaError_t launch_quant_act_step(int x_op, const void* x, const void* x2, void* x_out, int arg0, int arg1,
                                  const __nv_bfloat16* gain, float eps, int M, int K, int8_t* xq, float* d, int32_t* xsum,
                                  cudaStream_t st) {
    RowOp op;
    op.x2 = x2; op.x_out = x_out; op.op = x_op; op.arg0 = arg0; op.arg1 = arg1; op.pad = 0;
    const int vpt = (K / 8 + kQuantThreads - 1) / kQuantThreads;
    const dim3 grid((unsigned)M), block(kQuantThreads), gw((unsigned)((M + kQuantWarps - 1) / kQuantWarps));
    if (M >= 64) quant_act_step_warp_kernel<<<gw, block, 0, st>>>(op, x, gain, eps, M, K, xq, d, xsum);
    else if (vpt <= 1) quant_act_step_kernel<1><<<grid, block, 0, st>>>(op, x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 2) quant_act_step_kernel<2><<<grid, block, 0, st>>>(op, x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 4) quant_act_step_kernel<4><<<grid, block, 0, st>>>(op, x, gain, eps, K, xq, d, xsum);
    else quant_act_step_kernel<8><<<grid, block, 0, st>>>(op, x, gain, eps, K, xq, d, xsum);
    return cudaGetLastError();
}

cudaError_t launch_quant_act(const __nv_bfloat16* x, const __nv_bfloat16* gain, float eps, int M, int K,
                             int8_t* xq, float* d, int32_t* xsum, cudaStream_t st) {
    const int n_vec = K / 8;
    const int vpt = (n_vec + kQuantThreads - 1) / kQuantThreads;
    const dim3 grid((unsigned)M), block(kQuantThreads), gw((unsigned)((M + kQuantWarps - 1) / kQuantWarps));
    if (M >= 64) {
        quant_act_warp_kernel<<<gw, block, 0, st>>>(x, gain, eps, M, K, xq, d, xsum);
        return cudaGetLastError();
    }
    if (vpt <= 1) quant_act_kernel<1><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 2) quant_act_kernel<2><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else if (vpt <= 4) quant_act_kernel<4><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);
    else quant_act_kernel<8><<<grid, block, 0, st>>>(x, gain, eps, K, xq, d, xsum);  // K <= 16384
    return cudaGetLastError();
}

}  // namespace bitlinear
