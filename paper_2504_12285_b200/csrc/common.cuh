// Shared declarations of the BitLinear CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bitlinear.h"

namespace bitlinear {

// Packed layout constants (see "Packed weight layout" in bitlinear.h).
constexpr int kTileRows = 16;
constexpr int kTileCols = 256;
constexpr int kTileBytes = 1024;
constexpr int kMaxK = 16384;
// Dense layout (five ternary values per byte): tiles of 16 rows x 320 columns, also 1024 bytes; K is padded with zero
// weights to a whole number of tiles.
constexpr int kDenseTileCols = 320;
__host__ __device__ inline int dense_k_tiles(int K) { return (K + kDenseTileCols - 1) / kDenseTileCols; }
constexpr int kGemvMaxTokens = 16;

__host__ __device__ inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline bool shape_ok(int N, int K) {
    return N > 0 && K >= kTileCols && K <= kMaxK && (N % kTileRows) == 0 && (K % kTileCols) == 0;
}
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Layout of the forward workspace: [xq M*K][d M floats][xsum M ints][tensor-core scratch].
struct ForwardWorkspace {
    size_t xq_off, d_off, xsum_off, mm_off, total;
};
ForwardWorkspace forward_workspace(int M, int N, int K, size_t mm_bytes);

// ---- kernel launchers (each returns a cudaError_t from the launch) ---------------------------
cudaError_t launch_absmean(const void* W, int w_dtype, size_t count, float eps_w, double* partials,
                           int n_partials, float* s_w_out, cudaStream_t st);
cudaError_t launch_quant_pack(const void* W, int w_dtype, int N, int K, const float* s_w, uint32_t* packed,
                              cudaStream_t st);
cudaError_t launch_unpack_i8(const uint32_t* packed, int N, int K, int8_t* wq, cudaStream_t st);
cudaError_t launch_unpack_codes_u8(const uint32_t* packed, int N, int K, uint8_t* codes, cudaStream_t st);
int absmean_num_partials(size_t count);
cudaError_t launch_quant_pack5(const void* W, int w_dtype, int N, int K, const float* s_w, uint32_t* packed, cudaStream_t st);
cudaError_t launch_unpack5_i8(const uint8_t* packed, int N, int K, int8_t* wq, cudaStream_t st);

cudaError_t launch_quant_act(const __nv_bfloat16* x, const __nv_bfloat16* gain, float eps, int M, int K,
                             int8_t* xq, float* d, int32_t* xsum, cudaStream_t st);

// The same with an element-wise step in front (x_op = BITLINEAR_X_*, operands as in bitlinear_problem).
cudaError_t launch_quant_act_step(int x_op, const void* x, const void* x2, void* x_out, int arg0, int arg1,
                                  const __nv_bfloat16* gain, float eps, int M, int K, int8_t* xq, float* d, int32_t* xsum,
                                  cudaStream_t st);

cudaError_t launch_gemv(const int8_t* xq, const float* d, const int32_t* xsum, const uint32_t* packed,
                        const float* s_w, int M, int N, int K, void* y, int y_dtype, int32_t* acc_out,
                        cudaStream_t st);

// One matmul of a group (device copy, read by the kernel through shared memory).
struct GemmProblem {
    const uint8_t* a_tiles;  // activations as 128 x 128 shared-memory tile images (A_TILED), else unused
    const uint8_t* codes;    // weight codes as 256 x 128 shared-memory tile images
    const float* d;
    const int32_t* xsum;
    const float* s_w;
    void* y;
    int32_t* acc_out;
    int M, N, K, y_dtype;
    int m_tiles;     // ceil(M / 128)
    int tile_begin;  // tiles of the problems before this one
    int nt_begin;    // 256-row weight tiles of the problems before this one (index into the ready counters)
    int at_begin;    // index of the token-tile counters of this problem's quantised activations (GemmGroupHeader::a_ready)
};
constexpr int kMaxGroup = 32;
struct GemmGroupHeader {
    int count, total_tiles;
    unsigned long long region_base;  // CTA-pair kernel: address its tensor map starts at (tile images are addressed as rows of 128 B)
    // CTA-pair kernel, or nullptr: ready[nt_begin + nt] counts the packed words of 256-row weight tile nt of a problem
    // whose codes have been written; the kernel runs beside the expansion launch and reads that tile only once the
    // count has reached rows_in_tile * K / 16
    const int* ready;
    // CTA-pair kernel: 1 if the launch right before it is the quantiser, whose results (token images, scales, code
    // sums) it must wait for with griddepcontrol.wait; 0 if it is the expansion launch, which `ready` covers
    int wait_primary;
    // CTA-pair kernel on packed weights: 1 if the (single) problem's activations are a row-major [M][K] matrix fetched
    // through a swizzling tensor map instead of tile images
    int a_row_major;
    // CTA-pair kernel, or nullptr: a_ready[at_begin + mt] counts the tokens of 256-token tile mt of a problem's activations
    // that the quantiser launch has finished (codes, scale and code sum written); the kernel then runs beside the quantiser
    // too and reads a token tile once the count has reached the tile's tokens
    const int* a_ready;
};
// layout of the uploaded group table: GemmGroupHeader, then count x GemmProblem
constexpr size_t kGroupTableBytes = sizeof(GemmGroupHeader) + kMaxGroup * sizeof(GemmProblem);
// the grouped launch keeps one 128-byte tensor map per problem (view of its packed weights) behind the table
constexpr size_t kGroupMapsOffset = (kGroupTableBytes + 127) / 128 * 128;
constexpr size_t kGroupTableDevBytes = kGroupMapsOffset + kMaxGroup * 128;

// Grouped launch: fills m_tiles / tile_begin, uploads the table to table_dev (kGroupTableDevBytes when `packed` is given,
// else kGroupTableBytes) and runs every tile of
// every problem in one persistent kernel.  a_tiled = activations given as tile images (any count), else one problem with
// row-major activations.  Returns a bitlinear_status.
// `before` (optional) is called after the table upload and before the GEMM kernel is launched: launches that produce
// the operands go there, so that no copy sits between them and the GEMM kernel.  With `ready` set (see
// GemmGroupHeader) the CTA-pair kernel is launched as a programmatic dependent of the last of those launches.
typedef int (*GemmBeforeKernel)(void* ctx);
int gemm_launch(GemmProblem* probs, int count, bool a_tiled, const int8_t* xq_row_major, uint8_t* table_dev, cudaStream_t st,
                const void* region_base = nullptr, size_t region_bytes = 0, const int* ready = nullptr,
                GemmBeforeKernel before = nullptr, void* before_ctx = nullptr, bool wait_primary = false,
                const int* a_ready = nullptr, const void* const* packed = nullptr);
size_t gemm_codes_bytes(int N, int K);
size_t gemm_a_tiles_bytes(int M, int K);

// tcgen05 tensor-core GEMM on unpacked codes; returns a bitlinear_status.
int gemm_tcgen05(const int8_t* xq, const float* d, const int32_t* xsum, const uint8_t* codes, const float* s_w,
                 int M, int N, int K, void* y, int y_dtype, int32_t* acc_out, cudaStream_t st);
size_t gemm_scratch_bytes(int N, int K);
int gemm_tcgen05_packed(const int8_t* xq, const float* d, const int32_t* xsum, const void* packed, const float* s_w, int M,
                        int N, int K, void* y, int y_dtype, int32_t* acc_out, uint8_t* table_dev, cudaStream_t st);
bool gemm_pairs_available();  // the SMs of the current device pair up (CTA-pair kernels can run)
int int8_mma_rate_probe(int n_mma, double* ops_out, cudaStream_t st);

// SM count of the current device (cached per device; BITLINEAR_ERR_ARCH unless it is compute capability 10.x).
int device_sm_count(int* sm_count);

// Sticky device-side status word (set by kernels whose bounded waits ran out).
int* device_status_word();

}  // namespace bitlinear
