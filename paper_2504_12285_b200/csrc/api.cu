// C ABI of the BitLinear library: argument checks, workspace carving and kernel dispatch.
#include <mutex>

#include "common.cuh"
#include "decode_level.cuh"
#include "sm100_sync.cuh"

namespace bitlinear {

namespace {

__device__ int g_status_word = 0;

// One CTA waits on an mbarrier that nobody ever arrives on: the bounded wait must give up after limit_ns, raise the
// CTA's abort flag and let the kernel end by itself with the sticky status word set - the path every production kernel
// takes when one of its waits runs out.
__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(unsigned long long limit_ns, int* status_word) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag) && status_word != nullptr) atomicExch(status_word, BITLINEAR_ERR_TIMEOUT);
}

constexpr size_t kWsAlign = 256;

// Per-device check that the GPU is compute capability 10.x (the kernels are built for sm_100a only).
int check_arch() {
    static std::mutex mu;
    static int verdict[64];  // 0 = unknown, 1 = ok, 2 = wrong arch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (dev < 0 || dev >= 64) return BITLINEAR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (verdict[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        verdict[dev] = (major == 10) ? 1 : 2;
    }
    return verdict[dev] == 1 ? BITLINEAR_OK : BITLINEAR_ERR_ARCH;
}

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? BITLINEAR_OK : BITLINEAR_ERR_CUDA; }

bool use_gemm(int M, int N, int path) {
    if (path == BITLINEAR_PATH_GEMM) return true;
    if (path == BITLINEAR_PATH_GEMV) return false;
    return M > kGemvMaxTokens && (N % 128) == 0;
}

}  // namespace

int device_sm_count(int* sm_count) {
    static std::mutex mu;
    static int sm_of[64];
    if (int rc = check_arch()) return rc;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (sm_of[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        sm_of[dev] = n;
    }
    *sm_count = sm_of[dev];
    return BITLINEAR_OK;
}

int* device_status_word() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return p;
}

ForwardWorkspace forward_workspace(int M, int N, int K, size_t mm_bytes) {
    (void)N;
    ForwardWorkspace w;
    size_t off = 0;
    w.xq_off = off;
    off = align_up(off + (size_t)M * K, kWsAlign);
    w.d_off = off;
    off = align_up(off + (size_t)M * sizeof(float), kWsAlign);
    w.xsum_off = off;
    off = align_up(off + (size_t)M * sizeof(int32_t), kWsAlign);
    w.mm_off = off;
    off = align_up(off + mm_bytes, kWsAlign);
    w.total = off;
    return w;
}

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

const char* bitlinear_status_string(int status) {
    switch (status) {
        case BITLINEAR_OK: return "ok";
        case BITLINEAR_ERR_NULL: return "null pointer";
        case BITLINEAR_ERR_SHAPE: return "unsupported shape";
        case BITLINEAR_ERR_ALIGN: return "pointer not 16-byte aligned";
        case BITLINEAR_ERR_WORKSPACE: return "workspace missing or too small";
        case BITLINEAR_ERR_DTYPE: return "unknown dtype code";
        case BITLINEAR_ERR_ARCH: return "device is not compute capability 10.x";
        case BITLINEAR_ERR_CUDA: return "CUDA call or launch failed";
        case BITLINEAR_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

int bitlinear_version(void) { return 100; }

size_t bitlinear_packed_bytes(int N, int K) { return shape_ok(N, K) ? (size_t)N * K / 4 : 0; }

size_t bitlinear_pack_workspace_bytes(int N, int K) {
    if (!shape_ok(N, K)) return 0;
    return align_up((size_t)absmean_num_partials((size_t)N * K) * sizeof(double), kWsAlign);
}

size_t bitlinear_matmul_workspace_bytes(int M, int N, int K, int path) {
    if (!shape_ok(N, K) || M < 0) return 0;
    if (path < BITLINEAR_PATH_AUTO || path > BITLINEAR_PATH_GEMM) return 0;
    if (!use_gemm(M, N, path)) return 0;
    return align_up(gemm_scratch_bytes(N, K), kWsAlign);
}

size_t bitlinear_workspace_bytes(int M, int N, int K) {
    if (!shape_ok(N, K) || M < 0) return 0;
    return forward_workspace(M, N, K, bitlinear_matmul_workspace_bytes(M, N, K, BITLINEAR_PATH_AUTO)).total;
}

int bitlinear_pack_weights(const void* W, int w_dtype, int N, int K, float eps_w, void* packed_out, float* s_w_out,
                           void* ws, size_t ws_bytes, void* stream) {
    if (!W || !packed_out || !s_w_out) return BITLINEAR_ERR_NULL;
    if (w_dtype != BITLINEAR_F32 && w_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (!shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(packed_out) || (reinterpret_cast<uintptr_t>(s_w_out) & 3u)) return BITLINEAR_ERR_ALIGN;
    if (!ws || ws_bytes < bitlinear_pack_workspace_bytes(N, K) || !aligned16(ws)) return BITLINEAR_ERR_WORKSPACE;
    if (int rc = check_arch()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t count = (size_t)N * K;
    cudaError_t e = launch_absmean(W, w_dtype, count, eps_w, static_cast<double*>(ws), absmean_num_partials(count),
                                   s_w_out, st);
    if (e != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return cuda_status(launch_quant_pack(W, w_dtype, N, K, s_w_out, static_cast<uint32_t*>(packed_out), st));
}

size_t bitlinear_packed5_bytes(int N, int K) {
    return shape_ok(N, K) ? (size_t)(N / kTileRows) * dense_k_tiles(K) * kTileBytes : 0;
}

int bitlinear_pack_weights5(const void* W, int w_dtype, int N, int K, float eps_w, void* packed5_out, float* s_w_out,
                            void* ws, size_t ws_bytes, void* stream) {
    if (!W || !packed5_out || !s_w_out) return BITLINEAR_ERR_NULL;
    if (w_dtype != BITLINEAR_F32 && w_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (!shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(packed5_out) || (reinterpret_cast<uintptr_t>(s_w_out) & 3u)) return BITLINEAR_ERR_ALIGN;
    if (!ws || ws_bytes < bitlinear_pack_workspace_bytes(N, K) || !aligned16(ws)) return BITLINEAR_ERR_WORKSPACE;
    if (int rc = check_arch()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t count = (size_t)N * K;
    cudaError_t e = launch_absmean(W, w_dtype, count, eps_w, static_cast<double*>(ws), absmean_num_partials(count),
                                   s_w_out, st);
    if (e != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return cuda_status(launch_quant_pack5(W, w_dtype, N, K, s_w_out, static_cast<uint32_t*>(packed5_out), st));
}

int bitlinear_unpack_weights5(const void* packed5, int N, int K, int8_t* wq_out, void* stream) {
    if (!packed5 || !wq_out) return BITLINEAR_ERR_NULL;
    if (!shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (!aligned16(packed5) || !aligned16(wq_out)) return BITLINEAR_ERR_ALIGN;
    if (int rc = check_arch()) return rc;
    return cuda_status(launch_unpack5_i8(static_cast<const uint8_t*>(packed5), N, K, wq_out, static_cast<cudaStream_t>(stream)));
}

int bitlinear_unpack_weights(const void* packed, int N, int K, int8_t* wq_out, void* stream) {
    if (!packed || !wq_out) return BITLINEAR_ERR_NULL;
    if (!shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(wq_out)) return BITLINEAR_ERR_ALIGN;
    if (int rc = check_arch()) return rc;
    return cuda_status(launch_unpack_i8(static_cast<const uint32_t*>(packed), N, K, wq_out,
                                        static_cast<cudaStream_t>(stream)));
}

int bitlinear_quant_act(const void* x_bf16, const void* gain, float rms_eps, int M, int K, int8_t* xq_out,
                        float* d_out, int32_t* xsum_out, void* stream) {
    if (M < 0 || !shape_ok(kTileRows, K)) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!x_bf16 || !xq_out || !d_out) return BITLINEAR_ERR_NULL;
    if (!aligned16(x_bf16) || !aligned16(xq_out) || (gain && !aligned16(gain)) ||
        (reinterpret_cast<uintptr_t>(d_out) & 3u) || (reinterpret_cast<uintptr_t>(xsum_out) & 3u))
        return BITLINEAR_ERR_ALIGN;
    if (int rc = check_arch()) return rc;
    return cuda_status(launch_quant_act(static_cast<const __nv_bfloat16*>(x_bf16),
                                        static_cast<const __nv_bfloat16*>(gain), rms_eps, M, K, xq_out, d_out,
                                        xsum_out, static_cast<cudaStream_t>(stream)));
}

int bitlinear_quant_act_relu2(const float* gate, const float* up, const void* gain, float rms_eps, int M, int F,
                              void* x_out_bf16, int8_t* xq_out, float* d_out, int32_t* xsum_out, void* stream) {
    if (M < 0 || !shape_ok(kTileRows, F)) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!gate || !up || !xq_out || !d_out) return BITLINEAR_ERR_NULL;
    if (!aligned16(gate) || !aligned16(up) || !aligned16(xq_out) || (gain && !aligned16(gain)) ||
        (x_out_bf16 && !aligned16(x_out_bf16)) || (reinterpret_cast<uintptr_t>(d_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(xsum_out) & 3u))
        return BITLINEAR_ERR_ALIGN;
    if (int rc = check_arch()) return rc;
    return cuda_status(launch_quant_act_step(BITLINEAR_X_RELU2, gate, up, x_out_bf16, 0, 0, static_cast<const __nv_bfloat16*>(gain),
                                             rms_eps, M, F, xq_out, d_out, xsum_out, static_cast<cudaStream_t>(stream)));
}

int bitlinear_matmul_q(const int8_t* xq, const float* d, const int32_t* xsum, const void* packed, const float* s_w,
                       int M, int N, int K, void* y_out, int y_dtype, int32_t* acc_out, int path, void* ws,
                       size_t ws_bytes, void* stream) {
    if (y_dtype != BITLINEAR_F32 && y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (path < BITLINEAR_PATH_AUTO || path > BITLINEAR_PATH_GEMM) return BITLINEAR_ERR_DTYPE;
    if (M < 0 || !shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    const bool gemm = use_gemm(M, N, path);
    if (gemm && (N % 128) != 0) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!xq || !d || !xsum || !packed || !s_w || !y_out) return BITLINEAR_ERR_NULL;
    if (!aligned16(xq) || !aligned16(packed) || !aligned16(y_out) || (acc_out && !aligned16(acc_out)) ||
        (reinterpret_cast<uintptr_t>(d) & 3u) || (reinterpret_cast<uintptr_t>(xsum) & 3u) ||
        (reinterpret_cast<uintptr_t>(s_w) & 3u))
        return BITLINEAR_ERR_ALIGN;
    const size_t need = bitlinear_matmul_workspace_bytes(M, N, K, path);
    if (need > 0 && (!ws || ws_bytes < need || !aligned16(ws))) return BITLINEAR_ERR_WORKSPACE;
    if (int rc = check_arch()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!gemm)
        return cuda_status(launch_gemv(xq, d, xsum, static_cast<const uint32_t*>(packed), s_w, M, N, K, y_out, y_dtype,
                                       acc_out, st));
    uint8_t* codes = static_cast<uint8_t*>(ws);
    // where the SMs pair up, the CTA-pair kernel reads the packed weights directly and expands them in shared memory
    if (gemm_pairs_available())
        return gemm_tcgen05_packed(xq, d, xsum, packed, s_w, M, N, K, y_out, y_dtype, acc_out,
                                   codes + align_up(gemm_codes_bytes(N, K), 256), st);
    cudaError_t e = launch_unpack_codes_u8(static_cast<const uint32_t*>(packed), N, K, codes, st);
    if (e != cudaSuccess) return BITLINEAR_ERR_CUDA;
    return gemm_tcgen05(xq, d, xsum, codes, s_w, M, N, K, y_out, y_dtype, acc_out, st);
}

int bitlinear_forward(const void* x_bf16, const void* gain, float rms_eps, const void* packed, const float* s_w, int M,
                      int N, int K, void* y_out, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    if (y_dtype != BITLINEAR_F32 && y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (M < 0 || !shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!x_bf16 || !packed || !s_w || !y_out) return BITLINEAR_ERR_NULL;
    const size_t mm_bytes = bitlinear_matmul_workspace_bytes(M, N, K, BITLINEAR_PATH_AUTO);
    const ForwardWorkspace w = forward_workspace(M, N, K, mm_bytes);
    if (!ws || ws_bytes < w.total || !aligned16(ws)) return BITLINEAR_ERR_WORKSPACE;
    char* base = static_cast<char*>(ws);
    int8_t* xq = reinterpret_cast<int8_t*>(base + w.xq_off);
    float* d = reinterpret_cast<float*>(base + w.d_off);
    int32_t* xsum = reinterpret_cast<int32_t*>(base + w.xsum_off);
    // one token: a single launch that fetches its weights while it quantises the row (decode_level.cu); the same
    // arithmetic as the two launches below, bit for bit
    int sm_count = 0;
    if (M == 1 && aligned16(x_bf16) && aligned16(packed) && aligned16(y_out) && (!gain || aligned16(gain)) &&
        !(reinterpret_cast<uintptr_t>(s_w) & 3u) && check_arch() == BITLINEAR_OK && device_sm_count(&sm_count) == BITLINEAR_OK &&
        decode_level_fits(1, N / kTileRows, K, sm_count)) {
        LevelParams P = {};
        P.count = 1;
        P.prob[0].packed = static_cast<const uint8_t*>(packed); P.prob[0].s_w = s_w; P.prob[0].y = y_out;
        P.prob[0].acc_out = nullptr; P.prob[0].N = N; P.prob[0].y_dtype = y_dtype;
        P.x = x_bf16; P.op.op = BITLINEAR_X_PLAIN;
        P.gain = static_cast<const __nv_bfloat16*>(gain); P.eps = rms_eps; P.K = K; P.x_row0 = 0;
        P.total_rb = N / kTileRows;
        P.status_word = device_status_word();
        return decode_level_forward(P, sm_count, static_cast<cudaStream_t>(stream), /*dependent=*/false);
    }
    int rc = bitlinear_quant_act(x_bf16, gain, rms_eps, M, K, xq, d, xsum, stream);
    if (rc != BITLINEAR_OK) return rc;
    return bitlinear_matmul_q(xq, d, xsum, packed, s_w, M, N, K, y_out, y_dtype, nullptr, BITLINEAR_PATH_AUTO,
                              mm_bytes ? base + w.mm_off : nullptr, mm_bytes, stream);
}

size_t bitlinear_forward_master_workspace_bytes(int M, int N, int K) {
    if (!shape_ok(N, K) || M < 0) return 0;
    return align_up(bitlinear_pack_workspace_bytes(N, K), 256) + align_up(bitlinear_packed_bytes(N, K), 256) + 256 /*scale*/ +
           bitlinear_workspace_bytes(M, N, K);
}

int bitlinear_forward_master(const void* x_bf16, const void* gain, float rms_eps, const void* W, int w_dtype, float eps_w,
                             int M, int N, int K, void* y_out, int y_dtype, void* packed_out, float* s_w_out, void* ws,
                             size_t ws_bytes, void* stream) {
    if (y_dtype != BITLINEAR_F32 && y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (w_dtype != BITLINEAR_F32 && w_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (M < 0 || !shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (!W || (M > 0 && (!x_bf16 || !y_out))) return BITLINEAR_ERR_NULL;
    if (!ws || !aligned16(ws) || ws_bytes < bitlinear_forward_master_workspace_bytes(M, N, K)) return BITLINEAR_ERR_WORKSPACE;
    if (packed_out && !aligned16(packed_out)) return BITLINEAR_ERR_ALIGN;
    char* base = static_cast<char*>(ws);
    const size_t pack_ws = align_up(bitlinear_pack_workspace_bytes(N, K), 256), packed_bytes = bitlinear_packed_bytes(N, K);
    void* packed = packed_out ? packed_out : static_cast<void*>(base + pack_ws);
    float* s_w = reinterpret_cast<float*>(base + pack_ws + align_up(packed_bytes, 256));
    if (const int rc = bitlinear_pack_weights(W, w_dtype, N, K, eps_w, packed, s_w, base, pack_ws, stream)) return rc;
    if (s_w_out && cudaMemcpyAsync(s_w_out, s_w, sizeof(float), cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) !=
                       cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (M == 0) return BITLINEAR_OK;
    char* fwd_ws = base + pack_ws + align_up(packed_bytes, 256) + 256;
    return bitlinear_forward(x_bf16, gain, rms_eps, packed, s_w, M, N, K, y_out, y_dtype, fwd_ws,
                             ws_bytes - (size_t)(fwd_ws - base), stream);
}

size_t bitlinear_host_staging_bytes(int M, int N, int K, int y_dtype) {
    if (!shape_ok(N, K) || M < 0) return 0;
    const size_t ysz = (y_dtype == BITLINEAR_BF16) ? 2 : 4;
    return align_up((size_t)M * K * 2, kWsAlign) + align_up((size_t)M * N * ysz, kWsAlign);
}

int bitlinear_forward_host(const void* x_host, const void* gain, float rms_eps, const void* packed, const float* s_w,
                           int M, int N, int K, void* y_host, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    if (y_dtype != BITLINEAR_F32 && y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (M < 0 || !shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (M == 0) return BITLINEAR_OK;
    if (!x_host || !y_host || !packed || !s_w) return BITLINEAR_ERR_NULL;
    const size_t fwd = bitlinear_workspace_bytes(M, N, K);
    const size_t stage = bitlinear_host_staging_bytes(M, N, K, y_dtype);
    if (!ws || ws_bytes < fwd + stage || !aligned16(ws)) return BITLINEAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t ysz = (y_dtype == BITLINEAR_BF16) ? 2 : 4;
    char* x_dev = static_cast<char*>(ws) + fwd;
    char* y_dev = x_dev + align_up((size_t)M * K * 2, kWsAlign);
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    int rc = bitlinear_forward(x_dev, gain, rms_eps, packed, s_w, M, N, K, y_dev, y_dtype, ws, fwd, stream);
    if (rc != BITLINEAR_OK) return rc;
    if (cudaMemcpyAsync(y_host, y_dev, (size_t)M * N * ysz, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

int bitlinear_selftest_wait_timeout(unsigned limit_us, void* stream) {
    if (limit_us == 0 || limit_us > 100000u) return BITLINEAR_ERR_SHAPE;  // 100 ms at most
    if (int rc = check_arch()) return rc;
    int* word = device_status_word();
    if (!word) return BITLINEAR_ERR_CUDA;
    wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>((unsigned long long)limit_us * 1000ull, word);
    return cuda_status(cudaGetLastError());
}

int bitlinear_probe_int8_mma_rate(int n_mma_per_sm, double* ops_out, void* stream) {
    if (n_mma_per_sm < 1 || n_mma_per_sm > 4000000) return BITLINEAR_ERR_SHAPE;  // a few milliseconds at most
    if (int rc = check_arch()) return rc;
    return int8_mma_rate_probe(n_mma_per_sm, ops_out, static_cast<cudaStream_t>(stream));
}

int bitlinear_poll_status(void* stream) {
    if (int rc = check_arch()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* word = device_status_word();
    if (!word) return BITLINEAR_ERR_CUDA;
    int host = 0;
    if (cudaMemcpyAsync(&host, word, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (host != 0) {
        if (cudaMemsetAsync(word, 0, sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        return host == BITLINEAR_ERR_WORKSPACE ? BITLINEAR_ERR_WORKSPACE : BITLINEAR_ERR_TIMEOUT;
    }
    return BITLINEAR_OK;
}

}  // extern "C"
