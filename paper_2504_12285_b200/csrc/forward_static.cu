// BitLinear decode forward for callers that cannot hand the library any scratch memory.
//
// bitlinear_forward needs a workspace (the int8 activations, their scales and code sums) that the
// caller allocates.  Some callers cannot allocate at that point: code that runs after a framework
// has handed all device memory to its own pool, plug-ins that are only given the input and output
// buffers of an operator, real-time loops that forbid allocator calls.  For them the workspace
// lives here, in a fixed array that is part of the library image: every GPU that loads the library
// carries these 256.5 KiB until the process exits, and nothing is ever allocated or freed.
//
// Host code must not pass the array's name to a kernel: on the host that name is only a stand-in
// for the symbol.  The device address is looked up once per device with cudaGetSymbolAddress and
// cached.
#include <mutex>

#include "common.cuh"

namespace bitlinear {

namespace {

constexpr int kStaticMaxTokens = BITLINEAR_STATIC_MAX_TOKENS;
constexpr int kStaticMaxK = BITLINEAR_STATIC_MAX_K;
constexpr size_t kStaticXqBytes = (size_t)kStaticMaxTokens * kStaticMaxK;  // int8 activations
constexpr size_t kStaticDOff = kStaticXqBytes;                              // fp32 scale per token
constexpr size_t kStaticXsumOff = kStaticDOff + 256;                        // int32 code sum per token
constexpr size_t kStaticBytes = kStaticXsumOff + 256;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;

// Device address of g_static_scratch on the current device (looked up on the first call per device).
int static_scratch(unsigned char** out) {
    static std::mutex mu;
    static unsigned char* addr[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        if (major != 10) return BITLINEAR_ERR_ARCH;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = addr[dev];
    return BITLINEAR_OK;
}

}  // namespace

}  // namespace bitlinear

using namespace bitlinear;

extern "C" {

size_t bitlinear_static_scratch_bytes(void) { return kStaticBytes; }

int bitlinear_forward_static(const void* x_bf16, const void* gain, float rms_eps, const void* packed, const float* s_w,
                             int M, int N, int K, void* y_out, int y_dtype, void* stream) {
    if (y_dtype != BITLINEAR_F32 && y_dtype != BITLINEAR_BF16) return BITLINEAR_ERR_DTYPE;
    if (M < 0 || !shape_ok(N, K)) return BITLINEAR_ERR_SHAPE;
    if (M > kStaticMaxTokens || K > kStaticMaxK) return BITLINEAR_ERR_WORKSPACE;  // beyond the built-in scratch
    if (M == 0) return BITLINEAR_OK;
    if (!x_bf16 || !packed || !s_w || !y_out) return BITLINEAR_ERR_NULL;
    if (!aligned16(x_bf16) || !aligned16(packed) || !aligned16(y_out) || (gain && !aligned16(gain)) ||
        (reinterpret_cast<uintptr_t>(s_w) & 3u))
        return BITLINEAR_ERR_ALIGN;
    unsigned char* base = nullptr;
    if (int rc = static_scratch(&base)) return rc;
    int8_t* xq = reinterpret_cast<int8_t*>(base);
    float* d = reinterpret_cast<float*>(base + kStaticDOff);
    int32_t* xsum = reinterpret_cast<int32_t*>(base + kStaticXsumOff);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Both kernels overwrite every scratch element they later read (M rows of K codes, M scales,
    // M sums), so nothing has to be cleared between calls.
    if (launch_quant_act(static_cast<const __nv_bfloat16*>(x_bf16), static_cast<const __nv_bfloat16*>(gain), rms_eps, M,
                         K, xq, d, xsum, st) != cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    if (launch_gemv(xq, d, xsum, static_cast<const uint32_t*>(packed), s_w, M, N, K, y_out, y_dtype, nullptr, st) !=
        cudaSuccess) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    return BITLINEAR_OK;
}

}  // extern "C"
