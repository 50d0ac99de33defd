// resq_project_quantize_static: the online-projection quantizer for callers that must not allocate.
//
// The regular entry point stages the fp32 coefficients C = X·P in a workspace the caller allocates.
// Some callers have no way to get one: a serving process that handed every free byte of the GPU to
// its own cache pool at start-up, a plug-in that runs inside someone else's memory plan, a
// latency-critical loop where cudaMalloc's implicit device-wide synchronisation is not acceptable.
// For them the staging panel lives in a fixed array inside the library image (below); every GPU
// that loads the library carries it until the process exits.
#include "internal.h"

namespace resq {
namespace {

constexpr size_t kStaticBytes = RESQ_STATIC_SCRATCH_BYTES;

// File-scope device array.  In host code this NAME is only a handle for the runtime's symbol table,
// not a device address: it must never be passed to a kernel.  The device address is looked up once
// per device with cudaGetSymbolAddress and that pointer is what the kernels get.
static __device__ __align__(256) unsigned char g_static_panel[kStaticBytes];

// Device address of the panel on the current device (set-up on first use, cached per device).
float* static_panel(cudaError_t* err) {
    static float* cache[64] = {};
    int dev = 0;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= 64) {
        *err = cudaErrorInvalidDevice;
        return nullptr;
    }
    if (!cache[dev]) {
        void* ptr = nullptr;
        *err = cudaGetSymbolAddress(&ptr, g_static_panel);
        if (*err != cudaSuccess) return nullptr;
        cache[dev] = static_cast<float*>(ptr);
    }
    return cache[dev];
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace resq

using namespace resq;

extern "C" int resq_project_quantize_static(const void* X, const void* P, int T, int K, int r, int8_t* x8,
                                            uint8_t* x4, float* s_x8, float* s_x4, int8_t* x4_i8, void* stream) {
    if (T < 1 || K <= 0 || r < 0 || r >= K || r % 32 != 0 || (K - r) % 32 != 0) return RESQ_ERR_SHAPE;
    if (!X || !P || (!x8 && r > 0) || !s_x8 || !s_x4 || (!x4 && !x4_i8)) return RESQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(P) || !aligned16(x8) || !aligned16(x4) || !aligned16(s_x8) ||
        !aligned16(s_x4) || !aligned16(x4_i8))
        return RESQ_ERR_ALIGN;
    // The whole [T][K] fp32 panel must fit the built-in array.
    if (static_cast<size_t>(T) * static_cast<size_t>(K) * sizeof(float) > kStaticBytes) return RESQ_ERR_WORKSPACE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return RESQ_ERR_CUDA;
    if (major != 10) return RESQ_ERR_ARCH;
    cudaError_t err = cudaSuccess;
    float* panel = static_panel(&err);
    if (!panel) return RESQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Nothing in the panel has to start at zero: the projection writes every element of rows [0, T)
    // before the quantizer reads them, so whatever an earlier call left behind is overwritten.
    if (launch_project_gemm(X, P, T, K, panel, st) != cudaSuccess) return RESQ_ERR_CUDA;
    if (launch_split_quantize(panel, true, T, K, r, x8, x4, s_x8, s_x4, false, x4_i8, static_cast<size_t>(K) * 4,
                              st) != cudaSuccess)
        return RESQ_ERR_CUDA;
    return RESQ_OK;
}
