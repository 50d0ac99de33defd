// C ABI of the library: argument validation, workspace carving and dispatch.  No arithmetic here.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {

struct __align__(16) DeviceState {
    int flags;                          // condition bits (kStatusBit*), cleared by resq_device_status
    int reserved;
    unsigned long long wait_limit_ns;   // limit of one bounded wait
};
__device__ DeviceState g_state = {0, 0, 2000000000ull};

// A CTA that waits for a barrier phase nothing will ever complete: the bounded wait runs out, the kernel records
// the condition and returns by itself.  Exercises the path every other kernel takes when a copy never lands.
__global__ void wait_runs_out_kernel(int* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
        abort_flag = 0;
    }
    __syncthreads();
    const bool done = mbar_wait(&bar, 0, &abort_flag, status);  // every thread polls; the first to time out tells the rest
    __syncthreads();
    if (threadIdx.x == 0 && (!done || abort_flag)) atomicOr(status, kStatusBitTimeout);
}

int* device_status_ptr() {
    static int* cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_state) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<int*>(p);
    }
    return cache[dev];
}

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }

void* tensor_map_encode_fn() {
    static void* fn = nullptr;
    if (!fn) {
        cudaDriverEntryPointQueryResult q;
        void* f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = f;
    }
    return fn;
}

namespace {

constexpr int kDecodeMaxT = 16;  // up to here the weight-streaming kernel runs, above it the tile kernel
constexpr int kPanelRows = 4096;  // token rows of fp32 coefficients staged per projection panel

inline size_t align_up(size_t x) { return (x + 255) & ~size_t(255); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int check_shape(int K, int n_out, int r) {
    if (K <= 0 || r < 0 || r >= K || n_out <= 0) return RESQ_ERR_SHAPE;  // r == 0: uniform INT4 (Section 4.3, down_proj)
    if (r % 32 != 0 || (K - r) % 32 != 0 || n_out % 8 != 0) return RESQ_ERR_SHAPE;
    return RESQ_OK;
}
int check_desc(const resq_layer_desc_t* d) {
    if (!d) return RESQ_ERR_NULL;
    if (d->w_scale_dtype != RESQ_SCALE_FP32 && d->w_scale_dtype != RESQ_SCALE_FP16) return RESQ_ERR_SHAPE;
    return check_shape(d->K, d->n_out, d->r);
}
int check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RESQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return RESQ_ERR_CUDA;
    return major == 10 ? RESQ_OK : RESQ_ERR_ARCH;
}

// Carving of the caller's workspace.  Every entry point uses the same map (and its own subset).
struct Workspace {
    size_t x8, x4, sx8, sx4, zx8, zx4, x4e, w4e, panel, total;  // panel: fp32 coefficients + the GEMM's split scratch
};
Workspace carve(int K, int n_out, int r, int T, bool has_P, bool has_w4_i8) {
    Workspace w{};
    const size_t K4 = static_cast<size_t>(K - r), Tz = static_cast<size_t>(T), N = static_cast<size_t>(n_out);
    size_t o = 0;
    w.x8 = o;  o += align_up(Tz * r);
    w.x4 = o;  o += align_up(Tz * K4 / 2);
    w.sx8 = o; o += align_up(Tz * 4);
    w.sx4 = o; o += align_up(Tz * 4);
    w.zx8 = o; o += align_up(Tz * 4);  // zero-points (asymmetric activations only)
    w.zx4 = o; o += align_up(Tz * 4);
    const bool tiles = T > kDecodeMaxT;
    w.x4e = o;    o += tiles ? align_up(Tz * K4) : 0;
    w.w4e = o;    o += (tiles && !has_w4_i8) ? align_up(N * K4) : 0;
    w.panel = o;  o += has_P ? align_up(static_cast<size_t>(T < kPanelRows ? T : kPanelRows) * K * 4) + align_up(project_split_scratch_bytes()) : 0;
    w.total = o;
    return w;
}

cudaError_t g_last_cuda_error = cudaSuccess;  // what the latest RESQ_ERR_CUDA stood for
int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return RESQ_OK;
    g_last_cuda_error = e;
    return RESQ_ERR_CUDA;
}

}  // namespace
}  // namespace resq

using namespace resq;

extern "C" {

size_t resq_w8_bytes(const resq_layer_desc_t* d) {
    return check_desc(d) ? 0 : static_cast<size_t>(d->n_out) * d->r;
}
size_t resq_w4_bytes(const resq_layer_desc_t* d) {
    return check_desc(d) ? 0 : static_cast<size_t>(d->n_out) * (d->K - d->r) / 2;
}
size_t resq_w4_i8_bytes(const resq_layer_desc_t* d) {
    return check_desc(d) ? 0 : static_cast<size_t>(d->n_out) * (d->K - d->r);
}
size_t resq_scale_bytes(const resq_layer_desc_t* d) {
    return check_desc(d) ? 0 : static_cast<size_t>(d->n_out) * (d->w_scale_dtype == RESQ_SCALE_FP16 ? 2 : 4);
}

size_t resq_workspace_bytes(const resq_layer_desc_t* d, int T, int has_P, int has_w4_i8) {
    if (check_desc(d) || T < 1) return 0;
    return carve(d->K, d->n_out, d->r, T, has_P != 0, has_w4_i8 != 0).total;
}

int resq_pack_weights(const resq_layer_desc_t* d, const float* W_proj, int8_t* w8, uint8_t* w4, void* s_w8,
                      void* s_w4, int8_t* w4_i8, void* stream) {
    if (int e = check_desc(d)) return e;
    if (!W_proj || (!w8 && d->r > 0) || !w4 || !s_w8 || !s_w4) return RESQ_ERR_NULL;
    if (!aligned16(W_proj) || !aligned16(w8) || !aligned16(w4) || !aligned16(s_w8) || !aligned16(s_w4) ||
        !aligned16(w4_i8))
        return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    return cuda_status(launch_split_quantize(W_proj, true, d->n_out, d->K, d->r, w8, w4, s_w8, s_w4,
                                             d->w_scale_dtype == RESQ_SCALE_FP16, w4_i8,
                                             static_cast<size_t>(d->K) * 4, static_cast<cudaStream_t>(stream)));
}

int resq_pack_weights_gptq(const resq_layer_desc_t* d, const float* W_proj, const float* U_inv, const uint8_t* dead_cols,
                           int8_t* w8, uint8_t* w4, void* s_w8, void* s_w4, int8_t* w4_i8, void* stream) {
    if (int e = check_desc(d)) return e;
    if (!W_proj || !U_inv || (!w8 && d->r > 0) || !w4 || !s_w8 || !s_w4) return RESQ_ERR_NULL;
    if (!aligned16(W_proj) || !aligned16(U_inv) || !aligned16(w8) || !aligned16(w4) || !aligned16(s_w8) ||
        !aligned16(s_w4) || !aligned16(w4_i8))
        return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    const cudaError_t e = launch_pack_gptq(W_proj, U_inv, dead_cols, d->n_out, d->K, d->r, w8, w4, s_w8, s_w4,
                                           d->w_scale_dtype == RESQ_SCALE_FP16, w4_i8, static_cast<cudaStream_t>(stream));
    return e == cudaErrorNotSupported ? RESQ_ERR_SHAPE : cuda_status(e);
}

size_t resq_pack_projected_workspace_bytes(const resq_layer_desc_t* d) {
    if (check_desc(d)) return 0;
    return align_up(static_cast<size_t>(d->n_out < kPanelRows ? d->n_out : kPanelRows) * d->K * 4);
}

int resq_pack_weights_projected(const resq_layer_desc_t* d, const void* W_raw, const void* U, int8_t* w8, uint8_t* w4,
                                void* s_w8, void* s_w4, int8_t* w4_i8, void* workspace, size_t workspace_bytes,
                                void* stream) {
    if (int e = check_desc(d)) return e;
    if (!W_raw || !U || (!w8 && d->r > 0) || !w4 || !s_w8 || !s_w4) return RESQ_ERR_NULL;
    if (!aligned16(W_raw) || !aligned16(U) || !aligned16(w8) || !aligned16(w4) || !aligned16(s_w8) ||
        !aligned16(s_w4) || !aligned16(w4_i8) || !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    if (!workspace || workspace_bytes < resq_pack_projected_workspace_bytes(d)) return RESQ_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* panel = static_cast<float*>(workspace);
    const size_t K = static_cast<size_t>(d->K), K4 = static_cast<size_t>(d->K - d->r);
    const size_t sb = d->w_scale_dtype == RESQ_SCALE_FP16 ? 2 : 4;
    for (int n0 = 0; n0 < d->n_out; n0 += kPanelRows) {
        const int rows = d->n_out - n0 < kPanelRows ? d->n_out - n0 : kPanelRows;
        const char* Wp = static_cast<const char*>(W_raw) + static_cast<size_t>(n0) * K * 2;
        if (cudaError_t e = launch_project_gemm(Wp, U, rows, d->K, panel, st); e != cudaSuccess) return cuda_status(e);
        if (cudaError_t e = launch_split_quantize(
                panel, true, rows, d->K, d->r, w8 ? w8 + static_cast<size_t>(n0) * d->r : nullptr, w4 + n0 * K4 / 2,
                static_cast<char*>(s_w8) + n0 * sb, static_cast<char*>(s_w4) + n0 * sb, sb == 2,
                w4_i8 ? w4_i8 + n0 * K4 : nullptr, K * 4, st);
            e != cudaSuccess)
            return cuda_status(e);
    }
    return RESQ_OK;
}

int resq_project_quantize(const void* X, const void* P, int T, int K, int r, int8_t* x8, uint8_t* x4, float* s_x8,
                          float* s_x4, int8_t* x4_i8, void* workspace, size_t workspace_bytes, void* stream) {
    if (T < 1) return RESQ_ERR_SHAPE;
    if (int e = check_shape(K, 8, r)) return e;
    if (!X || (!x8 && r > 0) || !s_x8 || !s_x4 || (!x4 && !x4_i8)) return RESQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(P) || !aligned16(x8) || !aligned16(x4) || !aligned16(s_x8) ||
        !aligned16(s_x4) || !aligned16(x4_i8) || !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!P)
        return cuda_status(launch_split_quantize(X, false, T, K, r, x8, x4, s_x8, s_x4, false, x4_i8,
                                                 static_cast<size_t>(K) * 2, st));
    // Online projection: panels of token rows, fp32 coefficients staged in the workspace.
    const int rows_max = T < kPanelRows ? T : kPanelRows;
    const size_t need = align_up(static_cast<size_t>(rows_max) * K * 4);
    if (!workspace || workspace_bytes < need) return RESQ_ERR_WORKSPACE;
    float* panel = static_cast<float*>(workspace);
    // what the workspace holds beyond the panel serves the GEMM's last-round split (resq_workspace_bytes includes it)
    const bool has_scratch = workspace_bytes >= need + project_split_scratch_bytes();
    void* scratch = has_scratch ? static_cast<char*>(workspace) + need : nullptr;
    const size_t K4 = static_cast<size_t>(K - r);
    for (int t0 = 0; t0 < T; t0 += kPanelRows) {
        const int rows = T - t0 < kPanelRows ? T - t0 : kPanelRows;
        const char* Xp = static_cast<const char*>(X) + static_cast<size_t>(t0) * K * 2;
        if (cudaError_t e = launch_project_gemm(Xp, P, rows, K, panel, st, scratch, project_split_scratch_bytes());
            e != cudaSuccess)
            return cuda_status(e);
        if (cudaError_t e = launch_split_quantize(panel, true, rows, K, r, x8 + static_cast<size_t>(t0) * r,
                                                  x4 ? x4 + static_cast<size_t>(t0) * K4 / 2 : nullptr, s_x8 + t0,
                                                  s_x4 + t0, false,
                                                  x4_i8 ? x4_i8 + static_cast<size_t>(t0) * K4 : nullptr,
                                                  static_cast<size_t>(K) * 4, st, true);
            e != cudaSuccess)
            return cuda_status(e);
    }
    return RESQ_OK;
}

int resq_hadamard_quantize(const void* X, int T, int K, int r, int8_t* x8, uint8_t* x4, float* s_x8, float* s_x4,
                           int8_t* x4_i8, void* stream) {
    if (T < 1) return RESQ_ERR_SHAPE;
    if (int e = check_shape(K, 8, r)) return e;
    if (!X || (!x8 && r > 0) || !s_x8 || !s_x4 || (!x4 && !x4_i8)) return RESQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(x8) || !aligned16(x4) || !aligned16(s_x8) || !aligned16(s_x4) || !aligned16(x4_i8))
        return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    const cudaError_t e = launch_hadamard_quantize(X, T, K, r, x8, x4, s_x8, s_x4, x4_i8, static_cast<cudaStream_t>(stream));
    return e == cudaErrorNotSupported ? RESQ_ERR_SHAPE : cuda_status(e);
}

size_t resq_project_workspace_bytes(void) { return project_split_scratch_bytes(); }

int resq_project(const void* X, const void* P, int T, int K, float* C, void* workspace, size_t workspace_bytes,
                 void* stream) {
    if (T < 1 || K <= 0 || K % 8 != 0) return RESQ_ERR_SHAPE;
    if (!X || !P || !C) return RESQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(P) || !aligned16(C) || !aligned16(workspace)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    const bool has_scratch = workspace && workspace_bytes >= project_split_scratch_bytes();
    return cuda_status(launch_project_gemm(X, P, T, K, C, static_cast<cudaStream_t>(stream),
                                           has_scratch ? workspace : nullptr, has_scratch ? workspace_bytes : 0));
}

static int mixed_gemm_impl(const resq_layer_desc_t* d, int T, const int8_t* x8, const uint8_t* x4,
                           const int8_t* x4e_ready, const float* s_x8, const float* s_x4, const resq_weights_t* W,
                           void* Y, int y_dtype, int32_t* dbg8, int32_t* dbg4, char* ws, const Workspace& map,
                           cudaStream_t st) {
    const bool fp16 = d->w_scale_dtype == RESQ_SCALE_FP16;
    const size_t K4 = static_cast<size_t>(d->K - d->r);
    if (T <= kDecodeMaxT) {
        const cudaError_t e = launch_mixed_gemm_stream(T, d->n_out, d->K, d->r, x8, x4, s_x8, s_x4, W->w8, W->w4,
                                                       W->s_w8, W->s_w4, fp16, Y, y_dtype, dbg8, dbg4, st);
        if (e != cudaErrorNotSupported) return cuda_status(e);
        // Rows too wide to stage 9-16 tokens of activation codes beside the weight rings run as two launches of at
        // most 8 tokens (the weights are streamed twice; only reduction lengths beyond ~24k reach this).
        if (T <= 8) return RESQ_ERR_SHAPE;
        const size_t ysz = y_dtype == RESQ_Y_BF16 ? 2 : 4;
        for (int t0 = 0; t0 < T; t0 += 8) {
            const int rows = T - t0 < 8 ? T - t0 : 8;
            const cudaError_t e2 = launch_mixed_gemm_stream(
                rows, d->n_out, d->K, d->r, x8 ? x8 + static_cast<size_t>(t0) * d->r : nullptr,
                x4 + static_cast<size_t>(t0) * (K4 / 2), s_x8 + t0, s_x4 + t0, W->w8, W->w4, W->s_w8, W->s_w4, fp16,
                static_cast<char*>(Y) + static_cast<size_t>(t0) * d->n_out * ysz, y_dtype,
                dbg8 ? dbg8 + static_cast<size_t>(t0) * d->n_out : nullptr,
                dbg4 ? dbg4 + static_cast<size_t>(t0) * d->n_out : nullptr, st);
            if (e2 == cudaErrorNotSupported) return RESQ_ERR_SHAPE;
            if (e2 != cudaSuccess) return cuda_status(e2);
        }
        return RESQ_OK;
    }
    const int8_t* x4e = x4e_ready;
    if (!x4e) {
        int8_t* buf = reinterpret_cast<int8_t*>(ws + map.x4e);
        if (cudaError_t e = launch_unpack_int4(x4, buf, T, K4, st); e != cudaSuccess) return cuda_status(e);
        x4e = buf;
    }
    const int8_t* w4e = W->w4_i8;
    if (!w4e) {
        int8_t* buf = reinterpret_cast<int8_t*>(ws + map.w4e);
        if (cudaError_t e = launch_unpack_int4(W->w4, buf, d->n_out, K4, st); e != cudaSuccess) return cuda_status(e);
        w4e = buf;
    }
    return cuda_status(launch_mixed_gemm_tiles(T, d->n_out, d->K, d->r, x8, x4e, s_x8, s_x4, W->w8, w4e, W->s_w8,
                                               W->s_w4, fp16, Y, y_dtype, dbg8, dbg4, st));
}

static int check_weights(const resq_weights_t* W, int r) {
    if (!W || (!W->w8 && r > 0) || !W->w4 || !W->s_w8 || !W->s_w4) return RESQ_ERR_NULL;
    if (!aligned16(W->w8) || !aligned16(W->w4) || !aligned16(W->s_w8) || !aligned16(W->s_w4) ||
        !aligned16(W->w4_i8))
        return RESQ_ERR_ALIGN;
    return RESQ_OK;
}

int resq_mixed_gemm(const resq_layer_desc_t* d, int T, const int8_t* x8, const uint8_t* x4, const int8_t* x4_i8,
                    const float* s_x8, const float* s_x4, const resq_weights_t* W, void* Y, int y_dtype,
                    int32_t* dbg_acc8, int32_t* dbg_acc4, void* workspace, size_t workspace_bytes, void* stream) {
    if (int e = check_desc(d)) return e;
    if (T < 1 || (y_dtype != RESQ_Y_BF16 && y_dtype != RESQ_Y_FP32)) return RESQ_ERR_SHAPE;
    if ((!x8 && d->r > 0) || !s_x8 || !s_x4 || !Y) return RESQ_ERR_NULL;
    if (!x4 && (!x4_i8 || T <= kDecodeMaxT)) return RESQ_ERR_NULL;
    if ((dbg_acc8 == nullptr) != (dbg_acc4 == nullptr)) return RESQ_ERR_NULL;
    if (int e = check_weights(W, d->r)) return e;
    if (!aligned16(x8) || !aligned16(x4) || !aligned16(x4_i8) || !aligned16(s_x8) || !aligned16(s_x4) ||
        !aligned16(Y) || !aligned16(dbg_acc8) || !aligned16(dbg_acc4) || !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    const Workspace map = carve(d->K, d->n_out, d->r, T, false, W->w4_i8 != nullptr);
    if (!workspace || workspace_bytes < map.total) return RESQ_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    return mixed_gemm_impl(d, T, x8, x4, x4_i8, s_x8, s_x4, W, Y, y_dtype, dbg_acc8, dbg_acc4,
                           static_cast<char*>(workspace), map, static_cast<cudaStream_t>(stream));
}

int resq_linear(const resq_layer_desc_t* d, int T, const void* X, const void* P, const resq_weights_t* W, void* Y,
                int y_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    if (int e = check_desc(d)) return e;
    if (T < 1 || (y_dtype != RESQ_Y_BF16 && y_dtype != RESQ_Y_FP32)) return RESQ_ERR_SHAPE;
    if (!X || !Y) return RESQ_ERR_NULL;
    if (int e = check_weights(W, d->r)) return e;
    if (!aligned16(X) || !aligned16(P) || !aligned16(Y) || !aligned16(workspace)) return RESQ_ERR_ALIGN;
    const Workspace map = carve(d->K, d->n_out, d->r, T, P != nullptr, W->w4_i8 != nullptr);
    if (!workspace || workspace_bytes < map.total) return RESQ_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    char* ws = static_cast<char*>(workspace);
    int8_t* x8 = reinterpret_cast<int8_t*>(ws + map.x8);
    uint8_t* x4 = reinterpret_cast<uint8_t*>(ws + map.x4);
    float* s_x8 = reinterpret_cast<float*>(ws + map.sx8);
    float* s_x4 = reinterpret_cast<float*>(ws + map.sx4);
    const bool tiles = T > kDecodeMaxT;
    int8_t* x4e = tiles ? reinterpret_cast<int8_t*>(ws + map.x4e) : nullptr;
    // The tile kernel consumes the one-code-per-byte layout, the streaming kernel the packed one.
    if (int e = resq_project_quantize(X, P, T, d->K, d->r, x8, tiles ? nullptr : x4, s_x8, s_x4, x4e, ws + map.panel,
                                      workspace_bytes - map.panel, stream))
        return e;
    return mixed_gemm_impl(d, T, x8, x4, x4e, s_x8, s_x4, W, Y, y_dtype, nullptr, nullptr, ws, map,
                           static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------- asymmetric activations (Section 5.1)
int resq_weight_row_sums(const resq_layer_desc_t* d, const resq_weights_t* W, int32_t* wsum8, int32_t* wsum4,
                         void* stream) {
    if (int e = check_desc(d)) return e;
    if (int e = check_weights(W, d->r)) return e;
    if (!wsum8 || !wsum4) return RESQ_ERR_NULL;
    if (!aligned16(wsum8) || !aligned16(wsum4)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    return cuda_status(launch_weight_row_sums(W->w8, W->w4, d->n_out, d->K, d->r, wsum8, wsum4,
                                              static_cast<cudaStream_t>(stream)));
}

int resq_project_quantize_asym(const void* X, const void* P, int T, int K, int r, uint8_t* u8, uint8_t* u4,
                               float* s_x8, float* s_x4, float* z_x8, float* z_x4, uint8_t* u4_u8, void* workspace,
                               size_t workspace_bytes, void* stream) {
    if (T < 1) return RESQ_ERR_SHAPE;
    if (int e = check_shape(K, 8, r)) return e;
    if (!X || (!u8 && r > 0) || !s_x8 || !s_x4 || !z_x8 || !z_x4 || (!u4 && !u4_u8)) return RESQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(P) || !aligned16(u8) || !aligned16(u4) || !aligned16(s_x8) || !aligned16(s_x4) ||
        !aligned16(z_x8) || !aligned16(z_x4) || !aligned16(u4_u8) || !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    if (static_cast<size_t>(K) * 4 > 200u * 1024u) return RESQ_ERR_SHAPE;  // row staging limit of this quantizer
    if (int e = check_arch()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!P)
        return cuda_status(launch_split_quantize_asym(X, false, T, K, r, u8, u4, s_x8, s_x4, z_x8, z_x4, u4_u8,
                                                      static_cast<size_t>(K) * 2, st));
    const int rows_max = T < kPanelRows ? T : kPanelRows;
    const size_t need = align_up(static_cast<size_t>(rows_max) * K * 4);
    if (!workspace || workspace_bytes < need) return RESQ_ERR_WORKSPACE;
    float* panel = static_cast<float*>(workspace);
    const bool has_scratch = workspace_bytes >= need + project_split_scratch_bytes();
    void* scratch = has_scratch ? static_cast<char*>(workspace) + need : nullptr;
    const size_t K4 = static_cast<size_t>(K - r);
    for (int t0 = 0; t0 < T; t0 += kPanelRows) {
        const int rows = T - t0 < kPanelRows ? T - t0 : kPanelRows;
        const char* Xp = static_cast<const char*>(X) + static_cast<size_t>(t0) * K * 2;
        if (cudaError_t e = launch_project_gemm(Xp, P, rows, K, panel, st, scratch, project_split_scratch_bytes());
            e != cudaSuccess)
            return cuda_status(e);
        if (cudaError_t e = launch_split_quantize_asym(panel, true, rows, K, r, u8 + static_cast<size_t>(t0) * r,
                                                       u4 ? u4 + static_cast<size_t>(t0) * K4 / 2 : nullptr, s_x8 + t0,
                                                       s_x4 + t0, z_x8 + t0, z_x4 + t0,
                                                       u4_u8 ? u4_u8 + static_cast<size_t>(t0) * K4 : nullptr,
                                                       static_cast<size_t>(K) * 4, st);
            e != cudaSuccess)
            return cuda_status(e);
    }
    return RESQ_OK;
}

static int mixed_gemm_asym_impl(const resq_layer_desc_t* d, int T, const uint8_t* u8, const uint8_t* u4,
                                const uint8_t* u4e_ready, const float* s_x8, const float* s_x4, const float* z_x8,
                                const float* z_x4, const resq_weights_t* W, const int32_t* wsum8, const int32_t* wsum4,
                                void* Y, int y_dtype, int32_t* dbg8, int32_t* dbg4, char* ws, const Workspace& map,
                                cudaStream_t st) {
    const size_t K4 = static_cast<size_t>(d->K - d->r);
    if (T <= kDecodeMaxT && u4) {
        // Few tokens and packed codes at hand: the weight-streaming kernel (falls through if it cannot stage them).
        const cudaError_t e = launch_mixed_gemm_stream(T, d->n_out, d->K, d->r, reinterpret_cast<const int8_t*>(u8), u4,
                                                       s_x8, s_x4, W->w8, W->w4, W->s_w8, W->s_w4,
                                                       d->w_scale_dtype == RESQ_SCALE_FP16, Y, y_dtype, dbg8, dbg4, st,
                                                       z_x8, z_x4, wsum8, wsum4);
        if (e != cudaErrorNotSupported) return cuda_status(e);
        if (T > 8) {
            // Rows too wide to stage 9-16 tokens beside the weight rings: two launches of at most 8 tokens, as in the
            // symmetric path (the tile kernel below would read one byte per INT4 weight for these few rows).
            const size_t ysz = y_dtype == RESQ_Y_BF16 ? 2 : 4;
            bool done = true;
            for (int t0 = 0; t0 < T && done; t0 += 8) {
                const int rows = T - t0 < 8 ? T - t0 : 8;
                const cudaError_t e2 = launch_mixed_gemm_stream(
                    rows, d->n_out, d->K, d->r, u8 ? reinterpret_cast<const int8_t*>(u8) + static_cast<size_t>(t0) * d->r : nullptr,
                    u4 + static_cast<size_t>(t0) * (K4 / 2), s_x8 + t0, s_x4 + t0, W->w8, W->w4, W->s_w8, W->s_w4,
                    d->w_scale_dtype == RESQ_SCALE_FP16, static_cast<char*>(Y) + static_cast<size_t>(t0) * d->n_out * ysz,
                    y_dtype, dbg8 ? dbg8 + static_cast<size_t>(t0) * d->n_out : nullptr,
                    dbg4 ? dbg4 + static_cast<size_t>(t0) * d->n_out : nullptr, st, z_x8 + t0, z_x4 + t0, wsum8, wsum4);
                if (e2 == cudaErrorNotSupported) {
                    if (t0 > 0) return RESQ_ERR_SHAPE;  // cannot happen: the plan does not depend on the row offset
                    done = false;
                } else if (e2 != cudaSuccess) {
                    return cuda_status(e2);
                }
            }
            if (done) return RESQ_OK;
        }
    }
    const int8_t* x4e = reinterpret_cast<const int8_t*>(u4e_ready);
    if (!x4e) {
        int8_t* buf = reinterpret_cast<int8_t*>(ws + map.x4e);
        if (cudaError_t e = launch_unpack_int4(u4, buf, T, K4, st, true); e != cudaSuccess) return cuda_status(e);
        x4e = buf;
    }
    const int8_t* w4e = W->w4_i8;
    if (!w4e) {
        int8_t* buf = reinterpret_cast<int8_t*>(ws + map.w4e);
        if (cudaError_t e = launch_unpack_int4(W->w4, buf, d->n_out, K4, st); e != cudaSuccess) return cuda_status(e);
        w4e = buf;
    }
    return cuda_status(launch_mixed_gemm_tiles(T, d->n_out, d->K, d->r, reinterpret_cast<const int8_t*>(u8), x4e, s_x8,
                                               s_x4, W->w8, w4e, W->s_w8, W->s_w4,
                                               d->w_scale_dtype == RESQ_SCALE_FP16, Y, y_dtype, dbg8, dbg4, st, z_x8,
                                               z_x4, wsum8, wsum4));
}

// The tile kernel serves every T here, so the workspace is carved as for T > 16.
static Workspace carve_asym(const resq_layer_desc_t* d, int T, bool has_P, bool has_w4_i8) {
    return carve(d->K, d->n_out, d->r, T > kDecodeMaxT ? T : kDecodeMaxT + 1, has_P, has_w4_i8);
}

int resq_mixed_gemm_asym(const resq_layer_desc_t* d, int T, const uint8_t* u8, const uint8_t* u4, const uint8_t* u4_u8,
                         const float* s_x8, const float* s_x4, const float* z_x8, const float* z_x4,
                         const resq_weights_t* W, const int32_t* wsum8, const int32_t* wsum4, void* Y, int y_dtype,
                         int32_t* dbg_acc8, int32_t* dbg_acc4, void* workspace, size_t workspace_bytes, void* stream) {
    if (int e = check_desc(d)) return e;
    if (T < 1 || (y_dtype != RESQ_Y_BF16 && y_dtype != RESQ_Y_FP32)) return RESQ_ERR_SHAPE;
    if ((!u8 && d->r > 0) || !s_x8 || !s_x4 || !z_x8 || !z_x4 || !wsum8 || !wsum4 || !Y || (!u4 && !u4_u8)) return RESQ_ERR_NULL;
    if ((dbg_acc8 == nullptr) != (dbg_acc4 == nullptr)) return RESQ_ERR_NULL;
    if (int e = check_weights(W, d->r)) return e;
    if (!aligned16(u8) || !aligned16(u4) || !aligned16(u4_u8) || !aligned16(s_x8) || !aligned16(s_x4) ||
        !aligned16(z_x8) || !aligned16(z_x4) || !aligned16(wsum8) || !aligned16(wsum4) || !aligned16(Y) ||
        !aligned16(dbg_acc8) || !aligned16(dbg_acc4) || !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    const Workspace map = carve_asym(d, T, false, W->w4_i8 != nullptr);
    if (!workspace || workspace_bytes < map.total) return RESQ_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    return mixed_gemm_asym_impl(d, T, u8, u4, u4_u8, s_x8, s_x4, z_x8, z_x4, W, wsum8, wsum4, Y, y_dtype, dbg_acc8,
                                dbg_acc4, static_cast<char*>(workspace), map, static_cast<cudaStream_t>(stream));
}

int resq_linear_asym(const resq_layer_desc_t* d, int T, const void* X, const void* P, const resq_weights_t* W,
                     const int32_t* wsum8, const int32_t* wsum4, void* Y, int y_dtype, void* workspace,
                     size_t workspace_bytes, void* stream) {
    if (int e = check_desc(d)) return e;
    if (T < 1 || (y_dtype != RESQ_Y_BF16 && y_dtype != RESQ_Y_FP32)) return RESQ_ERR_SHAPE;
    if (!X || !Y || !wsum8 || !wsum4) return RESQ_ERR_NULL;
    if (int e = check_weights(W, d->r)) return e;
    if (!aligned16(X) || !aligned16(P) || !aligned16(Y) || !aligned16(wsum8) || !aligned16(wsum4) ||
        !aligned16(workspace))
        return RESQ_ERR_ALIGN;
    const Workspace map = carve_asym(d, T, P != nullptr, W->w4_i8 != nullptr);
    if (!workspace || workspace_bytes < map.total) return RESQ_ERR_WORKSPACE;
    if (int e = check_arch()) return e;
    char* ws = static_cast<char*>(workspace);
    uint8_t* u8 = reinterpret_cast<uint8_t*>(ws + map.x8);
    uint8_t* u4e = reinterpret_cast<uint8_t*>(ws + map.x4e);
    float* s_x8 = reinterpret_cast<float*>(ws + map.sx8);
    float* s_x4 = reinterpret_cast<float*>(ws + map.sx4);
    float* z_x8 = reinterpret_cast<float*>(ws + map.zx8);
    float* z_x4 = reinterpret_cast<float*>(ws + map.zx4);
    // Few tokens: the streaming kernel wants the packed codes as well (the tile kernel, its fallback, the others).
    uint8_t* u4 = T <= kDecodeMaxT ? reinterpret_cast<uint8_t*>(ws + map.x4) : nullptr;
    if (int e = resq_project_quantize_asym(X, P, T, d->K, d->r, u8, u4, s_x8, s_x4, z_x8, z_x4, u4e, ws + map.panel,
                                           workspace_bytes - map.panel, stream))
        return e;
    return mixed_gemm_asym_impl(d, T, u8, u4, u4e, s_x8, s_x4, z_x8, z_x4, W, wsum8, wsum4, Y, y_dtype, nullptr,
                                nullptr, ws, map, static_cast<cudaStream_t>(stream));
}

size_t resq_workspace_bytes_asym(const resq_layer_desc_t* d, int T, int has_P, int has_w4_i8) {
    if (check_desc(d) || T < 1) return 0;
    return carve_asym(d, T, has_P != 0, has_w4_i8 != 0).total;
}

int resq_unpack_int4(const uint8_t* packed, int8_t* out, size_t rows, size_t cols, void* stream) {
    if (!packed || !out) return RESQ_ERR_NULL;
    if (cols % 8 != 0) return RESQ_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(out)) return RESQ_ERR_ALIGN;
    return cuda_status(launch_unpack_int4(packed, out, rows, cols, static_cast<cudaStream_t>(stream)));
}

int resq_set_option(int option, int value) {
    if (option == RESQ_OPT_DECODE_EARLY_WEIGHTS) {
        set_decode_early_weights(value);
        return RESQ_OK;
    }
    if (option == RESQ_OPT_WAIT_LIMIT_US) {
        if (value < 1) return RESQ_ERR_SHAPE;
        int* p = device_status_ptr();
        if (!p) return RESQ_ERR_CUDA;
        const unsigned long long ns = static_cast<unsigned long long>(value) * 1000ull;
        return cuda_status(cudaMemcpy(p + 2, &ns, sizeof(ns), cudaMemcpyHostToDevice));
    }
    return RESQ_ERR_SHAPE;
}

int resq_device_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return RESQ_ERR_CUDA;
    int* p = device_status_ptr();
    if (!p) return RESQ_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RESQ_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        cudaMemcpy(p, &zero, sizeof(int), cudaMemcpyHostToDevice);
        return (v & kStatusBitTimeout) ? RESQ_ERR_TIMEOUT : RESQ_ERR_INDEX;  // one bit per condition
    }
    return RESQ_OK;
}

int resq_selftest_wait_runs_out(void* stream) {
    if (int e = check_arch()) return e;
    int* p = device_status_ptr();
    if (!p) return RESQ_ERR_CUDA;
    count_launch();
    wait_runs_out_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cuda_status(cudaGetLastError());
}

// ---- attention-block path (resq_kv.h) ----
size_t resq_kv_block_bytes(int d_head) {
    return d_head == 128 ? RESQ_KV_BLOCK_BYTES : d_head == 64 ? kv64_block_bytes() : 0;
}

size_t resq_kv_cache_bytes(int n_seqs, int n_kv_heads, int d_head, int capacity) {
    if (n_seqs < 1 || n_kv_heads < 1 || (d_head != 128 && d_head != 64) || capacity < RESQ_KV_BLOCK ||
        capacity % RESQ_KV_BLOCK != 0)
        return 0;
    return static_cast<size_t>(n_seqs) * n_kv_heads * (capacity / RESQ_KV_BLOCK) * resq_kv_block_bytes(d_head);
}

static int check_cache(const resq_kv_cache_t* c) {
    if (!c) return RESQ_ERR_NULL;
    if (resq_kv_cache_bytes(c->n_seqs, c->n_kv_heads, c->d_head, c->capacity) == 0) return RESQ_ERR_SHAPE;
    if (!c->data) return RESQ_ERR_NULL;
    return aligned16(c->data) ? RESQ_OK : RESQ_ERR_ALIGN;
}

int resq_uc_quantize(const float* W_C, int d_head, int8_t* wq, float* s_u, void* stream) {
    if (d_head != 128 && d_head != 64) return RESQ_ERR_SHAPE;
    if (!W_C || !wq || !s_u) return RESQ_ERR_NULL;
    if (!aligned16(W_C) || !aligned16(wq) || !aligned16(s_u)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    if (d_head == 64) return cuda_status(launch_uc_quantize64(W_C, wq, s_u, static_cast<cudaStream_t>(stream)));
    return cuda_status(launch_uc_quantize(W_C, wq, s_u, static_cast<cudaStream_t>(stream)));
}

int resq_query_project(const void* q, int64_t rows, int d_head, const int8_t* wq, const float* s_u, void* q_out,
                       void* stream) {
    if ((d_head != 128 && d_head != 64) || rows < 0) return RESQ_ERR_SHAPE;
    if (!q || !wq || !s_u || !q_out) return RESQ_ERR_NULL;
    if (!aligned16(q) || !aligned16(wq) || !aligned16(s_u) || !aligned16(q_out)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    return cuda_status((d_head == 64 ? launch_qkv_project_append64 : launch_qkv_project_append)(nullptr, q, rows, q_out, nullptr, nullptr, 0, nullptr, nullptr, wq, s_u,
                                                 static_cast<cudaStream_t>(stream)));
}

int resq_kv_append(const resq_kv_cache_t* cache, const void* k, const void* v, int64_t T, const int32_t* seq_ids,
                   const int32_t* positions, const int8_t* wq, const float* s_u, void* stream) {
    if (int e = check_cache(cache)) return e;
    if (T < 0) return RESQ_ERR_SHAPE;
    if (!k || !v || !seq_ids || !positions || !wq || !s_u) return RESQ_ERR_NULL;
    if (!aligned16(k) || !aligned16(v) || !aligned16(wq) || !aligned16(s_u)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    return cuda_status((cache->d_head == 64 ? launch_qkv_project_append64 : launch_qkv_project_append)(cache, nullptr, 0, nullptr, k, v, T, seq_ids, positions, wq, s_u,
                                                 static_cast<cudaStream_t>(stream)));
}

int resq_qkv_project_append(const resq_kv_cache_t* cache, const void* q, int n_q_heads, void* q_out, const void* k,
                            const void* v, int64_t T, const int32_t* seq_ids, const int32_t* positions,
                            const int8_t* wq, const float* s_u, void* stream) {
    if (int e = check_cache(cache)) return e;
    if (T < 0 || n_q_heads < 1) return RESQ_ERR_SHAPE;
    if (!q || !q_out || !k || !v || !seq_ids || !positions || !wq || !s_u) return RESQ_ERR_NULL;
    if (!aligned16(q) || !aligned16(q_out) || !aligned16(k) || !aligned16(v) || !aligned16(wq) || !aligned16(s_u))
        return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    return cuda_status((cache->d_head == 64 ? launch_qkv_project_append64 : launch_qkv_project_append)(cache, q, T * n_q_heads, q_out, k, v, T, seq_ids, positions, wq, s_u,
                                                 static_cast<cudaStream_t>(stream)));
}

size_t resq_attention_workspace_bytes(int n_seqs, int n_q_heads, int n_kv_heads, int d_head) {
    if (n_seqs < 1 || n_kv_heads < 1 || (d_head != 128 && d_head != 64) || n_q_heads < n_kv_heads ||
        n_q_heads % n_kv_heads != 0 || n_q_heads / n_kv_heads > 8)
        return 0;
    if (d_head == 64) return 256;  // the d_head = 64 kernel keeps its state in registers; a token amount keeps the contract
    return attention_scratch_bytes(n_seqs, n_kv_heads);
}

int resq_attention_decode(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, const int32_t* seq_lens,
                          float* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (int e = check_cache(cache)) return e;
    const size_t need = resq_attention_workspace_bytes(cache->n_seqs, n_q_heads, cache->n_kv_heads, cache->d_head);
    if (need == 0) return RESQ_ERR_SHAPE;
    if (!q16 || !seq_lens || !out) return RESQ_ERR_NULL;
    if (!workspace || workspace_bytes < need) return RESQ_ERR_WORKSPACE;
    if (!aligned16(q16) || !aligned16(out) || !aligned16(workspace)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    if (cache->d_head == 64)
        return cuda_status(launch_attention64(*cache, q16, n_q_heads, cache->n_seqs, nullptr, seq_lens, -1, 0, out,
                                              static_cast<cudaStream_t>(stream)));
    return cuda_status(launch_attention_decode(*cache, q16, n_q_heads, seq_lens, out, workspace,
                                               static_cast<cudaStream_t>(stream)));
}

unsigned long long resq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t resq_attention_queries_workspace_bytes(int n_queries, int n_q_heads, int n_kv_heads, int d_head) {
    return resq_attention_workspace_bytes(n_queries, n_q_heads, n_kv_heads, d_head);
}

int resq_attention_queries(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, int n_queries,
                           const int32_t* q_seq, const int32_t* q_len, float* out, void* workspace,
                           size_t workspace_bytes, void* stream) {
    if (int e = check_cache(cache)) return e;
    const size_t need = resq_attention_queries_workspace_bytes(n_queries, n_q_heads, cache->n_kv_heads, cache->d_head);
    if (need == 0) return RESQ_ERR_SHAPE;
    if (!q16 || !q_seq || !q_len || !out) return RESQ_ERR_NULL;
    if (!workspace || workspace_bytes < need) return RESQ_ERR_WORKSPACE;
    if (!aligned16(q16) || !aligned16(out) || !aligned16(workspace)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    if (cache->d_head == 64)
        return cuda_status(launch_attention64(*cache, q16, n_q_heads, n_queries, q_seq, q_len, -1, 0, out,
                                              static_cast<cudaStream_t>(stream)));
    return cuda_status(launch_attention_decode(*cache, q16, n_q_heads, q_len, out, workspace,
                                               static_cast<cudaStream_t>(stream), n_queries, q_seq));
}

int resq_attention_prefill(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, int seq, int pos0, int T,
                           float* out, void* stream) {
    if (int e = check_cache(cache)) return e;
    if (resq_attention_workspace_bytes(1, n_q_heads, cache->n_kv_heads, cache->d_head) == 0) return RESQ_ERR_SHAPE;
    if (seq < 0 || seq >= cache->n_seqs || pos0 < 0 || T < 1 || pos0 > cache->capacity - T) return RESQ_ERR_SHAPE;
    if (!q16 || !out) return RESQ_ERR_NULL;
    if (!aligned16(q16) || !aligned16(out)) return RESQ_ERR_ALIGN;
    if (int e = check_arch()) return e;
    if (cache->d_head == 64)
        return cuda_status(launch_attention64(*cache, q16, n_q_heads, T, nullptr, nullptr, seq, pos0, out,
                                              static_cast<cudaStream_t>(stream)));
    return cuda_status(launch_attention_prefill(*cache, q16, n_q_heads, seq, pos0, T, out, static_cast<cudaStream_t>(stream)));
}

const char* resq_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

const char* resq_status_string(int s) {
    switch (s) {
        case RESQ_OK: return "ok";
        case RESQ_ERR_NULL: return "null pointer";
        case RESQ_ERR_SHAPE: return "invalid shape";
        case RESQ_ERR_ALIGN: return "pointer not 16-byte aligned";
        case RESQ_ERR_WORKSPACE: return "workspace missing or too small";
        case RESQ_ERR_ARCH: return "device is not compute capability 10.x";
        case RESQ_ERR_CUDA: return "CUDA call failed";
        case RESQ_ERR_TIMEOUT: return "bounded device wait ran out";
        case RESQ_ERR_INDEX: return "device-side index out of range";
        default: return "unknown status";
    }
}

}  // extern "C"
