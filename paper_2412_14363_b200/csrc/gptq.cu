// GPTQ rounding of projected weights at pack time (Section 5.1: the projected weights are quantized with GPTQ).
//
// For every output channel (row of W_proj) the columns are visited in order; a weight is rounded to its code
// with the row's round-to-nearest scale of Eq. 3, and the rounding error, divided by the diagonal entry of the
// upper Cholesky factor U of the inverse Hessian, is fed back into the columns not yet visited:
//     e = (w_j - code_j * s) / U[j][j],      w[j+1:] -= e * U[j][j+1:].
// Rows never interact, so a CTA owns R rows for the whole sweep: they live in shared memory as fp64, one
// thread per row rounds column j while the others wait, then all threads apply the update along the rows.
// Everything is fp64 with one rounding per operation (multiply, subtract, divide written out: no contraction),
// the order in which the definition states it, so the codes are those of an fp64 reference bit for bit.  The
// sweep is a chain of K dependent steps (two barriers and one row of U each); this is an offline step, sized
// for correctness and memory traffic (U is read once per CTA, from L2 when it fits), not for speed.
#include <cuda_fp16.h>

#include "internal.h"

namespace resq {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxRows = 8;
constexpr size_t kSmemBudget = 200 * 1024;

struct Params {
    const float* W;       // [N][K]
    const float* U;       // [K][K], upper triangular factor of H^-1
    const uint8_t* dead;  // [K] or NULL: columns whose weights are set to 0
    int N, K, r, R;
    int8_t* w8;
    uint8_t* w4;
    void* s8;
    void* s4;
    int fp16;
    int8_t* w4e;
};

__global__ void __launch_bounds__(kThreads) gptq_rows_kernel(const Params p) {
    extern __shared__ __align__(16) unsigned char smem[];
    double* Wd = reinterpret_cast<double*>(smem);                                   // [R][K]
    int8_t* code = reinterpret_cast<int8_t*>(smem + static_cast<size_t>(p.R) * p.K * 8);  // [R][K]
    __shared__ double err[kMaxRows];
    __shared__ float red[2][kMaxRows][kThreads / 32];
    __shared__ float scale[2][kMaxRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n0 = blockIdx.x * p.R;
    const int rows = min(p.R, p.N - n0);
    const int K = p.K, r = p.r;

    // Rows into shared memory (dead columns zeroed); per-row absmax of the two segments in fp32, as Eq. 3 takes it.
    for (int rr = 0; rr < rows; ++rr) {
        const float* src = p.W + static_cast<size_t>(n0 + rr) * K;
        float a8 = 0.f, a4 = 0.f;
        for (int c = tid; c < K; c += kThreads) {
            float w = src[c];
            if (p.dead && p.dead[c]) w = 0.f;
            Wd[static_cast<size_t>(rr) * K + c] = static_cast<double>(w);
            if (c < r) a8 = fmaxf(a8, fabsf(w));
            else a4 = fmaxf(a4, fabsf(w));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a8 = fmaxf(a8, __shfl_xor_sync(0xffffffffu, a8, o));
            a4 = fmaxf(a4, __shfl_xor_sync(0xffffffffu, a4, o));
        }
        if (lane == 0) {
            red[0][rr][warp] = a8;
            red[1][rr][warp] = a4;
        }
    }
    __syncthreads();
    if (tid < rows) {
        float a8 = 0.f, a4 = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) {
            a8 = fmaxf(a8, red[0][tid][w]);
            a4 = fmaxf(a4, red[1][tid][w]);
        }
        float s8 = __fdiv_rn(a8, 127.f), s4 = __fdiv_rn(a4, 7.f);
        if (p.fp16) {
            s8 = __half2float(__float2half_rn(s8));
            s4 = __half2float(__float2half_rn(s4));
        }
        scale[0][tid] = s8;
        scale[1][tid] = s4;
        const size_t n = n0 + tid;
        if (p.fp16) {
            reinterpret_cast<__half*>(p.s8)[n] = __float2half_rn(s8);
            reinterpret_cast<__half*>(p.s4)[n] = __float2half_rn(s4);
        } else {
            reinterpret_cast<float*>(p.s8)[n] = s8;
            reinterpret_cast<float*>(p.s4)[n] = s4;
        }
    }
    __syncthreads();

    // The sweep.  Thread rr < rows rounds column j of row rr; the diagonal entry of the next column is requested
    // one step ahead so that its latency is not on the chain.
    double diag = tid < rows ? static_cast<double>(p.U[0]) : 0.0;
    for (int j = 0; j < K; ++j) {
        double diag_next = 0.0;
        if (tid < rows) {
            if (j + 1 < K) diag_next = static_cast<double>(p.U[static_cast<size_t>(j + 1) * K + j + 1]);
            const double w = Wd[static_cast<size_t>(tid) * K + j];
            const double s = static_cast<double>(scale[j < r ? 0 : 1][tid]);
            double c = 0.0;
            if (s > 0.0) {
                c = rint(__ddiv_rn(w, s));
                const double lo = j < r ? -128.0 : -8.0, hi = j < r ? 127.0 : 7.0;
                c = fmin(fmax(c, lo), hi);
            }
            code[static_cast<size_t>(tid) * K + j] = static_cast<int8_t>(static_cast<int>(c));
            err[tid] = __ddiv_rn(__dsub_rn(w, __dmul_rn(c, s)), diag);
        }
        __syncthreads();
        const float* urow = p.U + static_cast<size_t>(j) * K;
        for (int c = j + 1 + tid; c < K; c += kThreads) {
            const double u = static_cast<double>(urow[c]);
            for (int rr = 0; rr < rows; ++rr) {
                double* w = &Wd[static_cast<size_t>(rr) * K + c];
                *w = __dsub_rn(*w, __dmul_rn(err[rr], u));
            }
        }
        diag = diag_next;
        __syncthreads();
    }

    // Codes out: INT8 segment, INT4 packed two per byte (code 2i in the low nibble) and, optionally, one per byte.
    const int K4 = K - r;
    for (int rr = 0; rr < rows; ++rr) {
        const size_t n = n0 + rr;
        const int8_t* c = code + static_cast<size_t>(rr) * K;
        for (int i = tid; i < r; i += kThreads) p.w8[n * r + i] = c[i];
        for (int i = tid; i < K4 / 2; i += kThreads)
            p.w4[n * (K4 / 2) + i] = static_cast<uint8_t>((c[r + 2 * i] & 0xF) | ((c[r + 2 * i + 1] & 0xF) << 4));
        if (p.w4e)
            for (int i = tid; i < K4; i += kThreads) p.w4e[n * K4 + i] = c[r + i];
    }
}

}  // namespace

// cudaErrorNotSupported: a row (9 bytes per weight) does not fit in shared memory.
cudaError_t launch_pack_gptq(const float* W, const float* U, const uint8_t* dead, int N, int K, int r, int8_t* w8,
                             uint8_t* w4, void* s8, void* s4, bool scale_fp16, int8_t* w4e, cudaStream_t st) {
    const size_t per_row = static_cast<size_t>(K) * 9;
    if (per_row > kSmemBudget) return cudaErrorNotSupported;
    int R = static_cast<int>((64u * 1024u) / per_row);  // about 64 KB per CTA: three CTAs per SM hide each other's waits
    if (R < 1) R = 1;
    if (R > kMaxRows) R = kMaxRows;
    const size_t smem = per_row * R;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(gptq_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemBudget));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    Params p{W, U, dead, N, K, r, R, w8, w4, s8, s4, scale_fp16 ? 1 : 0, w4e};
    count_launch();
    gptq_rows_kernel<<<(N + R - 1) / R, kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace resq
