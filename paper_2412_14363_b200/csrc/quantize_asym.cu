// Per-row split quantization with ASYMMETRIC per-token codes (Eq. 1, second form; the activation setting
// of the paper's experiments, Section 5.1): per segment z = min, s = (max - min) / (2^N - 1),
// code = round-half-even((x - z) / s) in [0, 2^N - 1].  HBM-bound.
//
// Same staging as the symmetric fast kernel: a CTA takes 1-8 consecutive rows (about 32 KB), one
// thread issues a bulk copy per row (completion counted on an mbarrier), and every row is read twice
// from shared memory -- once for the two (min, max) pairs, once for the codes.
//
// Rounding.  The definition is code = rint(fl(fl(x - z) / s)) with IEEE fp32 operations.  With
// d = fl(x - z), t = fma(d, inv, M), inv = RN(1 / s), M = 1.5 * 2^23, rounds the exact product d * inv
// to the nearest integer (ties to even) in one instruction and leaves the code in the low byte of
// t's bit pattern.  d * inv and fl(d / s) both lie within 2^-15 of d / s for d / s <= 256, so the two
// roundings can only disagree when d * inv is within 2^-15 of a half-integer; whenever the residual of a
// chunk comes within 2^-14 of one half, the chunk is redone with the true division.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int kThreads = 256;
constexpr int kGroupBytes = 32 * 1024;
constexpr int kMaxRowBytes = 200 * 1024;
constexpr float kMagic = 12582912.f;                     // 1.5 * 2^23
constexpr float kTieGuard = 0.5f - 0.00006103515625f;    // 1/2 - 2^-14

// Eight consecutive elements of a staged row as fp32.
template <bool F32>
__device__ __forceinline__ void lds8(const uint8_t* row, int c, float (&v)[8]) {
    if constexpr (F32) {
        const float4 a = reinterpret_cast<const float4*>(row)[2 * c], b = reinterpret_cast<const float4*>(row)[2 * c + 1];
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
        const uint4 u = reinterpret_cast<const uint4*>(row)[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

// Codes of one chunk as the low bytes of t[0..7].
__device__ __forceinline__ void asym_codes(const float (&x)[8], float z, float s, float inv, bool exact_only, float qmax,
                                           uint32_t (&t)[8]) {
    float dmax = 0.f;
    float d[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        d[i] = __fsub_rn(x[i], z);
        const float tf = fmaf(d[i], inv, kMagic);
        const float res = fmaf(d[i], inv, -(tf - kMagic));
        dmax = fmaxf(dmax, fabsf(res));
        t[i] = __float_as_uint(tf);
    }
    if (exact_only || !(dmax < kTieGuard)) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float q = fminf(fmaxf(rintf(__fdiv_rn(d[i], s)), 0.f), qmax);
            t[i] = __float_as_uint(q + kMagic);
        }
    }
}

__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

template <bool F32>
__global__ void __launch_bounds__(kThreads)
split_quantize_asym_kernel(const void* __restrict__ in, size_t in_row_bytes, size_t rows, int K, int r,
                           int rows_per_cta, uint8_t* __restrict__ u8, uint8_t* __restrict__ u4,
                           float* __restrict__ s8_out, float* __restrict__ s4_out, float* __restrict__ z8_out,
                           float* __restrict__ z4_out, uint8_t* __restrict__ u4e, int* __restrict__ status) {
    extern __shared__ __align__(128) uint8_t stage[];
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    __shared__ float red[4][kThreads / 32];
    const uint32_t row_bytes = static_cast<uint32_t>(K) * (F32 ? 4u : 2u);
    const size_t row0 = static_cast<size_t>(blockIdx.x) * rows_per_cta;
    const int nrows = static_cast<int>(rows - row0 < static_cast<size_t>(rows_per_cta) ? rows - row0 : rows_per_cta);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        fence_mbar_init();
        mbar_arrive_expect_tx(&bar, row_bytes * static_cast<uint32_t>(nrows));
        for (int i = 0; i < nrows; ++i)
            bulk_load(stage + static_cast<size_t>(i) * row_bytes,
                      reinterpret_cast<const char*>(in) + (row0 + i) * in_row_bytes, row_bytes, &bar);
    }
    __syncthreads();
    const bool landed = mbar_wait(&bar, 0, &abort_flag, status);
    if (__syncthreads_or(!landed)) {
        if (threadIdx.x == 0) atomicOr(status, kStatusBitTimeout);
        return;
    }

    const int tpr = kThreads / rows_per_cta;  // threads per row, a multiple of 32
    const int grp = threadIdx.x / tpr, j = threadIdx.x - grp * tpr;
    const int nchunks = K >> 3, rchunks = r >> 3;
    const int K4 = K - r;
    const bool live = grp < nrows;
    const uint8_t* srow = stage + static_cast<size_t>(live ? grp : 0) * row_bytes;

    // ---- pass 1: (min, max) of the two segments
    const float kBig = 3.402823466e38f;
    float lo8 = kBig, hi8 = -kBig, lo4 = kBig, hi4 = -kBig;
    if (live) {
        float v[8];
        for (int c = j; c < rchunks; c += tpr) {
            lds8<F32>(srow, c, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) { lo8 = fminf(lo8, v[i]); hi8 = fmaxf(hi8, v[i]); }
        }
        for (int c = rchunks + j; c < nchunks; c += tpr) {
            lds8<F32>(srow, c, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) { lo4 = fminf(lo4, v[i]); hi4 = fmaxf(hi4, v[i]); }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo8 = fminf(lo8, __shfl_xor_sync(0xffffffffu, lo8, o));
        hi8 = fmaxf(hi8, __shfl_xor_sync(0xffffffffu, hi8, o));
        lo4 = fminf(lo4, __shfl_xor_sync(0xffffffffu, lo4, o));
        hi4 = fmaxf(hi4, __shfl_xor_sync(0xffffffffu, hi4, o));
    }
    if (tpr > 32) {
        const int warp = threadIdx.x >> 5, wpr = tpr >> 5;
        if ((threadIdx.x & 31) == 0) {
            red[0][warp] = lo8; red[1][warp] = hi8; red[2][warp] = lo4; red[3][warp] = hi4;
        }
        __syncthreads();
        for (int w = 0; w < wpr; ++w) {
            lo8 = fminf(lo8, red[0][grp * wpr + w]);
            hi8 = fmaxf(hi8, red[1][grp * wpr + w]);
            lo4 = fminf(lo4, red[2][grp * wpr + w]);
            hi4 = fmaxf(hi4, red[3][grp * wpr + w]);
        }
    }
    if (!live) return;
    if (rchunks == 0) lo8 = hi8 = 0.f;  // uniform 4-bit layer: the empty INT8 segment has s = 0, z = 0

    // ---- scales, zero-points
    const size_t row = row0 + grp;
    const float s8 = __fdiv_rn(__fsub_rn(hi8, lo8), 255.f), s4 = __fdiv_rn(__fsub_rn(hi4, lo4), 15.f);
    const float inv8 = s8 > 0.f ? __frcp_rn(s8) : 0.f, inv4 = s4 > 0.f ? __frcp_rn(s4) : 0.f;
    const bool exact8 = s8 > 0.f && !(inv8 >= 1.1754944e-38f && inv8 <= 3.0e38f);
    const bool exact4 = s4 > 0.f && !(inv4 >= 1.1754944e-38f && inv4 <= 3.0e38f);
    if (j == 0) {
        s8_out[row] = s8; s4_out[row] = s4;
        z8_out[row] = lo8; z4_out[row] = lo4;
    }
    uint8_t* u8row = u8 + row * static_cast<size_t>(r);
    uint8_t* u4row = u4 ? u4 + row * static_cast<size_t>(K4 >> 1) : nullptr;
    uint8_t* u4e_row = u4e ? u4e + row * static_cast<size_t>(K4) : nullptr;

    // ---- pass 2: codes
    for (int c = j; c < rchunks; c += tpr) {
        float v[8];
        uint32_t t[8];
        lds8<F32>(srow, c, v);
        if (s8 > 0.f) asym_codes(v, lo8, s8, inv8, exact8, 255.f, t);
        else {
#pragma unroll
            for (int k = 0; k < 8; ++k) t[k] = 0;
        }
        *reinterpret_cast<uint2*>(u8row + c * 8) =
            make_uint2(pack_low_bytes(t[0], t[1], t[2], t[3]), pack_low_bytes(t[4], t[5], t[6], t[7]));
    }
    for (int c = rchunks + j; c < nchunks; c += tpr) {
        float v[8];
        uint32_t t[8];
        lds8<F32>(srow, c, v);
        if (s4 > 0.f) asym_codes(v, lo4, s4, inv4, exact4, 15.f, t);
        else {
#pragma unroll
            for (int k = 0; k < 8; ++k) t[k] = 0;
        }
        const int jj = (c - rchunks) * 8;
        if (u4e_row)
            *reinterpret_cast<uint2*>(u4e_row + jj) =
                make_uint2(pack_low_bytes(t[0], t[1], t[2], t[3]), pack_low_bytes(t[4], t[5], t[6], t[7]));
        if (u4row) {
            uint32_t packed = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) packed |= (t[k] & 0xFu) << (4 * k);
            *reinterpret_cast<uint32_t*>(u4row + (jj >> 1)) = packed;
        }
    }
}

// Row sums of the weight codes of one output channel: one warp per channel.
__global__ void __launch_bounds__(256)
weight_row_sums_kernel(const int8_t* __restrict__ w8, const uint8_t* __restrict__ w4, int N, int r, int row4,
                       int32_t* __restrict__ wsum8, int32_t* __restrict__ wsum4) {
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= N) return;
    int a8 = 0, a4 = 0;
    const uint32_t* p8 = reinterpret_cast<const uint32_t*>(w8 + static_cast<size_t>(n) * r);
    for (int i = lane; i < (r >> 2); i += 32) a8 = __dp4a(static_cast<int>(p8[i]), 0x01010101, a8);
    const uint32_t* p4 = reinterpret_cast<const uint32_t*>(w4 + static_cast<size_t>(n) * row4);
    for (int i = lane; i < (row4 >> 2); i += 32) {
        const uint32_t w = p4[i];
        // both nibble sets as int8 lanes times 16; the sum is divided by 16 at the end (exact)
        a4 = __dp4a(static_cast<int>((w << 4) & 0xF0F0F0F0u), 0x01010101, a4);
        a4 = __dp4a(static_cast<int>(w & 0xF0F0F0F0u), 0x01010101, a4);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a8 += __shfl_xor_sync(0xffffffffu, a8, o);
        a4 += __shfl_xor_sync(0xffffffffu, a4, o);
    }
    if (lane == 0) {
        wsum8[n] = a8;
        wsum4[n] = a4 >> 4;
    }
}

}  // namespace

cudaError_t launch_split_quantize_asym(const void* in, bool in_is_f32, size_t rows, int K, int r, uint8_t* u8,
                                       uint8_t* u4, float* s8, float* s4, float* z8, float* z4, uint8_t* u4_u8,
                                       size_t in_row_stride_bytes, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    const size_t row_bytes = static_cast<size_t>(K) * (in_is_f32 ? 4 : 2);
    if (row_bytes > static_cast<size_t>(kMaxRowBytes) || in_row_stride_bytes % 16 != 0) return cudaErrorNotSupported;
    int rpc = 1;  // rows per CTA: 1, 2, 4 or 8, about kGroupBytes of staging
    while (rpc < 8 && row_bytes * rpc * 2 <= static_cast<size_t>(kGroupBytes)) rpc *= 2;
    const size_t smem = row_bytes * rpc;
    auto kern = in_is_f32 ? split_quantize_asym_kernel<true> : split_quantize_asym_kernel<false>;
    static bool attr_set[2][64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[in_is_f32][dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxRowBytes);
        if (e != cudaSuccess) return e;
        attr_set[in_is_f32][dev] = true;
    }
    const size_t groups = (rows + rpc - 1) / rpc;
    if (groups > 0x7fffffffu) return cudaErrorNotSupported;
    count_launch();
    kern<<<static_cast<unsigned>(groups), kThreads, smem, st>>>(in, in_row_stride_bytes, rows, K, r, rpc, u8, u4, s8, s4,
                                                            z8, z4, u4_u8, device_status_ptr());
    return cudaGetLastError();
}

cudaError_t launch_weight_row_sums(const int8_t* w8, const uint8_t* w4, int N, int K, int r, int32_t* wsum8,
                                   int32_t* wsum4, cudaStream_t st) {
    count_launch();
    weight_row_sums_kernel<<<(N + 7) / 8, 256, 0, st>>>(w8, w4, N, r, (K - r) / 2, wsum8, wsum4);
    return cudaGetLastError();
}

}  // namespace resq
