// Per-row split quantization (Eq. 1 applied per segment, Eq. 2 / Eq. 3): HBM-bound.
//
// One CTA per row.  Each thread owns 8-element chunks (one 128-bit bf16 load, or two for fp32),
// keeps up to kMaxChunks of them in registers so the row is read from memory once, reduces the two
// per-segment absmax values with warp shuffles + one shared-memory step, then emits int8 codes
// (8-byte stores) and packed int4 codes (4-byte stores).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"

namespace resq {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxChunks = 8;  // register-cached chunks per thread: rows up to 8*8*256 = 16384 wide

// A chunk is kept in registers in its storage format: 4 words of bf16 pairs, or 8 fp32 words.
template <bool F32>
struct Chunk {
    uint32_t w[F32 ? 8 : 4];
    __device__ __forceinline__ float get(int i) const {
        if constexpr (F32) return __uint_as_float(w[i]);
        else return (i & 1) ? __uint_as_float(w[i >> 1] & 0xFFFF0000u) : __uint_as_float(w[i >> 1] << 16);
    }
};

template <bool F32>
__device__ __forceinline__ Chunk<F32> load_chunk(const void* row, int c) {
    Chunk<F32> o;
    if constexpr (F32) {
        const uint4* p = reinterpret_cast<const uint4*>(row) + 2 * c;
        uint4 a = __ldg(p), b = __ldg(p + 1);
        o.w[0] = a.x; o.w[1] = a.y; o.w[2] = a.z; o.w[3] = a.w;
        o.w[4] = b.x; o.w[5] = b.y; o.w[6] = b.z; o.w[7] = b.w;
    } else {
        uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + c);
        o.w[0] = u.x; o.w[1] = u.y; o.w[2] = u.z; o.w[3] = u.w;
    }
    return o;
}

template <bool F32>
__device__ __forceinline__ float chunk_absmax(const Chunk<F32>& c) {
    float m = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(c.get(i)));
    return m;
}

// code = clamp(round-half-even(x / s)); IEEE division, no reciprocal.
__device__ __forceinline__ int quant1(float x, float s, float lo, float hi) {
    float q = rintf(__fdiv_rn(x, s));
    q = fminf(fmaxf(q, lo), hi);
    return static_cast<int>(q);
}

template <bool F32>
__device__ __forceinline__ void store_chunk(const Chunk<F32>& ch, int col, int r, float s8, float s4, int8_t* q8row,
                                            uint8_t* q4row, int8_t* q4e_row) {
    if (col < r) {
        uint32_t w0 = 0, w1 = 0;
        if (s8 > 0.f) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                w0 |= (static_cast<uint32_t>(quant1(ch.get(i), s8, -128.f, 127.f)) & 0xFFu) << (8 * i);
                w1 |= (static_cast<uint32_t>(quant1(ch.get(4 + i), s8, -128.f, 127.f)) & 0xFFu) << (8 * i);
            }
        }
        *reinterpret_cast<uint2*>(q8row + col) = make_uint2(w0, w1);
    } else {
        const int j = col - r;
        uint32_t packed = 0, w0 = 0, w1 = 0;
        if (s4 > 0.f) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t q = static_cast<uint32_t>(quant1(ch.get(i), s4, -8.f, 7.f));
                packed |= (q & 0xFu) << (4 * i);
                if (i < 4) w0 |= (q & 0xFFu) << (8 * i);
                else w1 |= (q & 0xFFu) << (8 * (i - 4));
            }
        }
        if (q4row) *reinterpret_cast<uint32_t*>(q4row + (j >> 1)) = packed;
        if (q4e_row) *reinterpret_cast<uint2*>(q4e_row + j) = make_uint2(w0, w1);
    }
}

template <bool F32>
__global__ void __launch_bounds__(kThreads)
split_quantize_kernel(const void* __restrict__ in, size_t in_row_bytes, size_t rows, int K, int r,
                      int8_t* __restrict__ q8, uint8_t* __restrict__ q4, void* __restrict__ s8_out,
                      void* __restrict__ s4_out, int scale_fp16, int8_t* __restrict__ q4e) {
    __shared__ float red[2][kThreads / 32];
    const int nchunks = K >> 3;
    const int K4 = K - r;
    for (size_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const char* rp = reinterpret_cast<const char*>(in) + row * in_row_bytes;
        Chunk<F32> cache[kMaxChunks];
        float a8 = 0.f, a4 = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = threadIdx.x + i * kThreads;
            if (c < nchunks) {
                cache[i] = load_chunk<F32>(rp, c);
                const float m = chunk_absmax(cache[i]);
                if (c * 8 < r) a8 = fmaxf(a8, m);
                else a4 = fmaxf(a4, m);
            }
        }
        for (int c = threadIdx.x + kMaxChunks * kThreads; c < nchunks; c += kThreads) {  // rows wider than the cache
            const float m = chunk_absmax(load_chunk<F32>(rp, c));
            if (c * 8 < r) a8 = fmaxf(a8, m);
            else a4 = fmaxf(a4, m);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a8 = fmaxf(a8, __shfl_xor_sync(0xffffffffu, a8, o));
            a4 = fmaxf(a4, __shfl_xor_sync(0xffffffffu, a4, o));
        }
        __syncthreads();  // previous row's readers of `red` are done
        if ((threadIdx.x & 31) == 0) {
            red[0][threadIdx.x >> 5] = a8;
            red[1][threadIdx.x >> 5] = a4;
        }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            a8 = fmaxf(a8, red[0][w]);
            a4 = fmaxf(a4, red[1][w]);
        }
        float s8 = __fdiv_rn(a8, 127.f), s4 = __fdiv_rn(a4, 7.f);
        if (scale_fp16) {
            s8 = __half2float(__float2half_rn(s8));
            s4 = __half2float(__float2half_rn(s4));
        }
        if (threadIdx.x == 0) {
            if (scale_fp16) {
                reinterpret_cast<__half*>(s8_out)[row] = __float2half_rn(s8);
                reinterpret_cast<__half*>(s4_out)[row] = __float2half_rn(s4);
            } else {
                reinterpret_cast<float*>(s8_out)[row] = s8;
                reinterpret_cast<float*>(s4_out)[row] = s4;
            }
        }
        int8_t* q8row = q8 + row * static_cast<size_t>(r);
        uint8_t* q4row = q4 ? q4 + row * static_cast<size_t>(K4 >> 1) : nullptr;
        int8_t* q4e_row = q4e ? q4e + row * static_cast<size_t>(K4) : nullptr;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = threadIdx.x + i * kThreads;
            if (c < nchunks) store_chunk(cache[i], c * 8, r, s8, s4, q8row, q4row, q4e_row);
        }
        for (int c = threadIdx.x + kMaxChunks * kThreads; c < nchunks; c += kThreads)
            store_chunk(load_chunk<F32>(rp, c), c * 8, r, s8, s4, q8row, q4row, q4e_row);
    }
}

__global__ void unpack_int4_kernel(const uint8_t* __restrict__ packed, int8_t* __restrict__ out, size_t nwords) {
    // one 32-bit packed word (8 codes) per thread -> 8 bytes
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < nwords;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(packed) + i);
        uint32_t o[2] = {0, 0};
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            int v = static_cast<int>((w >> (4 * k)) & 0xFu);
            v = (v ^ 8) - 8;  // sign-extend the nibble
            o[k >> 2] |= (static_cast<uint32_t>(v) & 0xFFu) << (8 * (k & 3));
        }
        reinterpret_cast<uint2*>(out)[i] = make_uint2(o[0], o[1]);
    }
}

}  // namespace

cudaError_t launch_split_quantize(const void* in, bool in_is_f32, size_t rows, int K, int r, int8_t* q8,
                                  uint8_t* q4, void* s8, void* s4, bool scale_fp16, int8_t* q4_i8,
                                  size_t in_row_stride_bytes, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    const unsigned grid = static_cast<unsigned>(rows < 148u * 64u ? rows : 148u * 64u);
    if (in_is_f32)
        split_quantize_kernel<true><<<grid, kThreads, 0, st>>>(in, in_row_stride_bytes, rows, K, r, q8, q4, s8, s4,
                                                               scale_fp16 ? 1 : 0, q4_i8);
    else
        split_quantize_kernel<false><<<grid, kThreads, 0, st>>>(in, in_row_stride_bytes, rows, K, r, q8, q4, s8, s4,
                                                                scale_fp16 ? 1 : 0, q4_i8);
    return cudaGetLastError();
}

cudaError_t launch_unpack_int4(const uint8_t* packed, int8_t* out, size_t rows, size_t cols, cudaStream_t st) {
    const size_t nwords = rows * cols / 8;
    if (nwords == 0) return cudaSuccess;
    size_t blocks = (nwords + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    unpack_int4_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(packed, out, nwords);
    return cudaGetLastError();
}

}  // namespace resq
