// Per-row split quantization (Eq. 1 applied per segment, Eq. 2 / Eq. 3): HBM-bound.
//
// One CTA per row.  Each thread owns 8-element chunks (one 128-bit bf16 load, or two for fp32),
// keeps up to kMaxChunks of them in registers so the row is read from memory once, reduces the two
// per-segment absmax values with warp shuffles + one shared-memory step, then emits int8 codes
// (8-byte stores) and packed int4 codes (4-byte stores).
#include <cmath>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"
#include "ptx.cuh"

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
    if constexpr (F32) {
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(c.get(i)));
        return m;
    } else {
        // bf16 pairs: clear the signs, then compare as packed bf16 (exact: max selects one of its inputs)
        __nv_bfloat162 m = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = c.w[i] & 0x7FFF7FFFu;
            m = __hmax2(m, *reinterpret_cast<const __nv_bfloat162*>(&a));
        }
        return fmaxf(__low2float(m), __high2float(m));
    }
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

// ---------------------------------------------------------------------------------------------
// Fast path (fp32 scales).  Same codes as the kernel above, bit for bit, at a fraction of its
// instructions and with the row staged in shared memory instead of registers.
//
// Staging.  A CTA takes a group of 1, 2, 4 or 8 consecutive rows (about 32 KB); one thread issues a
// bulk copy (cp.async.bulk, completion counted on an mbarrier) per row, so the whole group is in
// flight at once and several CTAs per SM keep HBM busy while others compute.  Each row is then read
// twice from shared memory: once for the two absmax values, once for the codes.
//
// Rounding.  The definition is code = round-half-even(fl(x / s)) with an IEEE division.  Here
// t = fma(x, v, M) with M = 1.5 * 2^23 rounds the exact product x * v to the nearest integer (ties to
// even) in one instruction, and the low byte of t's bit pattern is the two's-complement code.  It is
// evaluated for two factors that bracket 1 / s, v_lo = RN(inv (1 - 2^-20)) and v_hi = RN(inv (1 + 2^-20))
// with inv = RN(1 / s): fl(x / s) lies between x * v_lo and x * v_hi (the division and the reciprocal
// are each off by at most 2^-24 relative, the bracket is 2^-21 wide at least on either side), rounding to
// nearest is monotone, so when both products round to the same integer, that integer is the defined code;
// when they differ (the quotient is within |x / s| * 2^-19 of a half-integer, ties included) the chunk is
// redone with the true division.
constexpr int kFastGroupBytes = 32 * 1024;
constexpr int kFastMaxRowBytes = 200 * 1024;
constexpr float kMagic = 12582912.f;                    // 1.5 * 2^23
constexpr float kBracket = 9.5367431640625e-07f;        // 2^-20

template <bool F32>
__device__ __forceinline__ Chunk<F32> lds_chunk(const uint8_t* row, int c) {
    Chunk<F32> o;
    if constexpr (F32) {
        const uint4* p = reinterpret_cast<const uint4*>(row) + 2 * c;
        const uint4 a = p[0], b = p[1];
        o.w[0] = a.x; o.w[1] = a.y; o.w[2] = a.z; o.w[3] = a.w;
        o.w[4] = b.x; o.w[5] = b.y; o.w[6] = b.z; o.w[7] = b.w;
    } else {
        const uint4 u = reinterpret_cast<const uint4*>(row)[c];
        o.w[0] = u.x; o.w[1] = u.y; o.w[2] = u.z; o.w[3] = u.w;
    }
    return o;
}

template <bool F32>
__device__ __forceinline__ void fast_codes(const Chunk<F32>& ch, float s, float inv, bool exact_only, uint32_t (&t)[8]) {
    const float v_lo = fmaf(inv, -kBracket, inv), v_hi = fmaf(inv, kBracket, inv);
    uint32_t differ = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float x = ch.get(i);
        t[i] = __float_as_uint(fmaf(x, v_lo, kMagic));
        differ |= t[i] ^ __float_as_uint(fmaf(x, v_hi, kMagic));
    }
    if (exact_only || differ != 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = __float_as_uint(rintf(__fdiv_rn(ch.get(i), s)) + kMagic);
    }
}

// Low bytes of four words -> one word.
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

template <bool F32>
__global__ void __launch_bounds__(kThreads)
split_quantize_fast_kernel(const void* __restrict__ in, size_t in_row_bytes, size_t rows, int K, int r,
                           int rows_per_cta, int nstages, int8_t* __restrict__ q8, uint8_t* __restrict__ q4,
                           float* __restrict__ s8_out, float* __restrict__ s4_out, int8_t* __restrict__ q4e,
                           int* __restrict__ status) {
    extern __shared__ __align__(128) uint8_t stage[];
    __shared__ uint64_t bar[2];
    __shared__ int abort_flag;
    __shared__ float red[2][kThreads / 32];
    // A kernel enqueued behind this one with programmatic stream serialization may start its own
    // input-independent prologue now; it still waits for this grid to finish before reading the codes.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Enqueued with programmatic stream serialization itself (behind the projection GEMM), this grid may have been
    // scheduled before its input was complete: wait for the preceding grid (returns at once otherwise).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t row_bytes = static_cast<uint32_t>(K) * (F32 ? 4u : 2u);
    const size_t group_bytes = static_cast<size_t>(row_bytes) * rows_per_cta;
    const size_t groups = (rows + rows_per_cta - 1) / rows_per_cta;
    auto rows_of = [&](size_t g) {
        const size_t row0 = g * rows_per_cta;
        return static_cast<int>(rows - row0 < static_cast<size_t>(rows_per_cta) ? rows - row0 : rows_per_cta);
    };
    auto issue = [&](size_t g, int buf) {  // one thread: the rows of group g, one bulk copy each
        const int n = rows_of(g);
        mbar_arrive_expect_tx(&bar[buf], row_bytes * static_cast<uint32_t>(n));
        for (int i = 0; i < n; ++i)
            bulk_load(stage + buf * group_bytes + static_cast<size_t>(i) * row_bytes,
                      reinterpret_cast<const char*>(in) + (g * rows_per_cta + i) * in_row_bytes, row_bytes, &bar[buf]);
    };
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        fence_mbar_init();
        if (blockIdx.x < groups) issue(blockIdx.x, 0);
    }
    __syncthreads();

    const int tpr = kThreads / rows_per_cta;  // threads per row, a multiple of 32
    const int grp = threadIdx.x / tpr, j = threadIdx.x - grp * tpr;
    const int nchunks = K >> 3, rchunks = r >> 3;
    const int K4 = K - r;

    // The CTA walks its groups (grid-stride); with two stages the rows of the next group are in flight while this
    // one is quantized, so the copy engine never waits for the arithmetic of the same CTA.
    int it = 0;
    for (size_t g = blockIdx.x; g < groups; g += gridDim.x, ++it) {
        const int buf = nstages == 2 ? (it & 1) : 0;
        const uint32_t parity = nstages == 2 ? (it >> 1) & 1 : it & 1;
        const bool more = g + gridDim.x < groups;
        if (nstages == 2 && more && threadIdx.x == 0) issue(g + gridDim.x, buf ^ 1);
        const bool landed = mbar_wait(&bar[buf], parity, &abort_flag, status);
        if (__syncthreads_or(!landed)) {
            // The copy did not land in time: report it and leave the outputs of the remaining groups unwritten.
            if (threadIdx.x == 0) {
                atomicOr(status, kStatusBitTimeout);
                if (nstages == 2 && more) {  // the copies of the next group are still this CTA's to wait for
                    int keep_waiting = 0;
                    (void)mbar_wait(&bar[buf ^ 1], ((it + 1) >> 1) & 1, &keep_waiting, status);
                }
            }
            return;
        }
        const int nrows = rows_of(g);
        const size_t row0 = g * rows_per_cta;
        const bool live = grp < nrows;
        const uint8_t* srow = stage + buf * group_bytes + static_cast<size_t>(live ? grp : 0) * row_bytes;

        float a8 = 0.f, a4 = 0.f;
        if (live) {
            if constexpr (F32) {
                for (int c = j; c < rchunks; c += tpr) a8 = fmaxf(a8, chunk_absmax(lds_chunk<F32>(srow, c)));
                float m0 = 0.f, m1 = 0.f;  // two chains: the INT4 segment is 7/8 of the row
                int c = rchunks + j;
                for (; c + tpr < nchunks; c += 2 * tpr) {
                    m0 = fmaxf(m0, chunk_absmax(lds_chunk<F32>(srow, c)));
                    m1 = fmaxf(m1, chunk_absmax(lds_chunk<F32>(srow, c + tpr)));
                }
                if (c < nchunks) m0 = fmaxf(m0, chunk_absmax(lds_chunk<F32>(srow, c)));
                a4 = fmaxf(m0, m1);
            } else {
                // bf16 rows: sign bits cleared, maxima kept as packed pairs until the end (two operations per pair)
                const uint4* v = reinterpret_cast<const uint4*>(srow);
                uint32_t m8 = 0, m4a = 0, m4b = 0;
                auto acc = [](uint32_t& m, const uint4 u) {
                    const uint32_t w[4] = {u.x & 0x7FFF7FFFu, u.y & 0x7FFF7FFFu, u.z & 0x7FFF7FFFu, u.w & 0x7FFF7FFFu};
                    __nv_bfloat162 mm = *reinterpret_cast<const __nv_bfloat162*>(&m);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mm = __hmax2(mm, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
                    m = *reinterpret_cast<const uint32_t*>(&mm);
                };
                for (int c = j; c < rchunks; c += tpr) acc(m8, v[c]);
                int c = rchunks + j;
#pragma unroll 2
                for (; c + tpr < nchunks; c += 2 * tpr) {
                    acc(m4a, v[c]);
                    acc(m4b, v[c + tpr]);
                }
                if (c < nchunks) acc(m4a, v[c]);
                auto unpack = [](uint32_t m) { return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u)); };
                a8 = unpack(m8);
                a4 = fmaxf(unpack(m4a), unpack(m4b));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a8 = fmaxf(a8, __shfl_xor_sync(0xffffffffu, a8, o));
            a4 = fmaxf(a4, __shfl_xor_sync(0xffffffffu, a4, o));
        }
        if (tpr > 32) {
            const int warp = threadIdx.x >> 5, wpr = tpr >> 5;
            if ((threadIdx.x & 31) == 0) {
                red[0][warp] = a8;
                red[1][warp] = a4;
            }
            __syncthreads();
            for (int w = 0; w < wpr; ++w) {
                a8 = fmaxf(a8, red[0][grp * wpr + w]);
                a4 = fmaxf(a4, red[1][grp * wpr + w]);
            }
        }
        if (live) {
            const size_t row = row0 + grp;
            const float s8 = __fdiv_rn(a8, 127.f), s4 = __fdiv_rn(a4, 7.f);
            const float inv8 = s8 > 0.f ? __frcp_rn(s8) : 0.f, inv4 = s4 > 0.f ? __frcp_rn(s4) : 0.f;
            // The product form needs a finite, normal reciprocal; otherwise every chunk takes the division.
            const bool exact8 = s8 > 0.f && !(inv8 >= 1.1754944e-38f && inv8 <= 3.0e38f);
            const bool exact4 = s4 > 0.f && !(inv4 >= 1.1754944e-38f && inv4 <= 3.0e38f);
            if (j == 0) {
                s8_out[row] = s8;
                s4_out[row] = s4;
            }
            int8_t* q8row = q8 + row * static_cast<size_t>(r);
            uint8_t* q4row = q4 ? q4 + row * static_cast<size_t>(K4 >> 1) : nullptr;
            int8_t* q4e_row = q4e ? q4e + row * static_cast<size_t>(K4) : nullptr;

            for (int c = j; c < rchunks; c += tpr) {
                uint32_t t[8];
                if (s8 > 0.f) fast_codes(lds_chunk<F32>(srow, c), s8, inv8, exact8, t);
                else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) t[k] = 0;
                }
                *reinterpret_cast<uint2*>(q8row + c * 8) =
                    make_uint2(pack_low_bytes(t[0], t[1], t[2], t[3]), pack_low_bytes(t[4], t[5], t[6], t[7]));
            }
#pragma unroll 2
            for (int c = rchunks + j; c < nchunks; c += tpr) {
                uint32_t t[8];
                if (s4 > 0.f) fast_codes(lds_chunk<F32>(srow, c), s4, inv4, exact4, t);
                else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) t[k] = 0;
                }
                const int jj = (c - rchunks) * 8;
                const uint32_t lo = pack_low_bytes(t[0], t[1], t[2], t[3]), hi = pack_low_bytes(t[4], t[5], t[6], t[7]);
                if (q4e_row) *reinterpret_cast<uint2*>(q4e_row + jj) = make_uint2(lo, hi);
                if (q4row) {
                    // two's-complement nibbles of the eight bytes: byte pairs (b0 | b1 << 4) sit in bytes 0 and 2 of
                    // x | x >> 4 once the high nibbles are cleared
                    const uint32_t xl = lo & 0x0F0F0F0Fu, xh = hi & 0x0F0F0F0Fu;
                    *reinterpret_cast<uint32_t*>(q4row + (jj >> 1)) = __byte_perm(xl | (xl >> 4), xh | (xh >> 4), 0x6420);
                }
            }
        }
        __syncthreads();  // every thread is done with this stage (and with `red`) before it is refilled
        if (nstages == 1 && more && threadIdx.x == 0) issue(g + gridDim.x, 0);
    }
}

template <bool UNSIGNED>
__global__ void unpack_int4_kernel(const uint8_t* __restrict__ packed, int8_t* __restrict__ out, size_t nwords) {
    // one 32-bit packed word (8 codes) per thread -> 8 bytes
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < nwords;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(packed) + i);
        uint32_t o[2] = {0, 0};
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            int v = static_cast<int>((w >> (4 * k)) & 0xFu);
            if (!UNSIGNED) v = (v ^ 8) - 8;  // sign-extend the nibble
            o[k >> 2] |= (static_cast<uint32_t>(v) & 0xFFu) << (8 * (k & 3));
        }
        reinterpret_cast<uint2*>(out)[i] = make_uint2(o[0], o[1]);
    }
}

// ---------------------------------------------------------------------------------------------
// Hadamard basis for the down_proj input (Section 4.3: U_D is a Hadamard matrix so that the projection
// that cannot be folded costs a fast transform instead of a dense product), fused with the per-token
// quantizer: C = X * H_K / sqrt(K), H_K = Sylvester(2^k) (x) H_m with coefficient index a * m + b, m = 1, or
// m = 12 / 28 with Paley's second construction (q = 5 / 13).  One CTA per row: the row is widened to fp32
// in shared memory, multiplied group-wise by the small factor (a compile-time table), run through the
// Sylvester butterflies up to five index bits per pass (32 values in registers),
// scaled, and then quantized exactly as in the fast path above (absmax per segment, reciprocal-product
// rounding with the exact fallback).  r = 0 gives the paper's uniform INT4 down_proj input.
// Paley's second construction for a prime q = 1 (mod 4): H = S (x) [[1,1],[1,-1]] + I (x) [[1,-1],[-1,-1]] of order
// 2 (q + 1), with S = [[0, 1^T], [1, chi(i - j)]] and chi the quadratic character of GF(q).  S is evaluated at compile
// time, so the product with H is additions and subtractions only: with p_i = x_2i + x_2i+1 and m_i = x_2i - x_2i+1,
//   y_2j = m_j + sum_i S_ij p_i,   y_2j+1 = -p_j + sum_i S_ij m_i,
// and the circulant block of S needs only its quadratic-residue half (see the kernel): about 290 operations for
// M = 28, not M * M = 784.
constexpr int quad_char(int q, int a) {
    a = ((a % q) + q) % q;
    if (a == 0) return 0;
    for (int x = 1; x < q; ++x)
        if ((x * x) % q == a) return 1;
    return -1;
}
template <int M>
struct Conference {
    int s[M / 2][M / 2];
    constexpr Conference() : s() {
        constexpr int q = M / 2 - 1;
        for (int i = 0; i < M / 2; ++i)
            for (int j = 0; j < M / 2; ++j)
                s[i][j] = i == 0 ? (j == 0 ? 0 : 1) : (j == 0 ? 1 : quad_char(q, (i - 1) - (j - 1)));
    }
};

constexpr int kWideThreads = 1024;  // threads per row when there are at most kWideMaxRows rows (one CTA per SM)
constexpr int kWideMaxRows = 148;
// One pass of the Sylvester butterflies: index bits [s, s + NB) of a, 2^NB values per thread in registers.  The last
// pass also scales by 1 / sqrt(K) and collects the two absmax values (elements below r belong to the INT8 segment).
template <int M, int NT, int NB>
__device__ __forceinline__ void butterfly_pass(float* hrow, int K, int s, int tid, bool last, float inv_sqrt_k, int r,
                                               float& a8, float& a4) {
    constexpr int N = 1 << NB;
    const int count = K >> NB;
    const int stride = M << s;
    for (int i = tid; i < count; i += NT) {
        const int arest = i / M, b = i - arest * M;
        const int a0 = ((arest >> s) << (s + NB)) | (arest & ((1 << s) - 1));
        float* base = hrow + a0 * M + b;
        float v[N];
#pragma unroll
        for (int j = 0; j < N; ++j) v[j] = base[j * stride];
#pragma unroll
        for (int bit = 0; bit < NB; ++bit) {
#pragma unroll
            for (int j = 0; j < N; ++j) {
                if (!(j & (1 << bit))) {
                    const float lo = v[j], hi = v[j | (1 << bit)];
                    v[j] = lo + hi;
                    v[j | (1 << bit)] = lo - hi;
                }
            }
        }
        if (last) {
            const int e0 = a0 * M + b;
#pragma unroll
            for (int j = 0; j < N; ++j) {
                v[j] *= inv_sqrt_k;
                if (e0 + j * stride < r) a8 = fmaxf(a8, fabsf(v[j]));
                else a4 = fmaxf(a4, fabsf(v[j]));
            }
        }
#pragma unroll
        for (int j = 0; j < N; ++j) base[j * stride] = v[j];
    }
}

// NT threads per row: 256 when rows outnumber the SMs (throughput: several CTAs per SM), 1024 for the few rows of a
// generation step, where one row's chain of passes is all there is to wait for.
template <int M, int NT>
__global__ void __launch_bounds__(NT)
hadamard_quantize_kernel(const __nv_bfloat16* __restrict__ X, size_t rows, int K, int kbits, int r, float inv_sqrt_k,
                         int8_t* __restrict__ q8, uint8_t* __restrict__ q4, float* __restrict__ s8_out,
                         float* __restrict__ s4_out, int8_t* __restrict__ q4e) {
    extern __shared__ __align__(16) float hrow[];  // [K]
    __shared__ float red[2][NT / 32];
    const int tid = threadIdx.x;
    const int nchunks = K >> 3, rchunks = r >> 3;
    const int K4 = K - r;
    const uint8_t* srow = reinterpret_cast<const uint8_t*>(hrow);
    for (size_t row = blockIdx.x; row < rows; row += gridDim.x) {
        // 1. widen the bf16 row (M = 1; otherwise the small factor below reads its groups straight from global memory)
        const uint4* xp = reinterpret_cast<const uint4*>(X + row * static_cast<size_t>(K));
        for (int c = tid; M == 1 && c < nchunks; c += NT) {
            const uint4 u = __ldg(xp + c);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
            float4 a, b;
            a.x = __uint_as_float(w[0] << 16); a.y = __uint_as_float(w[0] & 0xFFFF0000u);
            a.z = __uint_as_float(w[1] << 16); a.w = __uint_as_float(w[1] & 0xFFFF0000u);
            b.x = __uint_as_float(w[2] << 16); b.y = __uint_as_float(w[2] & 0xFFFF0000u);
            b.z = __uint_as_float(w[3] << 16); b.w = __uint_as_float(w[3] & 0xFFFF0000u);
            reinterpret_cast<float4*>(hrow)[2 * c] = a;
            reinterpret_cast<float4*>(hrow)[2 * c + 1] = b;
        }
        if constexpr (M == 1) __syncthreads();
        // 2. the small factor, one group of M consecutive coefficients per thread: bf16 from global memory (M * 2 bytes
        //    per group, a multiple of 8), fp32 result to the row buffer
        if constexpr (M > 1) {
            constexpr Conference<M> conf{};
            constexpr int H2 = M / 2;
            for (int a = tid; a < (K / M); a += NT) {
                // M * 4 bytes is a multiple of 16: the group moves as float4s (conflict-free at this stride)
                float4* gp = reinterpret_cast<float4*>(hrow + a * M);
                const uint2* xg = reinterpret_cast<const uint2*>(X + row * static_cast<size_t>(K) + static_cast<size_t>(a) * M);
                float x[M], y[M], ps[H2], ms[H2];
#pragma unroll
                for (int i = 0; i < M / 4; ++i) {
                    const uint2 u = __ldg(xg + i);
                    x[4 * i] = __uint_as_float(u.x << 16); x[4 * i + 1] = __uint_as_float(u.x & 0xFFFF0000u);
                    x[4 * i + 2] = __uint_as_float(u.y << 16); x[4 * i + 3] = __uint_as_float(u.y & 0xFFFF0000u);
                }
#pragma unroll
                for (int i = 0; i < H2; ++i) {
                    ps[i] = x[2 * i] + x[2 * i + 1];
                    ms[i] = x[2 * i] - x[2 * i + 1];
                }
                // S = [[0, 1^T], [1, Q]] with Q_ij = chi(i - j) circulant of order q = M / 2 - 1.  With t = sum of the
                // q inner entries and R_j = sum over the quadratic residues k of entry (j + k) mod q, the non-residues
                // sum to t - entry_j - R_j, so (Q v)_j = 2 R_j - t + v_j: (q - 1) / 2 + 2 operations instead of q - 1.
                constexpr int Q = H2 - 1;
                float tp = ps[1], tm = ms[1];
#pragma unroll
                for (int i = 2; i < H2; ++i) { tp += ps[i]; tm += ms[i]; }
                y[0] = ms[0] + tp;
                y[1] = tm - ps[0];
#pragma unroll
                for (int jp = 0; jp < Q; ++jp) {
                    float rp = 0.f, rm = 0.f;
#pragma unroll
                    for (int k = 1; k < Q; ++k) {
                        if (conf.s[1 + k][1] > 0) {  // chi(k) = +1
                            rp += ps[1 + (jp + k) % Q];
                            rm += ms[1 + (jp + k) % Q];
                        }
                    }
                    const float qp = fmaf(2.f, rp, ps[jp + 1] - tp), qm = fmaf(2.f, rm, ms[jp + 1] - tm);
                    y[2 * (jp + 1)] = (ms[jp + 1] + ps[0]) + qp;
                    y[2 * (jp + 1) + 1] = (ms[0] - ps[jp + 1]) + qm;
                }
#pragma unroll
                for (int i = 0; i < M / 4; ++i) gp[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
            }
            __syncthreads();
        }
        // 3. Sylvester butterflies over the index bits of a, up to five bits (32 values in registers) per pass.  With
        //    M = 1 a thread's values of the first pass are 2^nb consecutive words, i.e. the lanes of a warp sit 2^nb
        //    banks apart: three bits per pass there (an 8-way conflict on one pass instead of a 32-way one).
        constexpr int kMaxBits = M == 1 ? 3 : 5;
        float a8 = 0.f, a4 = 0.f;
        for (int s = 0; s < kbits;) {
            const int left = kbits - s;
            const int nb = left <= kMaxBits ? left : (left <= 2 * kMaxBits ? (left + 1) / 2 : kMaxBits);
            const bool last = s + nb >= kbits;
            if (nb == 1) butterfly_pass<M, NT, 1>(hrow, K, s, tid, last, inv_sqrt_k, r, a8, a4);
            else if (nb == 2) butterfly_pass<M, NT, 2>(hrow, K, s, tid, last, inv_sqrt_k, r, a8, a4);
            else if (nb == 3) butterfly_pass<M, NT, 3>(hrow, K, s, tid, last, inv_sqrt_k, r, a8, a4);
            else if constexpr (kMaxBits > 3) {
                if (nb == 4) butterfly_pass<M, NT, 4>(hrow, K, s, tid, last, inv_sqrt_k, r, a8, a4);
                else butterfly_pass<M, NT, 5>(hrow, K, s, tid, last, inv_sqrt_k, r, a8, a4);
            }
            s += nb;
            __syncthreads();
        }
        // 4. (no butterfly pass: K = M) scale and absmax in a pass of their own
        for (int c = tid; kbits == 0 && c < nchunks; c += NT) {
            float4* p = reinterpret_cast<float4*>(hrow) + 2 * c;
            float4 a = p[0], b = p[1];
            a.x *= inv_sqrt_k; a.y *= inv_sqrt_k; a.z *= inv_sqrt_k; a.w *= inv_sqrt_k;
            b.x *= inv_sqrt_k; b.y *= inv_sqrt_k; b.z *= inv_sqrt_k; b.w *= inv_sqrt_k;
            p[0] = a; p[1] = b;
            const float m = fmaxf(fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))),
                                  fmaxf(fmaxf(fabsf(b.x), fabsf(b.y)), fmaxf(fabsf(b.z), fabsf(b.w))));
            if (c < rchunks) a8 = fmaxf(a8, m);
            else a4 = fmaxf(a4, m);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a8 = fmaxf(a8, __shfl_xor_sync(0xffffffffu, a8, o));
            a4 = fmaxf(a4, __shfl_xor_sync(0xffffffffu, a4, o));
        }
        if ((tid & 31) == 0) {
            red[0][tid >> 5] = a8;
            red[1][tid >> 5] = a4;
        }
        __syncthreads();  // also: every thread's scaled values are in place
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) {
            a8 = fmaxf(a8, red[0][w]);
            a4 = fmaxf(a4, red[1][w]);
        }
        // 5. codes
        const float s8 = __fdiv_rn(a8, 127.f), s4 = __fdiv_rn(a4, 7.f);
        const float inv8 = s8 > 0.f ? __frcp_rn(s8) : 0.f, inv4 = s4 > 0.f ? __frcp_rn(s4) : 0.f;
        const bool exact8 = s8 > 0.f && !(inv8 >= 1.1754944e-38f && inv8 <= 3.0e38f);
        const bool exact4 = s4 > 0.f && !(inv4 >= 1.1754944e-38f && inv4 <= 3.0e38f);
        if (tid == 0) {
            s8_out[row] = s8;
            s4_out[row] = s4;
        }
        int8_t* q8row = q8 + row * static_cast<size_t>(r);
        uint8_t* q4row = q4 ? q4 + row * static_cast<size_t>(K4 >> 1) : nullptr;
        int8_t* q4e_row = q4e ? q4e + row * static_cast<size_t>(K4) : nullptr;
        for (int c = tid; c < nchunks; c += NT) {
            uint32_t t[8];
            const bool seg8 = c < rchunks;
            const float s = seg8 ? s8 : s4;
            if (s > 0.f) fast_codes(lds_chunk<true>(srow, c), s, seg8 ? inv8 : inv4, seg8 ? exact8 : exact4, t);
            else {
#pragma unroll
                for (int k = 0; k < 8; ++k) t[k] = 0;
            }
            const uint32_t w0 = pack_low_bytes(t[0], t[1], t[2], t[3]), w1 = pack_low_bytes(t[4], t[5], t[6], t[7]);
            if (seg8) {
                *reinterpret_cast<uint2*>(q8row + c * 8) = make_uint2(w0, w1);
            } else {
                const int jj = (c - rchunks) * 8;
                if (q4e_row) *reinterpret_cast<uint2*>(q4e_row + jj) = make_uint2(w0, w1);
                if (q4row) {
                    uint32_t packed = 0;
#pragma unroll
                    for (int k = 0; k < 8; ++k) packed |= (t[k] & 0xFu) << (4 * k);
                    *reinterpret_cast<uint32_t*>(q4row + (jj >> 1)) = packed;
                }
            }
        }
        __syncthreads();  // the row buffer is reused by the next row
    }
}

}  // namespace

cudaError_t launch_split_quantize(const void* in, bool in_is_f32, size_t rows, int K, int r, int8_t* q8,
                                  uint8_t* q4, void* s8, void* s4, bool scale_fp16, int8_t* q4_i8,
                                  size_t in_row_stride_bytes, cudaStream_t st, bool programmatic) {
    if (rows == 0) return cudaSuccess;
    const size_t row_bytes = static_cast<size_t>(K) * (in_is_f32 ? 4 : 2);
    if (!scale_fp16 && row_bytes <= static_cast<size_t>(kFastMaxRowBytes) && in_row_stride_bytes % 16 == 0) {
        int rpc = 1;  // rows per CTA and step: 1, 2, 4 or 8, about half of kFastGroupBytes of staging
        while (rpc < 8 && row_bytes * rpc * 2 <= static_cast<size_t>(kFastGroupBytes)) rpc *= 2;
        while (rpc > 1 && rows / rpc < 148) rpc /= 2;  // few rows (a generation step): all threads of a CTA on one row
        const size_t groups = (rows + rpc - 1) / rpc;
        const size_t group_bytes = row_bytes * rpc;
        // Two stages when they are cheap (several CTAs per SM still fit) and a CTA has more than one group to do.
        auto kern = in_is_f32 ? split_quantize_fast_kernel<true> : split_quantize_fast_kernel<false>;
        static bool attr_set[2][64] = {};
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 64 && !attr_set[in_is_f32][dev]) {
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kFastMaxRowBytes);
            if (e != cudaSuccess) return e;
            attr_set[in_is_f32][dev] = true;
        }
        auto ctas_per_sm = [](size_t smem) {  // shared memory and the 2048-thread limit; registers allow 8 CTAs of 256
            const size_t by_smem = (227u * 1024u) / (smem + 1024u);
            return by_smem < 1 ? size_t(1) : (by_smem > 8 ? size_t(8) : by_smem);
        };
        int nstages = 1;
        size_t grid = 148 * ctas_per_sm(group_bytes);
        if (groups > grid && 2 * group_bytes <= 64u * 1024u) {
            nstages = 2;
            grid = 148 * ctas_per_sm(2 * group_bytes);
        }
        if (grid > groups) grid = groups;
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
            cfg.blockDim = dim3(kThreads, 1, 1);
            cfg.dynamicSmemBytes = group_bytes * nstages;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            // The kernel waits for the preceding grid itself (griddepcontrol.wait on entry), so it may always be
            // scheduled while that grid drains; for the few rows of a generation step this hides most of its launch.
            (void)programmatic;
            cfg.numAttrs = 1;
            count_launch();
            return cudaLaunchKernelEx(&cfg, kern, in, in_row_stride_bytes, rows, K, r, rpc, nstages, q8, q4,
                                      static_cast<float*>(s8), static_cast<float*>(s4), q4_i8, device_status_ptr());
        }
    }
    const unsigned grid = static_cast<unsigned>(rows < 148u * 64u ? rows : 148u * 64u);
    count_launch();
    if (in_is_f32)
        split_quantize_kernel<true><<<grid, kThreads, 0, st>>>(in, in_row_stride_bytes, rows, K, r, q8, q4, s8, s4,
                                                               scale_fp16 ? 1 : 0, q4_i8);
    else
        split_quantize_kernel<false><<<grid, kThreads, 0, st>>>(in, in_row_stride_bytes, rows, K, r, q8, q4, s8, s4,
                                                                scale_fp16 ? 1 : 0, q4_i8);
    return cudaGetLastError();
}

cudaError_t launch_unpack_int4(const uint8_t* packed, int8_t* out, size_t rows, size_t cols, cudaStream_t st,
                               bool codes_unsigned) {
    const size_t nwords = rows * cols / 8;
    if (nwords == 0) return cudaSuccess;
    size_t blocks = (nwords + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    count_launch();
    if (codes_unsigned) unpack_int4_kernel<true><<<static_cast<unsigned>(blocks), 256, 0, st>>>(packed, out, nwords);
    else unpack_int4_kernel<false><<<static_cast<unsigned>(blocks), 256, 0, st>>>(packed, out, nwords);
    return cudaGetLastError();
}


// K = 2^k * m with m in {28, 12, 1} (largest first); false if K has no such form.
bool hadamard_factor(int K, int* kbits, int* m) {
    for (int mm : {28, 12, 1}) {
        if (K % mm) continue;
        const int a = K / mm;
        if (a & (a - 1)) continue;
        int kb = 0;
        while ((1 << kb) < a) ++kb;
        *kbits = kb;
        *m = mm;
        return true;
    }
    return false;
}

cudaError_t launch_hadamard_quantize(const void* X, size_t rows, int K, int r, int8_t* q8, uint8_t* q4, float* s8,
                                     float* s4, int8_t* q4_i8, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    int kbits = 0, m = 0;
    if (!hadamard_factor(K, &kbits, &m)) return cudaErrorNotSupported;
    const size_t smem = static_cast<size_t>(K) * 4;
    if (smem > 200u * 1024u) return cudaErrorNotSupported;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    static bool ready[64] = {};
    if (dev < 64 && !ready[dev]) {
        // Once per device: the shared-memory limit of the kernels.
        for (auto k : {hadamard_quantize_kernel<1, kThreads>, hadamard_quantize_kernel<12, kThreads>,
                       hadamard_quantize_kernel<28, kThreads>, hadamard_quantize_kernel<1, kWideThreads>,
                       hadamard_quantize_kernel<12, kWideThreads>, hadamard_quantize_kernel<28, kWideThreads>})
            if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess)
                return e;
        ready[dev] = true;
    }
    const float inv_sqrt_k = static_cast<float>(1.0 / sqrt(static_cast<double>(K)));
    const unsigned grid = static_cast<unsigned>(rows < 148u * 16u ? rows : 148u * 16u);
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(X);
    // 1024 threads per row only when rows do not outnumber the SMs: at 28672-wide rows (two 256-thread CTAs per SM)
    // the wide form measured slower for many rows (0.89 against 0.72 ms at 8192 rows).
    count_launch();
    if (rows <= kWideMaxRows) {
        if (m == 1) hadamard_quantize_kernel<1, kWideThreads><<<grid, kWideThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
        else if (m == 12) hadamard_quantize_kernel<12, kWideThreads><<<grid, kWideThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
        else hadamard_quantize_kernel<28, kWideThreads><<<grid, kWideThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
        return cudaGetLastError();
    }
    if (m == 1) hadamard_quantize_kernel<1, kThreads><<<grid, kThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
    else if (m == 12) hadamard_quantize_kernel<12, kThreads><<<grid, kThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
    else hadamard_quantize_kernel<28, kThreads><<<grid, kThreads, smem, st>>>(x, rows, K, kbits, r, inv_sqrt_k, q8, q4, s8, s4, q4_i8);
    return cudaGetLastError();
}

}  // namespace resq
