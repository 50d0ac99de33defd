// Attention-block path, cache side (Section 4.3, Eq. 8; Section 5.1): the 8-bit online U_C projection of query
// and key head vectors, and the per-head asymmetric 8/4-bit quantizer that writes key and value into the
// blocked cache.  HBM-light (a few MB per call); the contraction is 128 wide, so it runs on mma.sync s8
// fragments taken straight from the global loads -- a head vector never touches shared memory before its
// codes do.
//
// One warp owns 16 consecutive head vectors (rows).  Lane (g, c) = (lane / 4, lane % 4) loads, for rows g and
// g + 8, the elements [32 ks + 4c, +4) and [32 ks + 16 + 4c, +4), ks = 0..3: exactly the bytes of its A
// fragments of mma.m16n8k32, and 32 contiguous bytes per quad, so every sector fetched is used.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"
#include "../../include/resq_kv.h"

namespace resq {
namespace {

constexpr int kD = 128;
constexpr int kWStride = 144;  // bytes per staged W_C row: 36 words, so the 8 rows of a B fragment hit 8 bank groups
constexpr int kWarps = 4;
constexpr int kRec = 88;       // staged record of one head vector: 16 + 56 code bytes, 4 floats
constexpr float kMagic = 12582912.f;  // 1.5 * 2^23

// round-half-even(x / s) with the IEEE quotient's rounding: the product with inv = RN(1/s) lies within 2^-15
// (|q| <= 127) / 2^-14 (|q| <= 255) of the quotient, so the two can only round apart when the product is that
// close to a half-integer; there the true division decides.
__device__ __forceinline__ float code_rn(float x, float s, float inv, bool exact_only, float guard) {
    const float tf = fmaf(x, inv, kMagic);
    const float q = tf - kMagic;
    const float res = fabsf(fmaf(x, inv, -q));
    if (exact_only || !(res < guard)) return rintf(__fdiv_rn(x, s));
    return q;
}
__device__ __forceinline__ bool needs_division(float inv) { return !(inv >= 1.1754944e-38f && inv <= 3.0e38f); }

__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The lane's 32 elements of one row as fp32: v[8 ks + i] = x[32 ks + 4c + i], v[8 ks + 4 + i] = x[32 ks + 16 + 4c + i].
__device__ __forceinline__ void load_row(const __nv_bfloat16* row, int c, bool live, float (&v)[32]) {
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            uint2 u = make_uint2(0u, 0u);
            if (live) u = __ldg(reinterpret_cast<const uint2*>(row + 32 * ks + 16 * hf + 4 * c));
            float* o = v + 8 * ks + 4 * hf;
            o[0] = __uint_as_float(u.x << 16); o[1] = __uint_as_float(u.x & 0xFFFF0000u);
            o[2] = __uint_as_float(u.y << 16); o[3] = __uint_as_float(u.y & 0xFFFF0000u);
        }
}

__device__ __forceinline__ float quad_max(float v) {
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_min(float v) {
    v = fminf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fminf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}

// Asymmetric parameters of one segment from its (min, max): s, 1/s, whether the division must be used.
struct Asym {
    float z, s, inv;
    bool exact;
    __device__ __forceinline__ Asym(float lo, float hi, float qmax) {
        z = lo;
        s = __fdiv_rn(__fsub_rn(hi, lo), qmax);
        inv = s > 0.f ? __frcp_rn(s) : 0.f;
        exact = needs_division(inv);
    }
    __device__ __forceinline__ uint32_t code(float x, float qmax) const {
        if (!(s > 0.f)) return 0u;
        const float q = code_rn(__fsub_rn(x, z), s, inv, exact, 0.5f - 0.00006103515625f);
        return static_cast<uint32_t>(fminf(fmaxf(q, 0.f), qmax));
    }
};

// Where the record of head vector `row` goes: (block index) * 32 + slot in the block, or -1.
__device__ __forceinline__ long long cache_slot(long long row, int n_kv_heads, int n_seqs, int capacity,
                                                const int32_t* seq_ids, const int32_t* positions, int* status) {
    const long long t = row / n_kv_heads;
    const int h = static_cast<int>(row - t * n_kv_heads);
    const int b = seq_ids[t], pos = positions[t];
    if (b < 0 || b >= n_seqs || pos < 0 || pos >= capacity) {
        atomicOr(status, kStatusBitIndex);
        return -1;
    }
    const long long blk = (static_cast<long long>(b) * n_kv_heads + h) * (capacity / RESQ_KV_BLOCK) + pos / RESQ_KV_BLOCK;
    return blk * RESQ_KV_BLOCK + (pos % RESQ_KV_BLOCK);
}

// Copies the 16 staged records of a warp tile into the cache blocks (key: half 0, value: half 1).
__device__ __forceinline__ void flush_records(const uint8_t* rec, const long long* slot, uint8_t* cache, int half,
                                              int lane) {
    for (int u = lane; u < 16 * 11; u += 32) {
        const int row = u / 11, part = u - row * 11;  // 8-byte units: 0-1 codes8, 2-8 codes4, 9-10 scales
        const long long sl = slot[row];
        if (sl < 0) continue;
        uint8_t* blk = cache + (sl / RESQ_KV_BLOCK) * RESQ_KV_BLOCK_BYTES + half * 2816;
        const int p = static_cast<int>(sl % RESQ_KV_BLOCK);
        uint8_t* dst = part < 2 ? blk + p * 16 + part * 8
                     : part < 9 ? blk + 512 + p * 56 + (part - 2) * 8
                                : blk + 2304 + p * 16 + (part - 9) * 8;
        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(rec + row * kRec + part * 8);
    }
}

// Symmetric INT8 codes of the lane's part of two rows, packed as the A fragments a[ks][0..3]; returns the scales.
__device__ __forceinline__ void sym8_fragments(const float (&xv)[2][32], uint32_t (&a)[4][4], float (&sx)[2]) {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(xv[rr][i]));
        m = quad_max(m);
        const float s = __fdiv_rn(m, 127.f);
        const float inv = s > 0.f ? __frcp_rn(s) : 0.f;
        const bool exact = needs_division(inv);
        sx[rr] = s;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t w = 0;
                if (s > 0.f) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float q = code_rn(xv[rr][8 * ks + 4 * hf + i], s, inv, exact, 0.5f - 0.000030517578125f);
                        w |= (static_cast<uint32_t>(static_cast<int>(q)) & 0xFFu) << (8 * i);
                    }
                }
                a[ks][2 * hf + rr] = w;  // a0: row g, k 4c..; a1: row g+8; a2: row g, k 16+4c..; a3: row g+8
            }
    }
}

struct ProjectParams {
    const __nv_bfloat16* q;  // [q_rows][128] or null
    const __nv_bfloat16* k;  // [kv_rows][128] or null
    const __nv_bfloat16* v;
    long long q_rows, kv_rows;
    const int8_t* wq;
    const float* s_u;
    __half* q_out;
    uint8_t* cache;
    int n_seqs, n_kv_heads, capacity;
    const int32_t* seq_ids;
    const int32_t* positions;
    int* status;
};

// Asymmetric 8/4-bit codes of one row held by a quad: the lane's n8 values of the 8-bit segment and n4 of the
// 4-bit one.  Returns the two quantizers (min / max reduced over the quad).
template <int N8, int N4>
__device__ __forceinline__ void quad_ranges(const float* v8, const float* v4, float (&lohi)[4]) {
    float lo8 = 3.402823466e38f, hi8 = -3.402823466e38f, lo4 = lo8, hi4 = hi8;
#pragma unroll
    for (int i = 0; i < N8; ++i) { lo8 = fminf(lo8, v8[i]); hi8 = fmaxf(hi8, v8[i]); }
#pragma unroll
    for (int i = 0; i < N4; ++i) { lo4 = fminf(lo4, v4[i]); hi4 = fmaxf(hi4, v4[i]); }
    lohi[0] = quad_min(lo8); lohi[1] = quad_max(hi8); lohi[2] = quad_min(lo4); lohi[3] = quad_max(hi4);
}

// One warp per tile of 16 head vectors; the tiles of a call are the query tiles (projected, written as half),
// then the key tiles (projected, quantized, appended), then the value tiles (quantized, appended) -- three
// independent kinds, so a generation step's few tiles spread over as many warps and run side by side.
__global__ void __launch_bounds__(kWarps * 32) kv_project_kernel(const ProjectParams p) {
    __shared__ __align__(16) uint8_t w_s[kD * kWStride];
    __shared__ float su_s[kD];
    __shared__ __align__(16) uint8_t rec_s[kWarps][16 * kRec];
    __shared__ long long slot_s[kWarps][16];
    for (int i = threadIdx.x; i < kD * 8; i += blockDim.x) {  // 16-byte pieces of W_C's codes
        const int n = i >> 3, pc = i & 7;
        *reinterpret_cast<uint4*>(w_s + n * kWStride + pc * 16) = __ldg(reinterpret_cast<const uint4*>(p.wq + n * kD) + pc);
    }
    for (int i = threadIdx.x; i < kD; i += blockDim.x) su_s[i] = p.s_u[i];
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const long long q_tiles = (p.q_rows + 15) / 16, kv_tiles = (p.kv_rows + 15) / 16, tiles = q_tiles + 2 * kv_tiles;
    uint8_t* rec = rec_s[warp];
    for (long long tile = static_cast<long long>(blockIdx.x) * kWarps + warp; tile < tiles;
         tile += static_cast<long long>(gridDim.x) * kWarps) {
        const int kind = tile < q_tiles ? 0 : (tile < q_tiles + kv_tiles ? 1 : 2);  // query, key, value
        const long long t0 = kind == 0 ? tile : (kind == 1 ? tile - q_tiles : tile - q_tiles - kv_tiles);
        const long long rows = kind == 0 ? p.q_rows : p.kv_rows;
        const __nv_bfloat16* x = kind == 0 ? p.q : (kind == 1 ? p.k : p.v);
        const long long r0 = t0 * 16 + g, r1 = r0 + 8;
        const bool live0 = r0 < rows, live1 = r1 < rows;
        float xv[2][32];
        load_row(x + r0 * kD, c, live0, xv[0]);
        load_row(x + r1 * kD, c, live1, xv[1]);
        if (kind != 0 && lane < 16) {
            const long long r = t0 * 16 + lane;
            slot_s[warp][lane] = r < rows ? cache_slot(r, p.n_kv_heads, p.n_seqs, p.capacity, p.seq_ids, p.positions, p.status) : -1;
        }
        if (kind == 2) {
            // ---- value: the bf16 head vectors quantized directly; elements 0-3 of the lane are columns
            // [4c, 4c + 4), the 8-bit segment
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                float lohi[4];
                quad_ranges<4, 28>(xv[rr], xv[rr] + 4, lohi);
                const Asym q8(lohi[0], lohi[1], 255.f), q4(lohi[2], lohi[3], 15.f);
                uint8_t* rrow = rec + (g + 8 * rr) * kRec;
                uint32_t w8 = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) w8 |= q8.code(xv[rr][i], 255.f) << (8 * i);
                *reinterpret_cast<uint32_t*>(rrow + 4 * c) = w8;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        if (ks == 0 && hf == 0) continue;
                        const float* e = xv[rr] + 8 * ks + 4 * hf;
                        const int col = 32 * ks + 16 * hf + 4 * c;  // >= 16
                        *reinterpret_cast<uint16_t*>(rrow + 16 + (col - 16) / 2) = static_cast<uint16_t>(
                            q4.code(e[0], 15.f) | (q4.code(e[1], 15.f) << 4) | (q4.code(e[2], 15.f) << 8) | (q4.code(e[3], 15.f) << 12));
                    }
                if (c == 0) {
                    float* m = reinterpret_cast<float*>(rrow + 72);
                    m[0] = q8.s; m[1] = q8.z; m[2] = q4.s; m[3] = q4.z;
                }
            }
            __syncwarp();
            flush_records(rec, slot_s[warp], p.cache, 1, lane);
            __syncwarp();
            continue;
        }
        float sx[2];
        uint32_t a[4][4];
        sym8_fragments(xv, a, sx);
        // ---- y = x W_C^T: 16 column tiles of 8, exact int32
        int acc[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0;
            const uint8_t* wrow = w_s + (8 * nt + g) * kWStride + 4 * c;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                mma_s8(acc[nt], a[ks], *reinterpret_cast<const uint32_t*>(wrow + 32 * ks),
                       *reinterpret_cast<const uint32_t*>(wrow + 32 * ks + 16));
        }
        // y[row g][8 nt + 2c + e] = acc[nt][e], y[row g + 8][...] = acc[nt][2 + e]
        if (kind == 0) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) {
                const float u0 = su_s[8 * nt + 2 * c], u1 = su_s[8 * nt + 2 * c + 1];
                if (live0)
                    *reinterpret_cast<__half2*>(p.q_out + r0 * kD + 8 * nt + 2 * c) = __floats2half2_rn(
                        __fmul_rn(static_cast<float>(acc[nt][0]), __fmul_rn(sx[0], u0)),
                        __fmul_rn(static_cast<float>(acc[nt][1]), __fmul_rn(sx[0], u1)));
                if (live1)
                    *reinterpret_cast<__half2*>(p.q_out + r1 * kD + 8 * nt + 2 * c) = __floats2half2_rn(
                        __fmul_rn(static_cast<float>(acc[nt][2]), __fmul_rn(sx[1], u0)),
                        __fmul_rn(static_cast<float>(acc[nt][3]), __fmul_rn(sx[1], u1)));
            }
            continue;
        }
        // ---- key: asymmetric 8/4-bit codes of the fp32 coefficients (column tiles 0-1 are the 8-bit segment)
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            float y[32];  // y[2 nt + e]
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    y[2 * nt + e] = __fmul_rn(static_cast<float>(acc[nt][2 * rr + e]), __fmul_rn(sx[rr], su_s[8 * nt + 2 * c + e]));
            float lohi[4];
            quad_ranges<4, 28>(y, y + 4, lohi);
            const Asym q8(lohi[0], lohi[1], 255.f), q4(lohi[2], lohi[3], 15.f);
            uint8_t* rrow = rec + (g + 8 * rr) * kRec;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
                *reinterpret_cast<uint16_t*>(rrow + 8 * nt + 2 * c) =
                    static_cast<uint16_t>(q8.code(y[2 * nt], 255.f) | (q8.code(y[2 * nt + 1], 255.f) << 8));
#pragma unroll
            for (int nt = 2; nt < 16; ++nt)
                rrow[16 + 4 * (nt - 2) + c] = static_cast<uint8_t>(q4.code(y[2 * nt], 15.f) | (q4.code(y[2 * nt + 1], 15.f) << 4));
            if (c == 0) {
                float* m = reinterpret_cast<float*>(rrow + 72);
                m[0] = q8.s; m[1] = q8.z; m[2] = q4.s; m[3] = q4.z;
            }
        }
        __syncwarp();
        flush_records(rec, slot_s[warp], p.cache, 0, lane);
        __syncwarp();
    }
}

// W_C = U_C^T [d][d] fp32 -> symmetric per-row INT8 (one warp per row; offline, true divisions).
__global__ void __launch_bounds__(32) uc_quantize_kernel(const float* __restrict__ W, int8_t* __restrict__ wq,
                                                         float* __restrict__ s_u) {
    const int row = blockIdx.x, lane = threadIdx.x;
    const float4 x = reinterpret_cast<const float4*>(W + row * kD)[lane];
    float m = fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float s = __fdiv_rn(m, 127.f);
    const float in[4] = {x.x, x.y, x.z, x.w};
    uint32_t w = 0;
    if (s > 0.f)
#pragma unroll
        for (int i = 0; i < 4; ++i)
            w |= (static_cast<uint32_t>(static_cast<int>(fminf(fmaxf(rintf(__fdiv_rn(in[i], s)), -127.f), 127.f))) & 0xFFu)
                 << (8 * i);
    reinterpret_cast<uint32_t*>(wq + row * kD)[lane] = w;
    if (lane == 0) s_u[row] = s;
}

int grid_for(long long tiles) {
    const long long ctas = (tiles + kWarps - 1) / kWarps;
    return static_cast<int>(ctas < 148 * 8 ? (ctas > 0 ? ctas : 1) : 148 * 8);
}

cudaError_t launch_project(const ProjectParams& p, cudaStream_t st) {
    const long long tiles = (p.q_rows + 15) / 16 + 2 * ((p.kv_rows + 15) / 16);
    if (tiles == 0) return cudaSuccess;
    count_launch();
    kv_project_kernel<<<grid_for(tiles), kWarps * 32, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_uc_quantize(const float* W_C, int8_t* wq, float* s_u, cudaStream_t st) {
    count_launch();
    uc_quantize_kernel<<<kD, 32, 0, st>>>(W_C, wq, s_u);
    return cudaGetLastError();
}

// q (q_rows head vectors) and / or k, v (T tokens) in one launch; either part may be absent (null / 0).
cudaError_t launch_qkv_project_append(const resq_kv_cache_t* cache, const void* q, long long q_rows, void* q_out,
                                      const void* k, const void* v, long long T, const int32_t* seq_ids,
                                      const int32_t* positions, const int8_t* wq, const float* s_u, cudaStream_t st) {
    ProjectParams p{};
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.q_rows = q ? q_rows : 0;
    p.q_out = static_cast<__half*>(q_out);
    p.wq = wq;
    p.s_u = s_u;
    p.status = device_status_ptr();
    if (cache && k) {
        p.k = static_cast<const __nv_bfloat16*>(k);
        p.v = static_cast<const __nv_bfloat16*>(v);
        p.kv_rows = T * cache->n_kv_heads;
        p.cache = static_cast<uint8_t*>(cache->data);
        p.n_seqs = cache->n_seqs;
        p.n_kv_heads = cache->n_kv_heads;
        p.capacity = cache->capacity;
        p.seq_ids = seq_ids;
        p.positions = positions;
    }
    return launch_project(p, st);
}

}  // namespace resq
