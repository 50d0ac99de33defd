// Attention-block path for d_head = 64 (Section 4.3, Eq. 8; Section 5.1): the same arithmetic and cache format as the
// d_head = 128 kernels -- 8-bit U_C projection of query and key, per-head asymmetric cache codes with the first
// d/8 = 8 coefficients in 8 bits and the other 56 in 4 -- written plainly: one warp per head vector, lane l owning
// coefficients l and l + 32, every division a true IEEE division.  Attention runs one warp per (query row, query
// head) with one cache position per lane and everything in fp32.  These kernels cover the small model geometry;
// the tuned paths (mma.sync single-query kernel, tcgen05 tile kernel) are those of d_head = 128.
//
// Block layout for d_head = 64 (the d = 128 layout with every code array halved): per half (key, then value)
//   c8 [32][8] | c4 [32][28] | meta [32][4] fp32      = 256 + 896 + 512 = 1664 bytes, 3328 per block.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"

namespace resq {
namespace {

constexpr int D = 64, R8 = D / 8, N4 = D - R8;
constexpr int kC8 = 32 * R8, kC4 = 32 * (N4 / 2), kHalf = kC8 + kC4 + 512, kBlock = 2 * kHalf;
constexpr int kWarps = 4;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// W_C [64][64] fp32 -> symmetric per-row INT8 codes and scales (one warp per row).
__global__ void __launch_bounds__(32) uc_quantize64_kernel(const float* __restrict__ W, int8_t* __restrict__ wq,
                                                           float* __restrict__ s_u) {
    const int row = blockIdx.x, lane = threadIdx.x;
    const float x0 = W[row * D + lane], x1 = W[row * D + lane + 32];
    const float m = warp_max(fmaxf(fabsf(x0), fabsf(x1)));
    const float s = __fdiv_rn(m, 127.f);
    int c0 = 0, c1 = 0;
    if (s > 0.f) {
        c0 = static_cast<int>(fminf(fmaxf(rintf(__fdiv_rn(x0, s)), -127.f), 127.f));
        c1 = static_cast<int>(fminf(fmaxf(rintf(__fdiv_rn(x1, s)), -127.f), 127.f));
    }
    wq[row * D + lane] = static_cast<int8_t>(c0);
    wq[row * D + lane + 32] = static_cast<int8_t>(c1);
    if (lane == 0) s_u[row] = s;
}

struct Project64Params {
    const __nv_bfloat16 *q, *k, *v;
    long long q_rows, kv_rows;  // head vectors
    __half* q_out;
    const int8_t* wq;
    const float* s_u;
    uint8_t* cache;
    int n_seqs, n_kv_heads, capacity;
    const int32_t *seq_ids, *positions;
    int* status;
};

// y = x U_C through the 8-bit product: lane l returns y[l] and y[l + 32].  xs: the warp's 64 code bytes in shared memory.
__device__ __forceinline__ void project64(float x0, float x1, const int8_t* wq_s, const float* s_u, int8_t* xs, int lane,
                                          float& y0, float& y1) {
    const float m = warp_max(fmaxf(fabsf(x0), fabsf(x1)));
    const float s = __fdiv_rn(m, 127.f);
    int c0 = 0, c1 = 0;
    if (s > 0.f) {
        c0 = static_cast<int>(rintf(__fdiv_rn(x0, s)));
        c1 = static_cast<int>(rintf(__fdiv_rn(x1, s)));
    }
    __syncwarp();
    xs[lane] = static_cast<int8_t>(c0);
    xs[lane + 32] = static_cast<int8_t>(c1);
    __syncwarp();
    const int* xw = reinterpret_cast<const int*>(xs);
    const int* w0 = reinterpret_cast<const int*>(wq_s + lane * D);
    const int* w1 = reinterpret_cast<const int*>(wq_s + (lane + 32) * D);
    int a0 = 0, a1 = 0;
#pragma unroll
    for (int i = 0; i < D / 4; ++i) {
        const int w = (i + lane) & (D / 4 - 1);  // rotated per lane: the lanes' rows are 16 words apart
        const int xi = xw[w];
        a0 = __dp4a(xi, w0[w], a0);
        a1 = __dp4a(xi, w1[w], a1);
    }
    y0 = __fmul_rn(static_cast<float>(a0), __fmul_rn(s, s_u[lane]));
    y1 = __fmul_rn(static_cast<float>(a1), __fmul_rn(s, s_u[lane + 32]));
}

// Asymmetric codes of one head vector (lane l holds coefficients l and l + 32) written at `half_base` (the key or
// value half of a cache block), slot p.
__device__ __forceinline__ void quantize_store64(float y0, float y1, uint8_t* half_base, int p, int lane) {
    const bool in8 = lane < R8;  // coefficient `lane` is in the 8-bit segment; `lane + 32` never is
    const float lo8 = warp_min(in8 ? y0 : INFINITY), hi8 = warp_max(in8 ? y0 : -INFINITY);
    const float lo4 = warp_min(in8 ? y1 : fminf(y0, y1)), hi4 = warp_max(in8 ? y1 : fmaxf(y0, y1));
    const float s8 = __fdiv_rn(__fsub_rn(hi8, lo8), 255.f), s4 = __fdiv_rn(__fsub_rn(hi4, lo4), 15.f);
    auto code = [](float x, float z, float s, float qmax) -> uint32_t {
        if (!(s > 0.f)) return 0u;
        return static_cast<uint32_t>(fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(x, z), s)), 0.f), qmax));
    };
    const uint32_t c0 = in8 ? code(y0, lo8, s8, 255.f) : code(y0, lo4, s4, 15.f);
    const uint32_t c1 = code(y1, lo4, s4, 15.f);
    // 4-bit coefficient j sits at u = j - 8: byte u / 2, low nibble for even u.  u has the parity of the lane.
    const uint32_t n0 = __shfl_down_sync(0xffffffffu, c0, 1), n1 = __shfl_down_sync(0xffffffffu, c1, 1);
    uint8_t* c8 = half_base + p * R8;
    uint8_t* c4 = half_base + kC8 + p * (N4 / 2);
    if (in8) {
        c8[lane] = static_cast<uint8_t>(c0);
    } else if ((lane & 1) == 0) {
        c4[(lane - R8) >> 1] = static_cast<uint8_t>(c0 | (n0 << 4));
    }
    if ((lane & 1) == 0) c4[(lane + 32 - R8) >> 1] = static_cast<uint8_t>(c1 | (n1 << 4));
    if (lane == 0) *reinterpret_cast<float4*>(half_base + kC8 + kC4 + p * 16) = make_float4(s8, lo8, s4, lo4);
}

__global__ void __launch_bounds__(kWarps * 32) project_append64_kernel(const Project64Params p) {
    __shared__ __align__(16) int8_t wq_s[D * D];
    __shared__ float su_s[D];
    __shared__ __align__(16) int8_t xs[kWarps][D];
    for (int i = threadIdx.x; i < D * D / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(wq_s)[i] = __ldg(reinterpret_cast<const uint4*>(p.wq) + i);
    for (int i = threadIdx.x; i < D; i += blockDim.x) su_s[i] = p.s_u[i];
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = p.q_rows + 2 * p.kv_rows;
    for (long long item = static_cast<long long>(blockIdx.x) * kWarps + warp; item < total;
         item += static_cast<long long>(gridDim.x) * kWarps) {
        const int kind = item < p.q_rows ? 0 : item < p.q_rows + p.kv_rows ? 1 : 2;  // query, key, value
        const long long row = kind == 0 ? item : kind == 1 ? item - p.q_rows : item - p.q_rows - p.kv_rows;
        const __nv_bfloat16* src = (kind == 0 ? p.q : kind == 1 ? p.k : p.v) + row * D;
        const float x0 = __bfloat162float(src[lane]), x1 = __bfloat162float(src[lane + 32]);
        float y0 = x0, y1 = x1;
        if (kind != 2) project64(x0, x1, wq_s, su_s, xs[warp], lane, y0, y1);
        if (kind == 0) {
            p.q_out[row * D + lane] = __float2half_rn(y0);
            p.q_out[row * D + lane + 32] = __float2half_rn(y1);
            continue;
        }
        const long long t = row / p.n_kv_heads;
        const int h = static_cast<int>(row - t * p.n_kv_heads);
        const int b = p.seq_ids[t], pos = p.positions[t];
        if (b < 0 || b >= p.n_seqs || pos < 0 || pos >= p.capacity) {
            if (lane == 0) atomicOr(p.status, kStatusBitIndex);
            continue;
        }
        const size_t blk = (static_cast<size_t>(b) * p.n_kv_heads + h) * (p.capacity / RESQ_KV_BLOCK) + pos / RESQ_KV_BLOCK;
        quantize_store64(y0, y1, p.cache + blk * kBlock + (kind == 2 ? kHalf : 0), pos % RESQ_KV_BLOCK, lane);
    }
}

struct Attn64Params {
    const uint8_t* cache;
    const __half* q;   // [rows][Hq][64]
    float* out;
    int rows, Hq, Hkv, n_seqs, capacity;
    const int32_t* seq_of_row;  // null: seq_const if >= 0, else the row index
    const int32_t* len_of_row;  // null: len0 + row + 1
    int seq_const, len0;
    int* status;
};

// One warp per (row, query head): 32 cache positions at a time, one per lane for the scores, then coefficient-owning
// lanes (l and l + 32) for the weighted sum of the dequantized values.  Softmax is the running-maximum form in fp32.
__global__ void __launch_bounds__(kWarps * 32) attention64_kernel(const Attn64Params p) {
    __shared__ float qs[kWarps][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long item = static_cast<long long>(blockIdx.x) * kWarps + warp;
    if (item >= static_cast<long long>(p.rows) * p.Hq) return;
    const int row = static_cast<int>(item / p.Hq), hq = static_cast<int>(item % p.Hq);
    const int kvh = hq / (p.Hq / p.Hkv);
    float* dst = p.out + item * D;
    int b = p.seq_of_row ? p.seq_of_row[row] : (p.seq_const >= 0 ? p.seq_const : row);
    int len = p.len_of_row ? p.len_of_row[row] : p.len0 + row + 1;
    if (b < 0 || b >= p.n_seqs) {
        if (lane == 0) atomicOr(p.status, kStatusBitIndex);
        b = 0;
        len = 0;
    }
    if (len < 0 || len > p.capacity) {
        if (lane == 0) atomicOr(p.status, kStatusBitIndex);
        len = len < 0 ? 0 : p.capacity;
    }
    qs[warp][lane] = __half2float(p.q[item * D + lane]);
    qs[warp][lane + 32] = __half2float(p.q[item * D + lane + 32]);
    __syncwarp();
    const float* qv = qs[warp];
    const uint8_t* blocks = p.cache + (static_cast<size_t>(b) * p.Hkv + kvh) * (p.capacity / RESQ_KV_BLOCK) * kBlock;
    float m = -INFINITY, l = 0.f, acc0 = 0.f, acc1 = 0.f;
    for (int j0 = 0; j0 < len; j0 += 32) {
        const uint8_t* blk = blocks + static_cast<size_t>(j0 / 32) * kBlock;
        // score of position j0 + lane
        float sc = -INFINITY;
        if (j0 + lane < len) {
            const float4 km = *reinterpret_cast<const float4*>(blk + kC8 + kC4 + lane * 16);
            const uint8_t* c8 = blk + lane * R8;
            const uint8_t* c4 = blk + kC8 + lane * (N4 / 2);
            float dot = 0.f;
#pragma unroll
            for (int i = 0; i < R8; ++i) dot = fmaf(qv[i], fmaf(static_cast<float>(c8[i]), km.x, km.y), dot);
#pragma unroll
            for (int i = 0; i < N4 / 2; ++i) {
                const uint32_t by = c4[i];
                dot = fmaf(qv[R8 + 2 * i], fmaf(static_cast<float>(by & 15u), km.z, km.w), dot);
                dot = fmaf(qv[R8 + 2 * i + 1], fmaf(static_cast<float>(by >> 4), km.z, km.w), dot);
            }
            sc = dot * 0.125f;  // 1 / sqrt(64)
        }
        const float m_new = fmaxf(m, warp_max(sc));
        const float corr = __expf(m - m_new);  // 0 on the first block (m = -inf)
        const float pj = j0 + lane < len ? __expf(sc - m_new) : 0.f;
        l = l * corr + warp_sum(pj);
        acc0 *= corr;
        acc1 *= corr;
        m = m_new;
        // values: lane owns coefficients lane and lane + 32
        const uint8_t* vb = blk + kHalf;
        const int n = min(32, len - j0);
        for (int j = 0; j < n; ++j) {
            const float pw = __shfl_sync(0xffffffffu, pj, j);
            const float4 vm = *reinterpret_cast<const float4*>(vb + kC8 + kC4 + j * 16);
            float v0;
            if (lane < R8) {
                v0 = fmaf(static_cast<float>(vb[j * R8 + lane]), vm.x, vm.y);
            } else {
                const uint32_t by = vb[kC8 + j * (N4 / 2) + ((lane - R8) >> 1)];
                v0 = fmaf(static_cast<float>((lane & 1) ? by >> 4 : by & 15u), vm.z, vm.w);
            }
            const uint32_t by1 = vb[kC8 + j * (N4 / 2) + ((lane + 32 - R8) >> 1)];
            const float v1 = fmaf(static_cast<float>((lane & 1) ? by1 >> 4 : by1 & 15u), vm.z, vm.w);
            acc0 = fmaf(pw, v0, acc0);
            acc1 = fmaf(pw, v1, acc1);
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    dst[lane] = acc0 * inv;
    dst[lane + 32] = acc1 * inv;
}

}  // namespace

size_t kv64_block_bytes() { return kBlock; }

cudaError_t launch_uc_quantize64(const float* W_C, int8_t* wq, float* s_u, cudaStream_t st) {
    count_launch();
    uc_quantize64_kernel<<<D, 32, 0, st>>>(W_C, wq, s_u);
    return cudaGetLastError();
}

cudaError_t launch_qkv_project_append64(const resq_kv_cache_t* cache, const void* q, long long q_rows, void* q_out,
                                        const void* k, const void* v, long long T, const int32_t* seq_ids,
                                        const int32_t* positions, const int8_t* wq, const float* s_u, cudaStream_t st) {
    Project64Params p{};
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
    const long long total = p.q_rows + 2 * p.kv_rows;
    if (total == 0) return cudaSuccess;
    const long long ctas = (total + kWarps - 1) / kWarps;
    count_launch();
    project_append64_kernel<<<static_cast<unsigned>(ctas < 148 * 8 ? ctas : 148 * 8), kWarps * 32, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_attention64(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, int rows,
                               const int32_t* seq_of_row, const int32_t* len_of_row, int seq_const, int len0, float* out,
                               cudaStream_t st) {
    Attn64Params p{};
    p.cache = static_cast<const uint8_t*>(cache.data);
    p.q = static_cast<const __half*>(q16);
    p.out = out;
    p.rows = rows;
    p.Hq = n_q_heads;
    p.Hkv = cache.n_kv_heads;
    p.n_seqs = cache.n_seqs;
    p.capacity = cache.capacity;
    p.seq_of_row = seq_of_row;
    p.len_of_row = len_of_row;
    p.seq_const = seq_const;
    p.len0 = len0;
    p.status = device_status_ptr();
    const long long items = static_cast<long long>(rows) * n_q_heads;
    count_launch();
    attention64_kernel<<<static_cast<unsigned>((items + kWarps - 1) / kWarps), kWarps * 32, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace resq
