// Causal attention of a run of new tokens over the quantized KV cache (Section 4.3, Eq. 8; cache format of
// Section 5.1) on the tcgen05 tensor cores: the prefill form, where every cache block is read once per tile of
// 128 (token, query head) rows instead of once per query.
//
// One CTA of 256 threads owns 128 rows that share a KV head -- 128 / g consecutive tokens times the g query heads
// of the group -- and walks the cache of its sequence in steps of 64 positions (two cache blocks, brought in whole
// by bulk copies, double buffered).  Two threads share a row: thread (row, h) handles the 32 positions of cache
// block h of the step; their partial maxima and sums meet in shared memory between the passes and at the end.
// Two CTAs fit on an SM (256 TMEM columns and about 108 KB of shared memory each), so one's tensor-core work and
// waits overlap the other's expansion and softmax arithmetic.  Per step:
//   keys     the 8-bit and 4-bit CODES are expanded to fp16 integers (exact) into a K-major operand tile; the
//            tensor core forms S8 = Q[:, :16]·C8^T and S4 = Q[:, 16:]·C4^T as two TMEM accumulators, and the thread
//            that owns a row applies the per-position scales and zero-points in fp32:
//                score = (s8·S8 + z8·sum(q[:16]) + s4·S4 + z4·sum(q[16:])) / sqrt(d).
//   softmax  fp32 (TMEM lane = row).  Two passes over the cache: the first finds each row's maximum score (and the
//            tile's largest value scale, for the normalisation below), the second forms p = exp(score - max), so the
//            output accumulator never has to be rescaled.  Steps that lie wholly below the tile's first position
//            skip the causal comparison.
//   values   P8' = half(p · s8_v · 2^-E) and P4' = half(p · s4_v · 2^-E) are written as two K-major operand tiles
//            (2^E = the tile's largest value scale rounded down to a power of two, so the products stay in half's
//            normal range), the value codes are expanded, transposed, into an operand tile [coefficient][position],
//            (centred: code - 128, code - 8) and the tensor core accumulates O[:, :16] += P8'·C8v,
//            O[:, 16:] += P4'·C4v in TMEM.  The zero-points (plus the centres times the scales) enter as
//            sum_j p_j (z_j + c0 s_j) per segment, in registers.
//   out      (O · 2^E + zero-point sums) / sum_j p_j, fp32.
// The contraction index of the score product and the output columns are stored in a fixed permutation of the
// coefficients inside every group of eight (so that one shift-and-mask of a 32-bit word of nibbles yields two
// neighbouring tile elements); the query tile is written in the same permutation and the output is un-permuted on
// the way out.
// Positions beyond a row's own position are masked by selection (never by multiplying), so unwritten cache
// positions of a loaded block may hold anything.  All waits are bounded; on a failed wait every thread leaves
// through the same path, which frees the TMEM columns.
#include "internal.h"
#include "ptx.cuh"

#include <cuda_fp16.h>

namespace resq {
namespace {

constexpr int kRows = 128;          // (token, head) rows per CTA = TMEM lanes
constexpr int kStep = 64;           // cache positions per step
constexpr int kBlockBytes = RESQ_KV_BLOCK_BYTES;
constexpr int kOffK4 = 512, kOffKm = 2304, kOffV8 = 2816, kOffV4 = 3328, kOffVm = 5120;
constexpr int kKeyBytes = 2816;     // k8 + k4 + km of one block
constexpr int kMetaBytes = 512;
constexpr int kQBytes = 2 * kRows * 128;  // two 64-coefficient halves of [128 rows][128 B]
constexpr int kKVBytes = 16384;           // keys [64 pos][128 coef] (two halves) or values [128 coef][64 pos]
constexpr int kPBytes = 16384;            // [128 rows][64 pos]
constexpr int kRawBytes = 2 * kBlockBytes;
constexpr uint32_t kTmemCols = 256;       // S8: 0..63, S4: 64..127, O: 128..255
constexpr int kThreads = 256;

struct Shared {
    float4 colK[kStep];    // per position of the step: key (s8, z8, s4, z4) times log2(e) / sqrt(d)
    float4 colV[kStep];    // value (s8 2^-E, z8 + 128 s8, s4 2^-E, z4 + 8 s4)
    float xch[3][2][kRows];  // partial results of the two threads of a row
    float vmax[kStep];
    uint64_t load[2];
    uint64_t mma;
    uint32_t tmem_base;
    int abort_flag;
};

constexpr size_t kSmemBytes = 1024 + kQBytes + kKVBytes + 2 * kPBytes + 2 * kRawBytes + sizeof(Shared);

struct PrefillParams {
    const uint8_t* blocks;  // first cache block of the sequence (KV head 0)
    size_t head_stride;     // bytes between the KV heads of the sequence
    const __half* q;        // [T][Hq][128]
    float* out;             // [T][Hq][128]
    int T, Hq, g, pos0;
    int* status;
};

__host__ __device__ constexpr uint32_t make_idesc_f16(int M, int N) {  // f16 x f16 -> f32, K-major A and B
    return (1u << 4) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// Two bytes of w (selected by SEL, a prmt selector whose odd bytes pick the constant 0x64) as two halves holding
// the integers exactly.
// BIAS is the half bit pattern of 1024 + c0: the result is the code minus c0 (0x6400: the code itself).
template <uint32_t SEL, uint16_t BIAS = 0x6400>
__device__ __forceinline__ uint32_t bytes_to_h2(uint32_t w) {
    const uint32_t biased = __byte_perm(w, 0x64646464u, SEL);  // 1024 + byte in each half
    const __half2 v = __hsub2(*reinterpret_cast<const __half2*>(&biased), __half2half2(__ushort_as_half(BIAS)));
    return *reinterpret_cast<const uint32_t*>(&v);
}
// Nibbles m and m + 4 of w (shift = 4 m) as two halves.
template <uint16_t BIAS = 0x6400>
__device__ __forceinline__ uint32_t nibbles_to_h2(uint32_t w, int shift) {
    const uint32_t biased = ((w >> shift) & 0x000F000Fu) | 0x64006400u;
    const __half2 v = __hsub2(*reinterpret_cast<const __half2*>(&biased), __half2half2(__ushort_as_half(BIAS)));
    return *reinterpret_cast<const uint32_t*>(&v);
}
// Value codes enter the second product centred (code - 128, code - 8): the rounding of the softmax weights to half
// then acts on at most half the segment's range, and the centre joins the zero-point: z + c0 * s.
constexpr uint16_t kBias8 = 0x6480, kBias4 = 0x6408;  // 1024 + 128, 1024 + 8 as half

__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
    const __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Keys of the step: position j = tid % 64, quarter tid / 64 of the row's sixteen 16-byte chunks.
__device__ __forceinline__ void expand_keys(const uint8_t* raw, uint8_t* tile, int tid) {
    const int j = tid & 63, qtr = tid >> 6;
    const uint8_t* blk = raw + (j >> 5) * kBlockBytes;
    const int jp = j & 31;
    uint8_t* row = tile + (qtr >> 1) * (kStep * 128) + j * 128;
    const int sw = j & 7;
    const uint32_t* k4 = reinterpret_cast<const uint32_t*>(blk + kOffK4 + jp * 56);
    const int c0 = 4 * (qtr & 1);  // first chunk inside the 128-byte half row
    if (qtr == 0) {
        const uint4 k8 = *reinterpret_cast<const uint4*>(blk + jp * 16);
        *reinterpret_cast<uint4*>(row + ((0 ^ sw) << 4)) = make_uint4(bytes_to_h2<0x4140>(k8.x), bytes_to_h2<0x4342>(k8.x),
                                                                      bytes_to_h2<0x4140>(k8.y), bytes_to_h2<0x4342>(k8.y));
        *reinterpret_cast<uint4*>(row + ((1 ^ sw) << 4)) = make_uint4(bytes_to_h2<0x4140>(k8.z), bytes_to_h2<0x4342>(k8.z),
                                                                      bytes_to_h2<0x4140>(k8.w), bytes_to_h2<0x4342>(k8.w));
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t x = k4[i];
            *reinterpret_cast<uint4*>(row + (((2 + i) ^ sw) << 4)) =
                make_uint4(nibbles_to_h2(x, 0), nibbles_to_h2(x, 4), nibbles_to_h2(x, 8), nibbles_to_h2(x, 12));
        }
    } else {
        const int w0 = 4 * qtr - 2;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t x = k4[w0 + i];
            *reinterpret_cast<uint4*>(row + (((c0 + i) ^ sw) << 4)) =
                make_uint4(nibbles_to_h2(x, 0), nibbles_to_h2(x, 4), nibbles_to_h2(x, 8), nibbles_to_h2(x, 12));
        }
    }
}

// Values of the step, transposed: tile row n = output column, 64 positions (128 bytes) per row.
__device__ __forceinline__ void store_value(uint8_t* tile, int n, int j, uint32_t h) {
    *reinterpret_cast<uint16_t*>(tile + n * 128 + ((((j >> 3) ^ (n & 7)) << 4) | ((j & 7) << 1))) = static_cast<uint16_t>(h);
}
__device__ __forceinline__ void expand_value_word(uint8_t* tile, int w, int j, uint32_t x) {
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const uint32_t h2 = nibbles_to_h2<kBias4>(x, 4 * m);
        store_value(tile, 16 + 8 * w + 2 * m, j, h2 & 0xFFFF);
        store_value(tile, 16 + 8 * w + 2 * m + 1, j, h2 >> 16);
    }
}
__device__ __forceinline__ void expand_values(const uint8_t* raw, uint8_t* tile, int tid) {
    const int j = tid & 63, qtr = tid >> 6;
    const uint8_t* blk = raw + (j >> 5) * kBlockBytes;
    const int jp = j & 31;
    const uint32_t* v4 = reinterpret_cast<const uint32_t*>(blk + kOffV4 + jp * 56);
    if (qtr == 0) {
        const uint4 v8 = *reinterpret_cast<const uint4*>(blk + kOffV8 + jp * 16);
        const uint32_t w8[4] = {v8.x, v8.y, v8.z, v8.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = bytes_to_h2<0x4140, kBias8>(w8[i]), hi = bytes_to_h2<0x4342, kBias8>(w8[i]);
            store_value(tile, 4 * i + 0, j, lo & 0xFFFF);
            store_value(tile, 4 * i + 1, j, lo >> 16);
            store_value(tile, 4 * i + 2, j, hi & 0xFFFF);
            store_value(tile, 4 * i + 3, j, hi >> 16);
        }
        expand_value_word(tile, 0, j, v4[0]);
        expand_value_word(tile, 1, j, v4[1]);
    } else {
        const int w0 = 4 * qtr - 2;
#pragma unroll
        for (int i = 0; i < 4; ++i) expand_value_word(tile, w0 + i, j, v4[w0 + i]);
    }
}

// First pass over sixteen positions of one row: the running maximum of the scores.
template <bool MASKED>
__device__ __forceinline__ void scores_max(const uint32_t (&a8)[16], const uint32_t (&a4)[16], const float4* colK, int jb,
                                           int pos_i, float qsum8, float qsum4, float& m2) {
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        const float4 k = colK[c];
        const float sc = fmaf(k.x, __uint_as_float(a8[c]), fmaf(k.z, __uint_as_float(a4[c]), fmaf(k.y, qsum8, k.w * qsum4)));
        if (!MASKED || jb + c <= pos_i) m2 = fmaxf(m2, sc);
    }
}

// Second pass over sixteen positions of one row: softmax weights, their sums, and the two half-precision operand
// chunks (16 positions = 32 bytes of the row in each of P8' and P4').
template <bool MASKED>
__device__ __forceinline__ void scores_weights(const uint32_t (&a8)[16], const uint32_t (&a4)[16], const float4* colK,
                                               const float4* colV, int jb, int pos_i, float qsum8, float qsum4, float m2,
                                               float& l, float& zsum8, float& zsum4, uint32_t (&w8)[8], uint32_t (&w4)[8]) {
    float prev8 = 0.f, prev4 = 0.f;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        const float4 k = colK[c];
        const float sc = fmaf(k.x, __uint_as_float(a8[c]), fmaf(k.z, __uint_as_float(a4[c]), fmaf(k.y, qsum8, k.w * qsum4)));
        float p8 = 0.f, p4 = 0.f;
        if (!MASKED || jb + c <= pos_i) {
            const float pr = exp2f(sc - m2);
            const float4 v = colV[c];
            l += pr;
            zsum8 = fmaf(pr, v.y, zsum8);
            zsum4 = fmaf(pr, v.w, zsum4);
            p8 = pr * v.x;
            p4 = pr * v.z;
        }
        if (c & 1) {
            w8[c >> 1] = pack_h2(prev8, p8);
            w4[c >> 1] = pack_h2(prev4, p4);
        } else {
            prev8 = p8;
            prev4 = p4;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 2) attention_prefill_kernel(const PrefillParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;
    uint8_t* KV = Qs + kQBytes;
    uint8_t* P4 = KV + kKVBytes;
    uint8_t* P8 = P4 + kPBytes;
    uint8_t* raw = P8 + kPBytes;
    Shared* sh = reinterpret_cast<Shared*>(raw + 2 * kRawBytes);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int row = tid & (kRows - 1), half = tid >> 7;  // thread (row, half): cache block `half` of every step
    const int tile = static_cast<int>(gridDim.x) - 1 - static_cast<int>(blockIdx.x);  // long tiles first
    const int kvh = blockIdx.y;
    const int R = tile * kRows + row;
    const bool row_ok = R < p.T * p.g;
    const int tq = row_ok ? R / p.g : 0;
    const int hq = kvh * p.g + (row_ok ? R % p.g : 0);
    const int pos_i = row_ok ? p.pos0 + tq : -1;
    const int pos_first = p.pos0 + (tile * kRows) / p.g;  // position of the tile's first row: the smallest
    const int tq_max = min(p.T - 1, (tile * kRows + kRows - 1) / p.g);
    const int last_pos = p.pos0 + tq_max;
    const int n_steps = last_pos / kStep + 1;
    const int n_blocks = last_pos / RESQ_KV_BLOCK + 1;
    const uint8_t* blocks = p.blocks + static_cast<size_t>(kvh) * p.head_stride;

    if (tid == 0) {
        mbar_init(&sh->load[0], 1);
        mbar_init(&sh->load[1], 1);
        mbar_init(&sh->mma, 1);
        sh->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {  // a warp whose lanes have not diverged above: the allocation is a warp-wide instruction
        __syncwarp();
        tmem_alloc(&sh->tmem_base, kTmemCols);
        tmem_relinquish();
    }

    // ---- query tile: thread (row, half) writes half of the row's chunks, in the tile's permutation, and both
    // threads of a row form the sums of the two segments
    float qsum8 = 0.f, qsum4 = 0.f;
    {
        const uint4* src = reinterpret_cast<const uint4*>(p.q + (static_cast<size_t>(tq) * p.Hq + hq) * 128);
        const int sw = row & 7;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            uint4 v = row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
            const __half2* h = reinterpret_cast<const __half2*>(&v);
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h[i]);
                s += f.x + f.y;
            }
            if (c < 2) {
                qsum8 += s;
            } else {
                qsum4 += s;
                v = make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632), __byte_perm(v.y, v.w, 0x5410),
                               __byte_perm(v.y, v.w, 0x7632));
            }
            if ((c >> 3) == half)
                *reinterpret_cast<uint4*>(Qs + (c >> 3) * (kRows * 128) + row * 128 + (((c & 7) ^ sw) << 4)) = v;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);

    auto issue_load = [&](int gs) {
        const bool full = gs >= n_steps;
        const int s = full ? gs - n_steps : gs;
        const int b0 = 2 * s;
        const int nb = min(2, n_blocks - b0);
        uint64_t* bar = &sh->load[gs & 1];
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nb * (full ? kBlockBytes : kKeyBytes + kMetaBytes)));
        for (int b = 0; b < nb; ++b) {
            const uint8_t* src = blocks + static_cast<size_t>(b0 + b) * kBlockBytes;
            uint8_t* dst = raw + (gs & 1) * kRawBytes + b * kBlockBytes;
            if (full) {
                bulk_load(dst, src, kBlockBytes, bar);
            } else {
                bulk_load(dst, src, kKeyBytes, bar);
                bulk_load(dst + kOffVm, src + kOffVm, kMetaBytes, bar);
            }
        }
    };

    const uint32_t idS = make_idesc_f16(kRows, kStep);
    const uint32_t idO8 = make_idesc_f16(kRows, 16), idO4 = make_idesc_f16(kRows, 112);
    const uint64_t q_desc0 = make_smem_desc_k128(smem_u32(Qs)), q_desc1 = make_smem_desc_k128(smem_u32(Qs + kRows * 128));
    const uint64_t k_desc0 = make_smem_desc_k128(smem_u32(KV)), k_desc1 = make_smem_desc_k128(smem_u32(KV + kStep * 128));
    const uint64_t v_desc8 = make_smem_desc_k128(smem_u32(KV)), v_desc4 = make_smem_desc_k128(smem_u32(KV + 16 * 128));
    const uint64_t p_desc8 = make_smem_desc_k128(smem_u32(P8)), p_desc4 = make_smem_desc_k128(smem_u32(P4));

    const float kScoreScale = 1.4426950408889634f * 0.08838834764831845f;  // log2(e) / sqrt(128)
    float m2 = -INFINITY, vmax_col = 0.f, l = 0.f, zsum8 = 0.f, zsum4 = 0.f, out_scale = 1.f, p_scale = 1.f;
    uint32_t mma_phase = 0;
    int bad = 0;
    int loads_issued = 0;

    const int total = 2 * n_steps;
    if (tid == 0) {
        issue_load(0);
        loads_issued = 1;
    }
    for (int gs = 0; gs < total; ++gs) {
        const bool second = gs >= n_steps;
        const int s = second ? gs - n_steps : gs;
        const int j0 = s * kStep;
        if (gs == n_steps) {
            // between the passes: the two threads of a row merge their maxima; the tile's largest value scale gives
            // the power of two that normalises the second product's left operand
            sh->xch[0][half][row] = m2;
            if (tid < kStep) sh->vmax[tid] = vmax_col;
            __syncthreads();
            m2 = fmaxf(sh->xch[0][0][row], sh->xch[0][1][row]);
            float vmax = 0.f;
            for (int i = 0; i < kStep; ++i) vmax = fmaxf(vmax, sh->vmax[i]);
            int e = 0;
            if (vmax > 0.f) e = min(max(ilogbf(vmax), -100), 100);
            p_scale = ldexpf(1.f, -e);
            out_scale = ldexpf(1.f, e);
        }
        if (tid == 0 && gs + 1 < total) {
            issue_load(gs + 1);
            loads_issued = gs + 2;
        }
        const uint8_t* rb = raw + (gs & 1) * kRawBytes;
        if (!mbar_wait(&sh->load[gs & 1], (gs >> 1) & 1, &sh->abort_flag, p.status)) bad = 1;
        expand_keys(rb, KV, tid);
        if (tid < kStep) {  // the step's per-position constants
            const uint8_t* blk = rb + (tid >> 5) * kBlockBytes;
            const float4 k = reinterpret_cast<const float4*>(blk + kOffKm)[tid & 31];
            const float4 v = reinterpret_cast<const float4*>(blk + kOffVm)[tid & 31];
            sh->colK[tid] = make_float4(k.x * kScoreScale, k.y * kScoreScale, k.z * kScoreScale, k.w * kScoreScale);
            if (second)
                sh->colV[tid] = make_float4(v.x * p_scale, fmaf(128.f, v.x, v.y), v.z * p_scale, fmaf(8.f, v.z, v.w));
            else if (j0 + tid <= last_pos)
                vmax_col = fmaxf(vmax_col, fmaxf(v.x, v.z));
        }
        fence_proxy_async_smem();
        tc_fence_before();
        if (__syncthreads_or(bad)) {
            bad = 1;
            break;
        }
        if (tid == 0) {
            tc_fence_after();
            mma_f16_ss(tmem, q_desc0, k_desc0, idS, 0);
#pragma unroll
            for (int k = 1; k < 4; ++k) mma_f16_ss(tmem + 64, q_desc0 + 2 * k, k_desc0 + 2 * k, idS, k > 1);
#pragma unroll
            for (int k = 0; k < 4; ++k) mma_f16_ss(tmem + 64, q_desc1 + 2 * k, k_desc1 + 2 * k, idS, 1);
            tc_commit(&sh->mma);
        }
        if (!mbar_wait(&sh->mma, mma_phase, &sh->abort_flag, p.status)) bad = 1;
        mma_phase ^= 1;
        tc_fence_after();

        const bool masked = j0 + kStep - 1 > pos_first;  // uniform over the CTA
#pragma unroll 1
        for (int part = 0; part < 2; ++part) {  // sixteen positions at a time
            const int col = 32 * half + 16 * part;
            uint32_t a8[16], a4[16];
            __syncwarp();  // TMEM loads are warp-wide instructions
            tmem_ld16(lane_addr + col, a8);
            tmem_ld16(lane_addr + 64 + col, a4);
            tmem_ld_wait();
            if (!second) {
                if (masked)
                    scores_max<true>(a8, a4, sh->colK + col, j0 + col, pos_i, qsum8, qsum4, m2);
                else
                    scores_max<false>(a8, a4, sh->colK + col, j0 + col, pos_i, qsum8, qsum4, m2);
            } else {
                uint32_t w8[8], w4[8];
                if (masked)
                    scores_weights<true>(a8, a4, sh->colK + col, sh->colV + col, j0 + col, pos_i, qsum8, qsum4, m2, l,
                                         zsum8, zsum4, w8, w4);
                else
                    scores_weights<false>(a8, a4, sh->colK + col, sh->colV + col, j0 + col, pos_i, qsum8, qsum4, m2, l,
                                          zsum8, zsum4, w8, w4);
                const int sw = row & 7, chunk = col >> 3;
                *reinterpret_cast<uint4*>(P8 + row * 128 + ((chunk ^ sw) << 4)) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
                *reinterpret_cast<uint4*>(P8 + row * 128 + (((chunk + 1) ^ sw) << 4)) = make_uint4(w8[4], w8[5], w8[6], w8[7]);
                *reinterpret_cast<uint4*>(P4 + row * 128 + ((chunk ^ sw) << 4)) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                *reinterpret_cast<uint4*>(P4 + row * 128 + (((chunk + 1) ^ sw) << 4)) = make_uint4(w4[4], w4[5], w4[6], w4[7]);
            }
        }
        if (second) {
            // the score product is complete (waited above), so the key tile can become the value tile
            expand_values(rb, KV, tid);
            fence_proxy_async_smem();
            tc_fence_before();
            if (__syncthreads_or(bad)) {
                bad = 1;
                break;
            }
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t acc = (s > 0 || k > 0) ? 1u : 0u;
                    mma_f16_ss(tmem + 128, p_desc8 + 2 * k, v_desc8 + 2 * k, idO8, acc);
                    mma_f16_ss(tmem + 144, p_desc4 + 2 * k, v_desc4 + 2 * k, idO4, acc);
                }
                tc_commit(&sh->mma);
            }
            if (!mbar_wait(&sh->mma, mma_phase, &sh->abort_flag, p.status)) bad = 1;
            mma_phase ^= 1;
            tc_fence_after();
        }
        tc_fence_before();
        if (__syncthreads_or(bad)) {
            bad = 1;
            break;
        }
    }

    if (!bad) {  // uniform over the CTA: the TMEM loads are warp-wide instructions, only the stores depend on the row
        sh->xch[0][half][row] = l;
        sh->xch[1][half][row] = zsum8;
        sh->xch[2][half][row] = zsum4;
        __syncthreads();
        l = sh->xch[0][0][row] + sh->xch[0][1][row];
        zsum8 = sh->xch[1][0][row] + sh->xch[1][1][row];
        zsum4 = sh->xch[2][0][row] + sh->xch[2][1][row];
        const float inv = l > 0.f ? 1.f / l : 0.f;
        float* dst = p.out + (static_cast<size_t>(tq) * p.Hq + hq) * 128;
#pragma unroll 1
        for (int qd = 2 * half; qd < 2 * half + 2; ++qd) {  // thread (row, half): output columns [64 half, 64 half + 64)
            uint32_t o[32];
            __syncwarp();
            tmem_ld32(lane_addr + 128 + 32 * qd, o);
            tmem_ld_wait();
            if (!row_ok) continue;
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {  // eight output columns = eight coefficients
                const int n0 = 32 * qd + 8 * grp;
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(o[8 * grp + i]) * out_scale;
                float4 lo, hi;
                if (n0 < 16) {
                    lo = make_float4(f[0], f[1], f[2], f[3]);
                    hi = make_float4(f[4], f[5], f[6], f[7]);
                } else {
                    lo = make_float4(f[0], f[2], f[4], f[6]);
                    hi = make_float4(f[1], f[3], f[5], f[7]);
                }
                const float z = n0 < 16 ? zsum8 : zsum4;
                lo = make_float4((lo.x + z) * inv, (lo.y + z) * inv, (lo.z + z) * inv, (lo.w + z) * inv);
                hi = make_float4((hi.x + z) * inv, (hi.y + z) * inv, (hi.z + z) * inv, (hi.w + z) * inv);
                *reinterpret_cast<float4*>(dst + n0) = lo;
                *reinterpret_cast<float4*>(dst + n0 + 4) = hi;
            }
        }
    }

    // ---- teardown: copies still in flight are waited for (bounded), then the TMEM columns are returned
    if (bad && tid == 0) {
        int keep_waiting = 0;  // the shared abort flag is set by now; these waits run to their own limit
        for (int gs = max(0, loads_issued - 2); gs < loads_issued; ++gs)
            (void)mbar_wait(&sh->load[gs & 1], (gs >> 1) & 1, &keep_waiting, p.status);
        atomicOr(p.status, kStatusBitTimeout);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

cudaError_t launch_attention_prefill(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, int seq, int pos0,
                                     int T, float* out, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attention_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    PrefillParams p;
    const size_t nblk = static_cast<size_t>(cache.capacity / RESQ_KV_BLOCK);
    p.head_stride = nblk * kBlockBytes;
    p.blocks = static_cast<const uint8_t*>(cache.data) + static_cast<size_t>(seq) * cache.n_kv_heads * p.head_stride;
    p.q = static_cast<const __half*>(q16);
    p.out = out;
    p.T = T;
    p.Hq = n_q_heads;
    p.g = n_q_heads / cache.n_kv_heads;
    p.pos0 = pos0;
    p.status = device_status_ptr();
    const int rows = T * p.g;
    const dim3 grid(static_cast<unsigned>((rows + kRows - 1) / kRows), static_cast<unsigned>(cache.n_kv_heads));
    attention_prefill_kernel<<<grid, kThreads, kSmemBytes, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace resq
