// Many-token mixed-precision GEMM (Eq. 4 + dequantizing epilogue) on tcgen05 kind::i8, CTA pairs.
//
// Persistent, warp-specialised kernel.  Two CTAs on neighbouring SMs (a cluster of 2) share one
// 256 x 256 output tile (tcgen05 cta_group::2): each stages its own 128 token rows and only its own
// 128 of the tile's 256 weight rows, 32 KB per K block, so six stages fit and the shared-memory read
// rate per MMA is a third lower than with one CTA per 128 x 256 tile.
//   warp 0     TMA producer (both CTAs): streams 128-byte-wide K blocks of the activation and weight
//              codes into the ring (128-byte swizzle), first the INT4 segment (codes one per byte, so
//              both segments run on the i8 tensor path exactly), then the INT8 one.  Completion bytes
//              of both CTAs are counted on the even CTA's barrier.
//   warp 1     TMEM allocation (both CTAs; 512 columns); MMA issue (even CTA only): the INT8 segment
//              accumulates into columns [0,256), the INT4 segment into [256,512) -- two int32
//              accumulators per output because the two segments carry different (token, channel)
//              scales.  Each CTA's TMEM receives the rows of its own 128 tokens.
//   warps 2-9  epilogue (both CTAs), two threads per tile row (128 columns each).
// Two full-width accumulators fill TMEM, so there is no second buffer; the epilogue instead frees
// the tensor pipe early.  It first copies its INT4 accumulator values into registers (raw int32,
// 128 per thread) and releases those columns: the next tile's INT4 segment -- 7/8 of its work --
// starts at once, while the epilogue goes on to read the INT8 accumulator, form
// y = acc8*(sx8*sw8) + acc4*(sx4*sw4) in fp32, convert and store; the INT8 columns are released
// long before the next tile's short INT8 segment needs them.
// Barriers signalled across the pair: `full` (odd CTA's copies -> even CTA), `empty` and `acc_full`
// (tcgen05.commit, multicast to both), `acc4_empty` / `acc8_empty` (epilogue threads of both CTAs ->
// even CTA).  No TMA multicast.  Out-of-range rows/columns/K are zero-filled by TMA and masked at
// the store.  All waits are bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int BM = 128, BN = 256, BK = 128;  // BK in bytes == int8 elements
constexpr int STAGES = 6;
constexpr int BN_HALF = BN / 2;  // weight rows staged by each CTA of the pair
constexpr int A_BYTES = BM * BK, B_BYTES = BN_HALF * BK;
constexpr int kThreads = 320;
constexpr int kEpiThreads = 256;
constexpr uint32_t kTmemCols = 512;

struct Params {
    int T, N, r, K4;
    int m_tiles, n_tiles, kb8, kb4;
    int bn;  // output columns per tile: a multiple of 16, <= BN (the B loads and TMEM offsets stay BN wide)
    const float* s_x8;
    const float* s_x4;
    const void* s_w8;
    const void* s_w4;
    int w_fp16;
    // asymmetric activations only: per-token zero-points and per-channel row sums of the weight codes
    const float* z_x8;
    const float* z_x4;
    const int32_t* wsum8;
    const int32_t* wsum4;
    void* Y;
    int y_dtype;
    int32_t* dbg8;
    int32_t* dbg4;
    int* status;
};

struct __align__(8) Shared {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t acc_full;
    uint64_t acc4_empty;
    uint64_t acc8_empty;
    uint32_t tmem_base;
    int abort_flag;
    int epi_stop;
    float sw8[BN];
    float sw4[BN];
    float zc8[BN];  // asymmetric activations: (float)wsum8[n] * sw8[n], the column factor of the zero-point term
    float zc4[BN];
};

constexpr size_t kSmemBytes = 1024 + STAGES * (A_BYTES + B_BYTES) + sizeof(Shared);

__device__ __forceinline__ float load_scale(const void* p, int i, int fp16) {
    return fp16 ? __half2float(reinterpret_cast<const __half*>(p)[i]) : reinterpret_cast<const float*>(p)[i];
}

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

// ASYM: the activation codes are unsigned (u8 x s8 products) and every output gets the rank-one
// zero-point terms z_x8[t] * s_w8[n] * wsum8[n] + z_x4[t] * s_w4[n] * wsum4[n] (Eq. 1, second form).
template <bool ASYM>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
mixed_gemm_kernel(const __grid_constant__ CUtensorMap tmA8, const __grid_constant__ CUtensorMap tmA4,
                  const __grid_constant__ CUtensorMap tmB8, const __grid_constant__ CUtensorMap tmB4,
                  const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + STAGES * A_BYTES;
    Shared* sh = reinterpret_cast<Shared*>(smem + STAGES * (A_BYTES + B_BYTES));
    volatile int* abort_flag = &sh->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = static_cast<int>(cluster_ctarank());  // 0: even CTA (issues the MMAs), 1: its peer
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int num_tiles = p.m_tiles * p.n_tiles;  // m_tiles counts 256-row pair tiles
    const int kb_total = p.kb8 + p.kb4;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], 1);
        }
        mbar_init(&sh->acc_full, 1);
        mbar_init(&sh->acc4_empty, 2 * kEpiThreads);  // used in the even CTA: epilogue threads of both CTAs
        mbar_init(&sh->acc8_empty, 2 * kEpiThreads);
        sh->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmA8);
        tma_prefetch_desc(&tmA4);
        tma_prefetch_desc(&tmB8);
        tma_prefetch_desc(&tmB4);
    }
    if (warp == 1) {
        tmem_alloc_pair(&sh->tmem_base, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything is signalled across
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                const int m0 = (tile % p.m_tiles) * 2 * BM + rank * BM;        // this CTA's token rows
                const int n0 = (tile / p.m_tiles) * p.bn + rank * BN_HALF;     // this CTA's weight rows
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, p.status)) { ok = false; break; }
                    // The even CTA arms its barrier for the bytes of both CTAs; the peer only sends its
                    // bytes there (if they land first, the pending arrival keeps the phase open).
                    const uint32_t full_addr = cluster_map(&sh->full[stage], 0);
                    if (rank == 0) mbar_arrive_expect_tx(&sh->full[stage], 2 * (A_BYTES + B_BYTES));
                    if (kb < p.kb4) {
                        tma_load_2d_pair(sA + stage * A_BYTES, &tmA4, full_addr, kb * BK, m0);
                        tma_load_2d_pair(sB + stage * B_BYTES, &tmB4, full_addr, kb * BK, n0);
                    } else {
                        tma_load_2d_pair(sA + stage * A_BYTES, &tmA8, full_addr, (kb - p.kb4) * BK, m0);
                        tma_load_2d_pair(sB + stage * B_BYTES, &tmB8, full_addr, (kb - p.kb4) * BK, n0);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // Give the copies already in flight time to land before the CTA gives up its shared memory.
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 1000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = ASYM ? make_idesc_u8s8(2 * BM, p.bn) : make_idesc_i8(2 * BM, p.bn);
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                // INT4 columns are free once the previous tile's epilogue has copied them out.
                if (!mbar_wait(&sh->acc4_empty, acc_phase ^ 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < kb_total; ++kb) {
                    const bool seg4 = kb < p.kb4;
                    if (kb == p.kb4) {
                        // ... the INT8 columns once it has finished with the tile.
                        if (!mbar_wait(&sh->acc8_empty, acc_phase ^ 1, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                    }
                    if (!mbar_wait(&sh->full[stage], phase, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc_k128(smem_u32(sA + stage * A_BYTES));
                    const uint64_t b_desc = make_smem_desc_k128(smem_u32(sB + stage * B_BYTES));
                    const uint32_t d = tmem_base + (seg4 ? static_cast<uint32_t>(BN) : 0u);
                    const bool first = kb == 0 || kb == p.kb4;
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)
                        mma_i8_ss_pair(d, a_desc + 2 * k, b_desc + 2 * k, idesc, (first && k == 0) ? 0u : 1u);
                    tc_commit_pair(&sh->empty[stage], 3);  // frees the ring slot in both CTAs once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit_pair(&sh->acc_full, 3);
                acc_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;            // TMEM lane quadrant this warp may access
        const int ch = (warp - 2) >> 2;       // column half of the tile this warp handles
        const int et = threadIdx.x - 64;
        uint32_t acc_phase = 0;
        // The epilogue threads meet at named barriers, so they must leave the loop together:
        // one thread samples the abort flag and the others take its reading.
        for (int tile = pair; tile < num_tiles; tile += npairs) {
            const int m0 = (tile % p.m_tiles) * 2 * BM + rank * BM, n0 = (tile / p.m_tiles) * p.bn;
            epi_barrier();  // previous tile's readers of sw8/sw4/epi_stop are done
            if (et == 0) sh->epi_stop = *abort_flag;
            const int n_end = min(p.N, n0 + p.bn);  // first column past this tile
            {
                const int n = n0 + et;
                const float w8s = n < n_end ? load_scale(p.s_w8, n, p.w_fp16) : 0.f;
                const float w4s = n < n_end ? load_scale(p.s_w4, n, p.w_fp16) : 0.f;
                sh->sw8[et] = w8s;
                sh->sw4[et] = w4s;
                if (ASYM) {
                    sh->zc8[et] = n < n_end ? static_cast<float>(p.wsum8[n]) * w8s : 0.f;
                    sh->zc4[et] = n < n_end ? static_cast<float>(p.wsum4[n]) * w4s : 0.f;
                }
            }
            epi_barrier();
            if (sh->epi_stop) break;
            const int row = m0 + quad * 32 + lane;
            const bool row_ok = row < p.T;
            const float sx8 = row_ok ? __ldg(p.s_x8 + row) : 0.f;
            const float sx4 = row_ok ? __ldg(p.s_x4 + row) : 0.f;
            const float zx8 = ASYM && row_ok ? __ldg(p.z_x8 + row) : 0.f;
            const float zx4 = ASYM && row_ok ? __ldg(p.z_x4 + row) : 0.f;
            if (!mbar_wait(&sh->acc_full, acc_phase, abort_flag, p.status)) continue;  // flag is set; leave at the next sample
            acc_phase ^= 1;
            tc_fence_after();
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + ch * (BN / 2);
            // Phase 1: the INT4 accumulator values of this thread's 128 columns, raw, into registers.
            uint32_t a4[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(lane_addr + BN + c * 32, a4[c]);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive_cluster(cluster_map(&sh->acc4_empty, 0));
            // Phase 2: the INT8 accumulator, the scales, the store -- 16 columns at a time.
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t a8[16];
                tmem_ld16(lane_addr + c * 16, a8);
                tmem_ld_wait();
                if (p.kb8 == 0) {  // uniform INT4: the INT8 accumulator was never written
#pragma unroll
                    for (int j = 0; j < 16; ++j) a8[j] = 0;
                }
                const int cb = ch * (BN / 2) + c * 16;  // first column of the chunk inside the tile
                const int nb = n0 + cb;
                const uint32_t* a4c = &a4[c >> 1][(c & 1) * 16];
                if (row_ok) {
                    const size_t off = static_cast<size_t>(row) * p.N + nb;
                    if (p.dbg8) {
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            if (nb + g * 4 < n_end) {
                                reinterpret_cast<uint4*>(p.dbg8 + off)[g] =
                                    make_uint4(a8[4 * g], a8[4 * g + 1], a8[4 * g + 2], a8[4 * g + 3]);
                                reinterpret_cast<uint4*>(p.dbg4 + off)[g] =
                                    make_uint4(a4c[4 * g], a4c[4 * g + 1], a4c[4 * g + 2], a4c[4 * g + 3]);
                            }
                    }
                    float y[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float t8 = static_cast<float>(static_cast<int>(a8[j])) * (sx8 * sh->sw8[cb + j]);
                        const float t4 = static_cast<float>(static_cast<int>(a4c[j])) * (sx4 * sh->sw4[cb + j]);
                        y[j] = t8 + t4;
                        if (ASYM) y[j] += zx8 * sh->zc8[cb + j] + zx4 * sh->zc4[cb + j];
                    }
                    if (p.y_dtype == RESQ_Y_BF16) {
                        __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.Y) + off;
#pragma unroll
                        for (int g = 0; g < 2; ++g)
                            if (nb + g * 8 < n_end) {
                                uint32_t w[4];
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    __nv_bfloat162 h = __floats2bfloat162_rn(y[g * 8 + 2 * q], y[g * 8 + 2 * q + 1]);
                                    w[q] = *reinterpret_cast<uint32_t*>(&h);
                                }
                                reinterpret_cast<uint4*>(yp)[g] = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                    } else {
                        float* yp = reinterpret_cast<float*>(p.Y) + off;
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            if (nb + g * 4 < n_end)
                                reinterpret_cast<float4*>(yp)[g] =
                                    make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive_cluster(cluster_map(&sh->acc8_empty, 0));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves while the other may still read its shared memory or signal it
    if (threadIdx.x == 0 && sh->abort_flag) atomicOr(p.status, kStatusBitTimeout);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][kbytes] uint8 matrix, box = 128 bytes x box_rows, 128-byte swizzle, zero fill out of range.
bool make_map_u8(CUtensorMap* m, const void* base, uint64_t rows, uint64_t kbytes, uint32_t box_rows) {
    EncodeFn enc = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!enc) return false;
    cuuint64_t dims[2] = {kbytes, rows};
    cuuint64_t strides[1] = {kbytes};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_mixed_gemm_tiles(int T, int N, int K, int r, const int8_t* x8, const int8_t* x4e,
                                    const float* s_x8, const float* s_x4, const int8_t* w8, const int8_t* w4e,
                                    const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                    int32_t* dbg8, int32_t* dbg4, cudaStream_t st, const float* z_x8,
                                    const float* z_x4, const int32_t* wsum8, const int32_t* wsum4) {
    const bool asym = z_x8 != nullptr;  // then x8 / x4e hold unsigned codes
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(mixed_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(mixed_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int K4 = K - r;
    CUtensorMap tA8, tA4, tB8, tB4;
    if (!make_map_u8(&tA4, x4e, T, K4, BM) || !make_map_u8(&tB4, w4e, N, K4, BN_HALF)) return cudaErrorInvalidValue;
    if (r > 0) {
        if (!make_map_u8(&tA8, x8, T, r, BM) || !make_map_u8(&tB8, w8, N, r, BN_HALF)) return cudaErrorInvalidValue;
    } else {  // uniform INT4: no INT8 segment, its maps are never used
        tA8 = tA4;
        tB8 = tB4;
    }
    Params p;
    p.T = T; p.N = N; p.r = r; p.K4 = K4;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.m_tiles = (T + 2 * BM - 1) / (2 * BM);
    // The kernel takes any multiple of 16 up to BN here (B loads and TMEM offsets stay BN wide); tiles of 240 and
    // 192 columns measured 1.5-1.7 x slower per column than 256-wide ones, far more than a fuller last round saves.
    p.bn = BN;
    p.n_tiles = (N + p.bn - 1) / p.bn;
    p.kb8 = (r + BK - 1) / BK;
    p.kb4 = (K4 + BK - 1) / BK;
    p.s_x8 = s_x8; p.s_x4 = s_x4; p.s_w8 = s_w8; p.s_w4 = s_w4;
    p.w_fp16 = w_scale_fp16 ? 1 : 0;
    p.z_x8 = z_x8; p.z_x4 = z_x4; p.wsum8 = wsum8; p.wsum4 = wsum4;
    p.Y = Y; p.y_dtype = y_dtype; p.dbg8 = dbg8; p.dbg4 = dbg8 ? dbg4 : nullptr;
    p.status = device_status_ptr();
    const int tiles = p.m_tiles * p.n_tiles;
    const int pairs = tiles < sms / 2 ? tiles : sms / 2;
    count_launch();
    if (asym) mixed_gemm_kernel<true><<<2 * pairs, kThreads, kSmemBytes, st>>>(tA8, tA4, tB8, tB4, p);
    else mixed_gemm_kernel<false><<<2 * pairs, kThreads, kSmemBytes, st>>>(tA8, tA4, tB8, tB4, p);
    return cudaGetLastError();
}

}  // namespace resq
