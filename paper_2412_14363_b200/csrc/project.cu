// Online projection C = X·P (Section 4.3, the U_D-type projection that cannot be folded into a
// preceding weight) on CTA pairs: bf16 x bf16 -> fp32 with tcgen05.mma cta_group::2, fp32
// coefficients written to a panel that the split-quantize kernel then reads.
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 output tile.  Each CTA stages its
// own 128 rows of X and only its own half (128 columns) of the P block, so a K block costs each SM
// 32 KB of shared memory instead of 48 KB: six stages fit where the single-CTA kernel has four, and
// the shared-memory read rate per MMA falls by a third.  The MMA is issued by one thread of the
// even CTA and reads both CTAs' shared memory; each CTA's TMEM receives the accumulator rows of its
// own 128 tokens (two 256-column buffers, so the epilogue of tile n overlaps the main loop of tile
// n + 1).
//   warp 0     TMA producer (both CTAs).  X tile [128 tokens][64 i] is K-major; P is row-major
//              [i][j], i.e. the B operand is N-major, loaded as two [64 i][64 j] boxes per stage.
//              Completion bytes of both CTAs are counted on the even CTA's barrier.
//   warp 1     TMEM allocation (both CTAs); MMA issue (even CTA only).
//   warps 2-5  epilogue (both CTAs): tcgen05.ld -> fp32 stores of the CTA's 128 rows.
// Barriers that one CTA signals in the other: `full` (producer of the odd CTA -> even CTA),
// `empty` and `acc_full` (tcgen05.commit, multicast to both), `acc_empty` (epilogue threads of both
// CTAs -> even CTA).  No TMA multicast is used.  All waits are bounded.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int BM = 128;            // rows per CTA; the pair's tile has 2 * BM
constexpr int BN = 256, BK = 64;   // BK in bf16 elements (128 bytes)
constexpr int BN_HALF = BN / 2;    // P columns staged by each CTA
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;        // 16 KB
constexpr int B_BOX_BYTES = BK * 64 * 2;    // one [64 i][64 j] box: 8 KB
constexpr int B_BYTES = B_BOX_BYTES * (BN_HALF / 64);  // 16 KB
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr uint32_t kTmemCols = 512;

struct Params {
    int T, K;
    int m_tiles, n_tiles, kb_total;  // m_tiles counts 256-row pair tiles
    int panel_tiles;                 // pair tiles per row panel of the tile order
    float* C;
    int* status;
};

struct __align__(8) Shared {
    uint64_t full[STAGES];      // used in the even CTA: both CTAs' copies of a stage have landed
    uint64_t empty[STAGES];     // per CTA: the MMAs that read this stage are done
    uint64_t acc_full[2];       // per CTA: accumulator buffer complete
    uint64_t acc_empty[2];      // used in the even CTA: both CTAs' epilogues have drained the buffer
    uint32_t tmem_base;
    int abort_flag;
    int epi_stop;
};

constexpr size_t kSmemBytes = 1024 + STAGES * (A_BYTES + B_BYTES) + sizeof(Shared);

// N-major (MN-major) operand stored with the 128-byte swizzle: 64 contiguous bf16 of the N
// dimension per 128-byte row, 8 consecutive K rows per 1024-byte swizzle atom (stride byte offset),
// `lbo_bytes` between consecutive 64-wide N chunks (leading byte offset).
__device__ __forceinline__ uint64_t make_smem_desc_mn128(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

// Tile order: row panels of `panel_tiles` pair tiles; inside a panel the m index runs fastest.
__device__ __forceinline__ void tile_coords(const Params& p, int tile, int& m0, int& n0) {
    const int per_panel = p.panel_tiles * p.n_tiles;
    const int panel = tile / per_panel, rem = tile - panel * per_panel;
    const int mp = min(p.panel_tiles, p.m_tiles - panel * p.panel_tiles);
    const int n = rem / mp, m = rem - n * mp;
    m0 = (panel * p.panel_tiles + m) * 2 * BM;
    n0 = n * BN;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
project_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmP,
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
    const int num_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sh->full[s], 1);   // armed by the even CTA's producer for both CTAs' bytes
            mbar_init(&sh->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sh->acc_full[b], 1);
            mbar_init(&sh->acc_empty[b], 2 * kEpiThreads);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmP);
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
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                int m0, n0;
                tile_coords(p, tile, m0, n0);
                const int my_m = m0 + rank * BM, my_n = n0 + rank * BN_HALF;
                for (int kb = 0; kb < p.kb_total; ++kb) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                    // The even CTA arms its barrier for the bytes of both CTAs; the peer only sends its bytes
                    // there (they may land before the barrier is armed: the pending arrival keeps the phase open).
                    const uint32_t full_addr = cluster_map(&sh->full[stage], 0);
                    if (rank == 0) mbar_arrive_expect_tx(&sh->full[stage], 2 * (A_BYTES + B_BYTES));
                    tma_load_2d_pair(sA + stage * A_BYTES, &tmX, full_addr, kb * BK, my_m);
#pragma unroll
                    for (int c = 0; c < BN_HALF / 64; ++c)
                        tma_load_2d_pair(sB + stage * B_BYTES + c * B_BOX_BYTES, &tmP, full_addr, my_n + c * 64, kb * BK);
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
            constexpr uint32_t idesc = make_idesc_bf16(2 * BM, BN) | (1u << 16);  // B is N-major
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            int buf = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                if (!mbar_wait(&sh->acc_empty[buf], acc_phase[buf] ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + static_cast<uint32_t>(buf * BN);
                for (int kb = 0; kb < p.kb_total; ++kb) {
                    if (!mbar_wait(&sh->full[stage], phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc_k128(smem_u32(sA + stage * A_BYTES));
                    const uint64_t b_desc = make_smem_desc_mn128(smem_u32(sB + stage * B_BYTES), B_BOX_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)  // 16 k per instruction: 32 B of an A row, 2 KB of a B box
                        mma_f16_ss_pair(d, a_desc + 2 * k, b_desc + (2048 >> 4) * k, idesc, (kb == 0 && k == 0) ? 0u : 1u);
                    tc_commit_pair(&sh->empty[stage], 3);  // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit_pair(&sh->acc_full[buf], 3);
                acc_phase[buf] ^= 1;
                buf ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (both CTAs)
        const int quad = warp & 3;
        const int et = threadIdx.x - 64;
        uint32_t acc_phase[2] = {0, 0};
        int buf = 0;
        for (int tile = pair; tile < num_tiles; tile += npairs) {
            int m0, n0;
            tile_coords(p, tile, m0, n0);
            epi_barrier();
            if (et == 0) sh->epi_stop = *abort_flag;
            epi_barrier();
            if (sh->epi_stop) break;
            if (!mbar_wait(&sh->acc_full[buf], acc_phase[buf], abort_flag)) continue;
            acc_phase[buf] ^= 1;
            tc_fence_after();
            const int row = m0 + rank * BM + quad * 32 + lane;
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(lane_addr + c * 32, v);
                tmem_ld_wait();
                const int nb = n0 + c * 32;
                if (row < p.T) {
                    float* cp = p.C + static_cast<size_t>(row) * p.K + nb;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (nb + g * 4 < p.K)
                            reinterpret_cast<uint4*>(cp)[g] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                }
            }
            tc_fence_before();
            mbar_arrive_cluster(cluster_map(&sh->acc_empty[buf], 0));
            buf ^= 1;
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves while the other may still read its shared memory or signal it
    if (threadIdx.x == 0 && sh->abort_flag) atomicOr(p.status, RESQ_ERR_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][cols] bf16 matrix, box = 64 columns (128 bytes) x box_rows, 128-byte swizzle, zero fill.
bool make_map_bf16(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeFn enc = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_project_gemm(const void* X, const void* P, int T, int K, float* C, cudaStream_t st) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(project_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    CUtensorMap tX, tP;
    if (!make_map_bf16(&tX, X, T, K, BM) || !make_map_bf16(&tP, P, K, K, BK)) return cudaErrorInvalidValue;
    Params p;
    p.T = T; p.K = K;
    p.m_tiles = (T + 2 * BM - 1) / (2 * BM);
    p.n_tiles = (K + BN - 1) / BN;
    p.kb_total = (K + BK - 1) / BK;
    // Row panel: as many pair tiles as keep the panel of X (rows x K bf16) within about 64 MB of L2.
    {
        const size_t tile_bytes = static_cast<size_t>(2 * BM) * K * 2;
        size_t pt = (64u << 20) / tile_bytes;
        p.panel_tiles = pt < 1 ? 1 : (pt > static_cast<size_t>(p.m_tiles) ? p.m_tiles : static_cast<int>(pt));
    }
    p.C = C;
    p.status = device_status_ptr();
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = p.m_tiles * p.n_tiles;
    int pairs = sms / 2;
    if (tiles < pairs) pairs = tiles;
    project_gemm_pair_kernel<<<2 * pairs, kThreads, kSmemBytes, st>>>(tX, tP, p);
    return cudaGetLastError();
}

}  // namespace resq
