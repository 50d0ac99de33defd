// Online projection C = X·P (Section 4.3, the U_D-type projection that cannot be folded into a
// preceding weight): bf16 x bf16 -> fp32 on tcgen05 kind::f16, fp32 coefficients written to a panel
// that the split-quantize kernel then reads (no bf16 rounding of the coefficients in between).
//
// Persistent, warp-specialised, 128 x 256 output tiles, K blocks of 64:
//   warp 0     TMA producer.  X tile [128 tokens][64 i] is K-major; P is row-major [i][j], i.e. the
//              B operand is N-major, loaded as four [64 i][64 j] boxes per stage (128-byte swizzle);
//   warp 1     tcgen05.mma issuer; two 256-column fp32 accumulators in TMEM so that the epilogue of
//              tile n overlaps the main loop of tile n+1;
//   warps 2-5  epilogue: tcgen05.ld -> fp32 stores.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int BM = 128, BN = 256, BK = 64;  // BK in bf16 elements (128 bytes)
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;        // 16 KB
constexpr int B_BOX_BYTES = BK * 64 * 2;    // one [64 i][64 j] box: 8 KB
constexpr int B_BYTES = B_BOX_BYTES * (BN / 64);
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr uint32_t kTmemCols = 512;

struct Params {
    int T, K;
    int m_tiles, n_tiles, kb_total;
    int bn;          // output columns per tile: a multiple of 16, <= BN (B loads and TMEM offsets stay BN wide)
    int panel_tiles; // m tiles per row panel of the tile order
    float* C;
    int* status;
};

struct __align__(8) Shared {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t drain;
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

// Tile order: row panels of `panel_tiles` m tiles; inside a panel the m index runs fastest.  The CTAs
// of one round then share a panel of X small enough to stay in L2 while the columns of P stream by.
__device__ __forceinline__ void tile_coords(const Params& p, int tile, int& m0, int& n0) {
    const int per_panel = p.panel_tiles * p.n_tiles;
    const int panel = tile / per_panel, rem = tile - panel * per_panel;
    const int mp = min(p.panel_tiles, p.m_tiles - panel * p.panel_tiles);  // m tiles in this panel
    const int n = rem / mp, m = rem - n * mp;
    m0 = (panel * p.panel_tiles + m) * BM;
    n0 = n * p.bn;
}

__global__ void __launch_bounds__(kThreads, 1)
project_gemm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmP,
                    const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + STAGES * A_BYTES;
    Shared* sh = reinterpret_cast<Shared*>(smem + STAGES * (A_BYTES + B_BYTES));
    volatile int* abort_flag = &sh->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sh->acc_full[b], 1);
            mbar_init(&sh->acc_empty[b], kEpiThreads);
        }
        mbar_init(&sh->drain, 1);
        sh->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmP);
    }
    if (warp == 1) {
        tmem_alloc(&sh->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0, issued = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int m0, n0;
                tile_coords(p, tile, m0, n0);
                for (int kb = 0; kb < p.kb_total; ++kb) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(&sh->full[stage], A_BYTES + B_BYTES);
                    tma_load_2d(sA + stage * A_BYTES, &tmX, &sh->full[stage], kb * BK, m0);
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c)
                        tma_load_2d(sB + stage * B_BYTES + c * B_BOX_BYTES, &tmP, &sh->full[stage], n0 + c * 64,
                                    kb * BK);
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                int n = issued < STAGES ? issued : STAGES;
                for (int i = 0; i < n; ++i) {
                    if (stage == 0) { stage = STAGES; phase ^= 1; }
                    --stage;
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(&sh->full[stage], phase) && global_timer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(BM, p.bn) | (1u << 16);  // B is N-major
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            int buf = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
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
                        mma_f16_ss(d, a_desc + 2 * k, b_desc + (2048 >> 4) * k, idesc, (kb == 0 && k == 0) ? 0u : 1u);
                    tc_commit(&sh->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit(&sh->acc_full[buf]);
                acc_phase[buf] ^= 1;
                buf ^= 1;
            }
            if (!ok) {
                tc_commit(&sh->drain);
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(&sh->drain, 0) && global_timer_ns() - t0 < 100000000ull) {}
            }
        }
    } else {
        const int quad = warp & 3;
        const int et = threadIdx.x - 64;
        uint32_t acc_phase[2] = {0, 0};
        int buf = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            int m0, n0;
            tile_coords(p, tile, m0, n0);
            const int n_end = min(p.K, n0 + p.bn);  // first column past this tile
            epi_barrier();
            if (et == 0) sh->epi_stop = *abort_flag;
            epi_barrier();
            if (sh->epi_stop) break;
            if (!mbar_wait(&sh->acc_full[buf], acc_phase[buf], abort_flag)) continue;
            acc_phase[buf] ^= 1;
            tc_fence_after();
            const int row = m0 + quad * 32 + lane;
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
                        if (nb + g * 4 < n_end)
                            reinterpret_cast<uint4*>(cp)[g] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                }
            }
            tc_fence_before();
            mbar_arrive(&sh->acc_empty[buf]);
            buf ^= 1;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->abort_flag) atomicOr(p.status, RESQ_ERR_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
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
        e = cudaFuncSetAttribute(project_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    CUtensorMap tX, tP;
    if (!make_map_bf16(&tX, X, T, K, BM) || !make_map_bf16(&tP, P, K, K, BK)) return cudaErrorInvalidValue;
    Params p;
    p.T = T; p.K = K;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.m_tiles = (T + BM - 1) / BM;
    p.bn = pick_tile_width(p.m_tiles, K, sms);
    p.n_tiles = (K + p.bn - 1) / p.bn;
    // Row panel: as many m tiles as keep the panel of X (rows x K bf16) within about 64 MB of L2.
    {
        const size_t tile_bytes = static_cast<size_t>(BM) * K * 2;
        size_t pt = (64u << 20) / tile_bytes;
        p.panel_tiles = pt < 1 ? 1 : (pt > static_cast<size_t>(p.m_tiles) ? p.m_tiles : static_cast<int>(pt));
    }
    p.kb_total = (K + BK - 1) / BK;
    p.C = C;
    p.status = device_status_ptr();
    const int tiles = p.m_tiles * p.n_tiles;
    project_gemm_kernel<<<tiles < sms ? tiles : sms, kThreads, kSmemBytes, st>>>(tX, tP, p);
    return cudaGetLastError();
}

}  // namespace resq
