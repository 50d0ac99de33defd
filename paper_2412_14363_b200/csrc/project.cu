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
    // Tiles cut along K: the last `split_tiles` tiles of the order (the partly filled last round of the persistent
    // grid; with few token rows, every tile) become `splits` slices of `kb_slice` k-blocks each, one work item per
    // slice, written as partial tiles to `partial` ([split_tiles][splits][prows][256] fp32, prows = token rows kept
    // per tile) and summed in slice order by project_reduce_kernel.  0: no split.
    int full_items, split_tiles, splits, kb_slice, prows;
    float* partial;
};

struct Item {
    int m0, n0, kb0, nkb;
    float* dst;     // first element of the 256 x 256 output tile (C or a partial tile)
    size_t ld;      // its row pitch in floats
    bool bounded;   // rows >= T and columns >= K must not be written (C); partial tiles are written whole
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

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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

__device__ __forceinline__ Item item_info(const Params& p, int item) {
    Item it;
    if (item < p.full_items) {
        tile_coords(p, item, it.m0, it.n0);
        it.kb0 = 0;
        it.nkb = p.kb_total;
        it.dst = p.C + static_cast<size_t>(it.m0) * p.K + it.n0;
        it.ld = static_cast<size_t>(p.K);
        it.bounded = true;
    } else {
        const int j = item - p.full_items;
        int t = j / p.splits, sl = j - t * p.splits;
        if (p.full_items == 0) {  // every tile is cut: slice-major, so that the pairs of a round read the same rows of P
            sl = j / p.split_tiles;
            t = j - sl * p.split_tiles;
        }
        tile_coords(p, p.full_items + t, it.m0, it.n0);
        it.kb0 = sl * p.kb_slice;
        it.nkb = min(p.kb_slice, p.kb_total - it.kb0);
        it.dst = p.partial + static_cast<size_t>(t * p.splits + sl) * p.prows * BN;
        it.ld = BN;
        it.bounded = false;
    }
    return it;
}

// C tile = sum of its partial tiles, slices in index order (deterministic).  One thread per four columns of one
// row; the slices' loads are issued eight at a time and added in order.  Launched with programmatic stream
// serialization behind the GEMM: its CTAs are scheduled as the GEMM's retire and wait here for the whole grid.
__global__ void __launch_bounds__(256) project_reduce_kernel(const Params p) {
    griddep_launch_dependents();
    const int t = blockIdx.y;
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.prows * BN / 4) return;
    int m0, n0;
    tile_coords(p, p.full_items + t, m0, n0);
    const int row = q / (BN / 4), c4 = q - row * (BN / 4);
    const size_t tile_floats = static_cast<size_t>(p.prows) * BN;
    const float4* part = reinterpret_cast<const float4*>(p.partial + static_cast<size_t>(t) * p.splits * tile_floats) + q;
    const size_t step = tile_floats / 4;
    griddep_wait();
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < p.splits; s0 += 8) {
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            v[i] = s0 + i < p.splits ? __ldcg(part + static_cast<size_t>(s0 + i) * step) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (s0 + i < p.splits) {
                if (s0 + i == 0) a = v[0];
                else { a.x += v[i].x; a.y += v[i].y; a.z += v[i].z; a.w += v[i].w; }
            }
    }
    if (m0 + row < p.T && n0 + 4 * c4 < p.K)
        *reinterpret_cast<float4*>(p.C + static_cast<size_t>(m0 + row) * p.K + n0 + 4 * c4) = a;
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
    const int num_items = p.full_items + p.split_tiles * p.splits;

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
    griddep_launch_dependents();  // a kernel enqueued with programmatic serialization is scheduled as SMs free up

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = pair; item < num_items && ok; item += npairs) {
                const Item it = item_info(p, item);
                const int my_m = it.m0 + rank * BM, my_n = it.n0 + rank * BN_HALF;
                for (int kb = it.kb0; kb < it.kb0 + it.nkb; ++kb) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, p.status)) { ok = false; break; }
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
            for (int item = pair; item < num_items && ok; item += npairs) {
                const int nkb = item_info(p, item).nkb;
                if (!mbar_wait(&sh->acc_empty[buf], acc_phase[buf] ^ 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + static_cast<uint32_t>(buf * BN);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(&sh->full[stage], phase, abort_flag, p.status)) { ok = false; break; }
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
        for (int item = pair; item < num_items; item += npairs) {
            const Item it = item_info(p, item);
            epi_barrier();
            if (et == 0) sh->epi_stop = *abort_flag;
            epi_barrier();
            if (sh->epi_stop) break;
            if (!mbar_wait(&sh->acc_full[buf], acc_phase[buf], abort_flag, p.status)) continue;
            acc_phase[buf] ^= 1;
            tc_fence_after();
            const int lrow = rank * BM + quad * 32 + lane;  // row inside the pair's tile
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(lane_addr + c * 32, v);
                tmem_ld_wait();
                const int nb = it.n0 + c * 32;
                if (!it.bounded || it.m0 + lrow < p.T) {
                    float* cp = it.dst + static_cast<size_t>(lrow) * it.ld + c * 32;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (!it.bounded || nb + g * 4 < p.K)
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
    if (threadIdx.x == 0 && sh->abort_flag) atomicOr(p.status, kStatusBitTimeout);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------------------
// Few token rows (a generation step, T <= kFewMaxT): the product is a stream of P, and a 256-token tile would
// keep the tensor pipe as busy with zero rows as the stream keeps HBM.  The operands change roles instead:
// C^T = P^T · X^T, so the 256 rows of the pair's MMA are 256 columns j of P (the staged [64 i][128 j] half-tiles
// are the M-major A operand, the same bytes in the same layout as the tile kernel's B operand) and its N columns
// are the tokens, rounded up to a multiple of 16 (each CTA stages N/2 token rows of X, K-major).  A k-block then
// costs 16 KB + N/2 x 128 B of shared memory per CTA, so ten stages fit, and N/256 of the tile kernel's MMA time.
// Every tile is cut along K (Params::splits) so that all SM pairs stream an equal share of P.
constexpr int kFewMaxT = 64;
constexpr int FSTAGES = 10;
constexpr int FX_BYTES = (kFewMaxT / 2) * BK * 2;  // room for the CTA's token rows of one stage: 4 KB
constexpr uint32_t kFewTmemCols = 2 * kFewMaxT;     // two accumulator buffers of up to 64 columns

struct __align__(8) FewShared {
    uint64_t full[FSTAGES];
    uint64_t empty[FSTAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int epi_stop;
};

constexpr size_t kFewSmemBytes = 1024 + FSTAGES * (B_BYTES + FX_BYTES) + sizeof(FewShared);

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
project_gemm_few_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmP,
                        const Params p, const int ntok) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sP = smem;
    uint8_t* sX = smem + FSTAGES * B_BYTES;
    FewShared* sh = reinterpret_cast<FewShared*>(smem + FSTAGES * (B_BYTES + FX_BYTES));
    volatile int* abort_flag = &sh->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = static_cast<int>(cluster_ctarank());
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int num_items = p.full_items + p.split_tiles * p.splits;
    const int half_tok = ntok / 2;                                   // token rows staged by each CTA
    const uint32_t x_bytes = static_cast<uint32_t>(half_tok) * BK * 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < FSTAGES; ++s) {
            mbar_init(&sh->full[s], 1);
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
        tmem_alloc_pair(&sh->tmem_base, kFewTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    griddep_launch_dependents();  // a kernel enqueued with programmatic serialization is scheduled as SMs free up

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = pair; item < num_items && ok; item += npairs) {
                const Item it = item_info(p, item);
                const int my_j = it.n0 + rank * BN_HALF;
                for (int kb = it.kb0; kb < it.kb0 + it.nkb; ++kb) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t full_addr = cluster_map(&sh->full[stage], 0);
                    if (rank == 0) mbar_arrive_expect_tx(&sh->full[stage], 2 * (B_BYTES + x_bytes));
#pragma unroll
                    for (int c = 0; c < BN_HALF / 64; ++c)
                        tma_load_2d_pair(sP + stage * B_BYTES + c * B_BOX_BYTES, &tmP, full_addr, my_j + c * 64, kb * BK);
                    tma_load_2d_pair(sX + stage * FX_BYTES, &tmX, full_addr, kb * BK, rank * half_tok);
                    if (++stage == FSTAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 1000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc_bf16(2 * BM, ntok) | (1u << 15);  // A (the P tile) is M-major
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            int buf = 0;
            bool ok = true;
            for (int item = pair; item < num_items && ok; item += npairs) {
                const int nkb = item_info(p, item).nkb;
                if (!mbar_wait(&sh->acc_empty[buf], acc_phase[buf] ^ 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + static_cast<uint32_t>(buf * kFewMaxT);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(&sh->full[stage], phase, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc_mn128(smem_u32(sP + stage * B_BYTES), B_BOX_BYTES);
                    const uint64_t b_desc = make_smem_desc_k128(smem_u32(sX + stage * FX_BYTES));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)  // 16 i per instruction: 2 KB of a P box, 32 B of a token row
                        mma_f16_ss_pair(d, a_desc + (2048 >> 4) * k, b_desc + 2 * k, idesc, (kb == 0 && k == 0) ? 0u : 1u);
                    tc_commit_pair(&sh->empty[stage], 3);
                    if (++stage == FSTAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit_pair(&sh->acc_full[buf], 3);
                acc_phase[buf] ^= 1;
                buf ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (both CTAs): lane = column j of C
        const int quad = warp & 3;
        const int et = threadIdx.x - 64;
        uint32_t acc_phase[2] = {0, 0};
        int buf = 0;
        for (int item = pair; item < num_items; item += npairs) {
            const Item it = item_info(p, item);
            epi_barrier();
            if (et == 0) sh->epi_stop = *abort_flag;
            epi_barrier();
            if (sh->epi_stop) break;
            if (!mbar_wait(&sh->acc_full[buf], acc_phase[buf], abort_flag, p.status)) continue;
            acc_phase[buf] ^= 1;
            tc_fence_after();
            const int jj = rank * BM + quad * 32 + lane;  // column inside the tile
            const bool col_ok = !it.bounded || it.n0 + jj < p.K;
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kFewMaxT;
#pragma unroll 1
            for (int c = 0; c < ntok / 16; ++c) {
                uint32_t v[16];
                tmem_ld16(lane_addr + c * 16, v);
                tmem_ld_wait();
                if (col_ok) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c * 16 + i < p.T) it.dst[static_cast<size_t>(c * 16 + i) * it.ld + jj] = __uint_as_float(v[i]);
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
    cluster_sync_all();
    if (threadIdx.x == 0 && sh->abort_flag) atomicOr(p.status, kStatusBitTimeout);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kFewTmemCols);
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

namespace {

cudaError_t launch_reduce(const Params& p, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.prows * BN / 4 + 255) / 256, p.split_tiles, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, project_reduce_kernel, p);
}

// T <= kFewMaxT.  Chooses the K split: every tile becomes `s` slices; the cost of a choice is the number of k-blocks
// the busiest pair streams, rounds x slice length.  A finer split is taken only when it is at least 2 % better, and
// only while the partial tiles stay within the scratch and within 1/16 of the bytes of P.
cudaError_t launch_project_few(const void* X, const void* P, int T, int K, float* C, cudaStream_t st, void* scratch,
                               size_t scratch_bytes, int dev) {
    static bool attr_set[64] = {};
    if (dev < 64 && !attr_set[dev]) {
        if (cudaError_t e = cudaFuncSetAttribute(project_gemm_few_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 static_cast<int>(kFewSmemBytes));
            e != cudaSuccess)
            return e;
        attr_set[dev] = true;
    }
    const int ntok = (T + 15) / 16 * 16;
    CUtensorMap tX, tP;
    if (!make_map_bf16(&tX, X, T, K, ntok / 2) || !make_map_bf16(&tP, P, K, K, BK)) return cudaErrorInvalidValue;
    Params p;
    p.T = T; p.K = K;
    p.m_tiles = 1;
    p.n_tiles = (K + BN - 1) / BN;
    p.kb_total = (K + BK - 1) / BK;
    p.panel_tiles = 1;
    p.C = C;
    p.status = device_status_ptr();
    p.partial = static_cast<float*>(scratch);
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = p.n_tiles, all_pairs = sms / 2;
    int best_s = 1, best_slice = p.kb_total;
    long best_cost = static_cast<long>((tiles + all_pairs - 1) / all_pairs) * p.kb_total;
    if (scratch) {
        const size_t p_bytes = static_cast<size_t>(K) * K * 2;
        const size_t limit = scratch_bytes < p_bytes / 16 ? scratch_bytes : p_bytes / 16;
        for (int s = 2; s <= p.kb_total / 4; ++s) {
            const int kb_slice = (p.kb_total + s - 1) / s;
            if ((p.kb_total + kb_slice - 1) / kb_slice != s) continue;  // same slices as a smaller s
            if (static_cast<size_t>(tiles) * s * T * BN * sizeof(float) > limit) break;
            const long rounds = (static_cast<long>(tiles) * s + all_pairs - 1) / all_pairs;
            const long cost = rounds * kb_slice;
            if (cost * 50 < best_cost * 49) { best_cost = cost; best_s = s; best_slice = kb_slice; }
        }
    }
    if (best_s > 1) {
        p.full_items = 0; p.split_tiles = tiles; p.splits = best_s; p.kb_slice = best_slice; p.prows = T;
    } else {
        p.full_items = tiles; p.split_tiles = p.splits = p.kb_slice = p.prows = 0;
    }
    const int items = p.full_items + p.split_tiles * p.splits;
    const int pairs = items < all_pairs ? items : all_pairs;
    count_launch();
    project_gemm_few_kernel<<<2 * pairs, kThreads, kFewSmemBytes, st>>>(tX, tP, p, ntok);
    if (cudaError_t le = cudaGetLastError(); le != cudaSuccess) return le;
    if (p.split_tiles > 0) {
        return launch_reduce(p, st);
    }
    return cudaSuccess;
}

}  // namespace

size_t project_split_scratch_bytes() { return static_cast<size_t>(74) * (2 * BM) * BN * sizeof(float); }

cudaError_t launch_project_gemm(const void* X, const void* P, int T, int K, float* C, cudaStream_t st, void* scratch,
                                size_t scratch_bytes) {
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
    if (T <= kFewMaxT) return launch_project_few(X, P, T, K, C, st, scratch, scratch_bytes, dev);
    CUtensorMap tX, tP;
    if (!make_map_bf16(&tX, X, T, K, BM) || !make_map_bf16(&tP, P, K, K, BK)) return cudaErrorInvalidValue;
    Params p;
    p.T = T; p.K = K;
    p.m_tiles = (T + 2 * BM - 1) / (2 * BM);
    p.n_tiles = (K + BN - 1) / BN;
    p.kb_total = (K + BK - 1) / BK;
    // Row panel: as many pair tiles as keep the panel of X (rows x K bf16) within about 64 MB of L2, but 16 at
    // least: the 74 pairs of a round then work on a compact block of tiles (16 x 4-5) whose K slices of X and P are
    // shared while they pass through L2.  Measured at K = 28672 (4096 rows): 5.62 ms with 4-tile panels, 5.41 with 16.
    {
        const size_t tile_bytes = static_cast<size_t>(2 * BM) * K * 2;
        size_t pt = (64u << 20) / tile_bytes;
        if (pt < 16) pt = 16;
        p.panel_tiles = pt > static_cast<size_t>(p.m_tiles) ? p.m_tiles : static_cast<int>(pt);
    }
    p.C = C;
    p.status = device_status_ptr();
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = p.m_tiles * p.n_tiles;
    int pairs = sms / 2;
    if (tiles < pairs) pairs = tiles;
    // A last round that fills less than half of the grid is cut along K so that it takes a fraction of a round:
    // each of its tiles becomes `splits` work items whose partial tiles a second kernel adds up in slice order.
    p.full_items = tiles;
    p.split_tiles = p.splits = p.kb_slice = p.prows = 0;
    p.partial = static_cast<float*>(scratch);
    const int rem = tiles % pairs;
    if (scratch && tiles > pairs && rem > 0 && pairs / rem >= 2) {
        int splits = pairs / rem;
        if (splits > p.kb_total / 4) splits = p.kb_total / 4;  // at least four k-blocks per slice
        const int kb_slice = splits > 0 ? (p.kb_total + splits - 1) / splits : 0;
        if (splits >= 2) splits = (p.kb_total + kb_slice - 1) / kb_slice;  // no empty slice
        if (splits >= 2 && static_cast<size_t>(rem) * splits * (2 * BM) * BN * sizeof(float) <= scratch_bytes) {
            p.full_items = tiles - rem;
            p.split_tiles = rem;
            p.splits = splits;
            p.kb_slice = kb_slice;
            p.prows = 2 * BM;
        }
    }
    count_launch();
    project_gemm_pair_kernel<<<2 * pairs, kThreads, kSmemBytes, st>>>(tX, tP, p);
    if (cudaError_t le = cudaGetLastError(); le != cudaSuccess) return le;
    if (p.split_tiles > 0) return launch_reduce(p, st);
    return cudaSuccess;
}

}  // namespace resq
