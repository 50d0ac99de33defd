// Few-token (T <= 16) mixed-precision GEMM, streaming form: Eq. 4 and its dequantizing epilogue for a
// memory-bound step, where the only cost that matters is reading the packed weights once at HBM rate.
//
// Work split.  The weight rows are cut into units of 8 output channels; CTA b of a persistent grid
// (one CTA per SM) owns a contiguous, balanced range of units.  Inside the CTA the work is the
// sequence of (item, chunk) pairs -- an item is a pair of units (16 channels; the last item of a CTA
// may be a single unit, whose copies bring 8 rows), a chunk a slice of its reduction dimension -- cut
// into runs of equal cost, one per warp (an INT4 chunk counts about twice an INT8 chunk).  A warp that holds a whole item
// finishes it alone; an item shared by several warps is summed in a shared-memory slot with integer
// atomics and finished by whichever warp arrives last.  Integer sums do not depend on order, so the
// result is the same bit for bit whatever the split; no warp ever waits for another, and there is no
// reduction across CTAs, no global scratch.
//
// Data path.  Every warp runs its own ring of shared-memory stages fed by TMA: one tiled copy per
// stage brings 16 rows x one chunk of a weight row (first the INT8 columns of the item, then its
// packed INT4 columns; out-of-range columns arrive as zeros), completion counted on the stage's
// mbarrier, and the warp refills a stage as soon as it has read it.  The chunk is 192 or 320 bytes,
// = 64 mod 128, so that the dense tile TMA writes is free of bank conflicts for the operand loads
// below.  The rings together are as large as shared memory allows, so the bytes in flight per SM
// do not depend on how fast the arithmetic runs.
//
// Arithmetic.  mma.sync.m16n8k32 (s8) with the item's 16 weight rows (two units) as the 16-row operand and
// up to 8 tokens as the 8-column operand (a second product per step for tokens 9-16), so that a step over
// 64 bytes of each row costs as many products as there are token groups; the reduction index may be permuted
// freely as long as both operands use the same permutation, so each thread simply takes 16
// contiguous bytes of its row.  INT4 codes are never sign-extended one by one.  For a packed word w
// (code 2j in the low, 2j+1 in the high nibble of byte j):
//     w & 0xF0F0F0F0                      the odd codes times 16, as int8 lanes;
//     (w ^ 0x08080808) & 0x0F0F0F0F       the even codes plus 8 (0..15), as int8 lanes;
// the activations enter as their odd / even codes times 16.  The odd products accumulate 256 x their
// true sum, the even ones 16 x (true sum + 8 * sum of the token's even activation codes); that last
// sum is formed once per token, and the epilogue recovers the exact integer
//     acc4 = accO / 256 + accE / 16 - 8 * S_even[t]
// (every division exact; |accO| <= 256 * 49 * (K - r) / 2 < 2^31 for K - r < 342k).  INT4 forms of
// mma.sync compile for this architecture but run some forty times slower than the s8 form.
//
// Overlap with the preceding kernel.  The weights do not depend on it, so with the launch attribute
// for programmatic stream serialization every warp fills its ring at once and only then waits
// (griddepcontrol.wait) for the activations.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kUnitRows = 8;
constexpr int kItemRows = 16;  // two units share the token operand
constexpr int kMaxStages = 8;
constexpr int kMinStages = 2;
constexpr int kEarlyStages = 8;  // ring stages a warp requests before the activations are staged (1: 36.3 us for the 8B block at one token, 2: 33.6, 3: 32.7, 8: 32.5)
constexpr int kSmemLimit = 227 * 1024;
constexpr int kControlBytes = kWarps > 8 ? 2048 : 1024;
constexpr int kSlotInts = 2 * 2 * 128;  // [token group][acc8 | acc4][fragment element]: one shared item
constexpr int kSlotBytes = kWarps * kSlotInts * 4;
constexpr uint32_t kHi = 0xF0F0F0F0u, kLo = 0x0F0F0F0Fu, kFlip = 0x08080808u;

struct Params {
    int T, N, r, row4;     // row4 = (K - r) / 2: bytes of a packed INT4 weight row
    int TR;                // staged activation rows: T, plus a zero row unless the tokens fill their groups of 8
    int c8, c4;            // chunks per row in the INT8 / INT4 segment
    int pitch8, pitch4;    // bytes per token of the staged activations (zero padded to whole chunks)
    int nstages;           // stages per warp
    int ring_ofs;          // byte offset of the rings in shared memory (128-byte aligned)
    int early_weights;     // the launch allows an early start: the rings fill before the wait for the upstream kernel
    const int8_t* x8;
    const uint8_t* x4;
    const float* s_x8;
    const float* s_x4;
    const void* s_w8;
    const void* s_w4;
    int w_fp16;
    // asymmetric activations only (unsigned codes): zero-points per token, row sums of the weight codes
    const float* z_x8;
    const float* z_x4;
    const int32_t* wsum8;
    const int32_t* wsum4;
    void* Y;
    int y_dtype;
    int32_t* dbg8;
    int32_t* dbg4;
    int* status;
    // Work split: CTA b owns units [b * uq + floor(b * urem / grid), ...): uq or uq + 1 of them; tab[0] / tab[1] hold the warps' run
    // boundaries (run_boundary) for those two sizes.
    int uq, urem;
    int tab[2][kWarps + 1];
};

struct __align__(16) Control {
    uint64_t full[kWarps][kMaxStages];
    int s_even[16];  // per token: sum of the even-position INT4 activation codes
    int arrived[kWarps];  // per slot: warps that have added their part
    int abort_flag;
    uint64_t act_bar[kWarps];  // per warp: completion of the bulk copies it issued to stage activation rows (packed staging only)
};
static_assert(sizeof(Control) <= kControlBytes, "control block");

// D (16 x 8, int32) += A (16 x 32, s8: weight rows) * B (32 x 8: token columns; BU: unsigned bytes).
template <bool BU>
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    if constexpr (BU)
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// One per-channel scale: the raw bits now, the value when it is needed (an item's scales are requested when its
// first chunk is, and used after its last: converting at once would make the warp wait for a DRAM round trip
// before it touches the weights that are already in its ring).
__device__ __forceinline__ uint32_t load_scale_raw(const void* p, int n, int fp16) {
    if (fp16) return __ldg(reinterpret_cast<const unsigned short*>(p) + n);
    return __ldg(reinterpret_cast<const uint32_t*>(p) + n);
}
__device__ __forceinline__ float scale_value(uint32_t raw, int fp16) {
    return fp16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(raw))) : __uint_as_float(raw);
}

// floor(a * b / d) for small non-negative a * b (< 2^20) and 0 < d < 2^12, without an integer division: the
// quotient of (a * b + 0.5) by d stays clear of every integer by far more than fp32 rounding.
__device__ __forceinline__ int small_muldiv(int a, int b, int d) {
    return __float2int_rd(__fdividef(static_cast<float>(a * b) + 0.5f, static_cast<float>(d)));
}

// Cost of one chunk in the split of a CTA's work over its warps: an INT4 chunk takes about twice the
// instructions of an INT8 chunk of the same bytes (two products per packed word plus the nibble logic).
constexpr int kCost8 = 4, kCost4 = 7;

// Where the run of warp w begins when the (item, chunk) sequence of a CTA with `items` items is cut into kWarps runs
// of equal cost, packed as item << 16 | chunk; w = kWarps gives the end of the sequence.  Evaluated on the host
// for the two CTA sizes of a launch (Params::tab), so that the kernel's prologue has no divisions.
inline int run_boundary(int w, int items, int c8, int c4) {
    if (w >= kWarps || items == 0) return items << 16;
    const int cf = kCost8 * c8 + kCost4 * c4;
    const long long pos = static_cast<long long>(items) * cf * w / kWarps;
    const int item = static_cast<int>(pos / cf);
    const int q = static_cast<int>(pos - static_cast<long long>(item) * cf);
    const int chunk = q < kCost8 * c8 ? q / kCost8 : c8 + (q - kCost8 * c8) / kCost4;
    return item << 16 | chunk;
}

// TT:     1 for T <= 8 (token rows 8..15 of the 16-row operand are zero), 2 for T <= 16.
// CS:     64-byte steps per chunk (3 or 5).
// kSplit: the INT4 activations are staged already split into their even / odd codes times 16 (twice
//         the shared memory, a third of the logic operations); otherwise they stay packed and are
//         split when used.
// ASYM:   asymmetric activations: the codes are unsigned (0..255, 0..15; Eq. 1, second form).  The INT4
//         activations then enter as their even / odd codes themselves (no factor 16), so
//         acc4 = accO / 16 + accE - 8 * S_even[t], and the epilogue adds the zero-point terms
//         z_x8[t] * s_w8[n] * wsum8[n] + z_x4[t] * s_w4[n] * wsum4[n].
template <int TT, int CS, bool kSplit, bool ASYM>
__global__ void __launch_bounds__(kThreads, 1)
mixed_gemm_stream_kernel(const __grid_constant__ CUtensorMap tmW8, const __grid_constant__ CUtensorMap tmW4,
                         const __grid_constant__ CUtensorMap tmH8, const __grid_constant__ CUtensorMap tmH4,
                         const Params p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int kChunkBytes = CS * 64;
    constexpr int kStageBytes = kItemRows * kChunkBytes;
    Control* ctl = reinterpret_cast<Control*>(smem);
    int* slots = reinterpret_cast<int*>(smem + kControlBytes);                        // [kWarps][kSlotInts]
    // Staged activation codes: rows [0, T) are the tokens, row T (when T is not a multiple of 8) is all zeros: what
    // the token operand reads for its columns beyond T.
    const int TR = p.TR;
    uint8_t* act8 = smem + kControlBytes + kSlotBytes;                                // [T + 1][pitch8]
    uint8_t* act4 = act8 + static_cast<size_t>(TR) * p.pitch8;                        // kSplit: even [T + 1][pitch4], odd [T + 1][pitch4]; else packed [T + 1][pitch4]
    uint8_t* rings = smem + p.ring_ofs;                                               // [kWarps][nstages][16][chunk]
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmW8);
        tma_prefetch_desc(&tmW4);
    }
    const int g = lane >> 2, tig = lane & 3;
    const int bx = static_cast<int>(blockIdx.x);
    const int nbx = static_cast<int>(gridDim.x);
    const int u0 = bx * p.uq + small_muldiv(bx, p.urem, nbx), u1 = (bx + 1) * p.uq + small_muldiv(bx + 1, p.urem, nbx);
    const int big = u1 - u0 - p.uq;                                                   // 1: this CTA owns uq + 1 units
    const int cta_items = (u1 - u0 + 1) >> 1;
    const bool last_half = ((u1 - u0) & 1) != 0;
    const int nchunks = p.c8 + p.c4;
    const int* tab = p.tab[1 - big];
    auto linear = [&](int packed) { return (packed >> 16) * nchunks + (packed & 0xFFFF); };
    const int pb = tab[warp];
    const int cb = linear(pb), ce = linear(tab[warp + 1]);                            // this warp's run of (item, chunk) pairs
    uint8_t* ring = rings + static_cast<size_t>(warp) * p.nstages * kStageBytes;
    uint64_t* full = ctl->full[warp];

    // Each warp owns its barriers, so its lane 0 can start the first copies without a CTA-wide barrier.
    if (lane == 0) {
        for (int s = 0; s < p.nstages; ++s) mbar_init(&full[s], 1);
        fence_mbar_init();
    }
    griddep_launch_dependents();

    // Every weight byte is read once: mark the lines evict-first so that the activations, the scales
    // and whatever the neighbouring kernels keep in L2 stay there.
    const uint64_t stream_policy = l2_policy_evict_first();
    // (w ^ kFlip) & kLo as ONE three-input logic op: the instruction takes a single immediate, so with two
    // compile-time constants the assembler emits an XOR and an AND.  T is positive, which the compiler cannot know:
    // the two words stay in registers.
    const uint32_t never = p.T < 0 ? 1u : 0u;
    const uint32_t rflip = kFlip ^ never, rlo = kLo ^ never;
    auto even_codes = [&](uint32_t w) {
        uint32_t d;
        asm("lop3.b32 %0, %1, %2, %3, 0x28;" : "=r"(d) : "r"(w), "r"(rflip), "r"(rlo));  // (w ^ rflip) & rlo
        return d;
    };
    // Issue cursor of this warp (only lane 0 uses it): next (item, chunk) to copy.  A CTA's last item may be a
    // single unit: its copies bring 8 rows (the maps with the 8-row box) instead of 16.
    int is_idx = cb, is_item = pb >> 16, is_chunk = pb & 0xFFFF;
    auto issue = [&](int stage) {
        const int ub = u0 + 2 * is_item;
        const bool seg8 = is_chunk < p.c8;
        const bool half = last_half && is_item == cta_items - 1;
        const int x = (seg8 ? is_chunk : is_chunk - p.c8) * (kChunkBytes / 4);  // in 32-bit elements: a multiple of 16
        mbar_arrive_expect_tx(&full[stage], half ? kStageBytes / 2 : kStageBytes);
        const CUtensorMap* tm = half ? (seg8 ? &tmH8 : &tmH4) : (seg8 ? &tmW8 : &tmW4);
        tma_load_2d_hint(ring + static_cast<size_t>(stage) * kStageBytes, tm, &full[stage], x, ub * kUnitRows, stream_policy);
        ++is_idx;
        if (++is_chunk == nchunks) { is_chunk = 0; ++is_item; }
    };

    if (!p.early_weights) griddep_wait();
    int issued = 0;
    // One stage per warp goes out now; the rest follow once the (small, latency-critical) activation
    // loads below have been issued, so that those do not queue behind a full ring of weight traffic.
    const int first_burst = ce - cb < p.nstages ? ce - cb : p.nstages;
    if (lane == 0 && first_burst > 0) {
        issue(0);
        issued = 1;
        if (p.early_weights >= 2) {  // nothing of the preceding kernel is read before the wait below: fill the ring now
            for (int s = 1; s < first_burst; ++s) issue(s);
            issued = first_burst;
        }
    }
    for (int i = threadIdx.x; i < kWarps * kSlotInts; i += kThreads) slots[i] = 0;
    if (threadIdx.x < kWarps) ctl->arrived[threadIdx.x] = 0;
    if (threadIdx.x == 0) ctl->abort_flag = 0;
    if (p.early_weights) griddep_wait();

    // The tokens are the 8 columns of the product (one group of 8 per TT): this thread feeds the codes of token g
    // (and g + 8) and holds the sums of tokens 2 tig, 2 tig + 1 (and + 8).  Their scales and zero-points:
    const bool a_ok = g < p.T, b_ok = TT == 2 && g + 8 < p.T;
    float sx8t[TT][2], sx4t[TT][2], zx8t[TT][2], zx4t[TT][2];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int t = 8 * tt + 2 * tig + e;
            const bool t_ok = t < p.T;
            sx8t[tt][e] = t_ok ? p.s_x8[t] : 0.f;
            sx4t[tt][e] = t_ok ? p.s_x4[t] : 0.f;
            zx8t[tt][e] = ASYM && t_ok ? p.z_x8[t] : 0.f;
            zx4t[tt][e] = ASYM && t_ok ? p.z_x4[t] : 0.f;
        }
    // Stage the activation codes of the T tokens, zero padded to the pitch (the weights arrive as zeros there, but an
    // even INT4 weight code enters the product as code + 8), and the zero row.  The first batch of INT8 and
    // of INT4 vectors is loaded before anything is stored (one round trip to L2 for the usual sizes); the rest of
    // the ring goes out right behind those loads.  Meanwhile warp w sums the even-position INT4 codes of tokens
    // w and w + 8 straight from global memory.
    {
        const int v8 = p.pitch8 >> 4, v4 = p.pitch4 >> 4;  // 16-byte vectors per token
        const int r8 = p.r >> 4, r4 = p.row4 >> 4;         // ... that hold data
        const int n8 = TR * v8, n4 = TR * v4;
        constexpr int kBatch = 4;
        auto load8 = [&](int base, uint4 (&v)[kBatch]) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int i = base + b * kThreads + threadIdx.x;
                const int t = i / v8, o = i - t * v8;
                v[b] = make_uint4(0, 0, 0, 0);
                if (i < n8 && t < p.T && o < r8) v[b] = __ldg(reinterpret_cast<const uint4*>(p.x8 + static_cast<size_t>(t) * p.r) + o);
            }
        };
        auto store8 = [&](int base, const uint4 (&v)[kBatch]) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int i = base + b * kThreads + threadIdx.x;
                if (i >= n8) continue;
                const int t = i / v8, o = i - t * v8;
                *reinterpret_cast<uint4*>(act8 + static_cast<size_t>(t) * p.pitch8 + (o << 4)) = v[b];
            }
        };
        auto load4 = [&](int base, uint4 (&v)[kBatch]) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int i = base + b * kThreads + threadIdx.x;
                const int t = i / v4, o = i - t * v4;
                v[b] = make_uint4(0, 0, 0, 0);
                if (i < n4 && t < p.T && o < r4) v[b] = __ldg(reinterpret_cast<const uint4*>(p.x4 + static_cast<size_t>(t) * p.row4) + o);
            }
        };
        auto store4 = [&](int base, const uint4 (&v)[kBatch]) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int i = base + b * kThreads + threadIdx.x;
                if (i >= n4) continue;
                const int t = i / v4, o = i - t * v4;
                uint8_t* dst = act4 + static_cast<size_t>(t) * p.pitch4 + (o << 4);
                if (kSplit && ASYM) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(v[b].x & kLo, v[b].y & kLo, v[b].z & kLo, v[b].w & kLo);
                    *reinterpret_cast<uint4*>(dst + static_cast<size_t>(TR) * p.pitch4) =
                        make_uint4((v[b].x >> 4) & kLo, (v[b].y >> 4) & kLo, (v[b].z >> 4) & kLo, (v[b].w >> 4) & kLo);
                } else if (kSplit) {
                    *reinterpret_cast<uint4*>(dst) =
                        make_uint4((v[b].x << 4) & kHi, (v[b].y << 4) & kHi, (v[b].z << 4) & kHi, (v[b].w << 4) & kHi);
                    *reinterpret_cast<uint4*>(dst + static_cast<size_t>(TR) * p.pitch4) =
                        make_uint4(v[b].x & kHi, v[b].y & kHi, v[b].z & kHi, v[b].w & kHi);
                } else {
                    *reinterpret_cast<uint4*>(dst) = v[b];
                }
            }
        };
        uint4 va[kBatch], vb[kBatch];
        if constexpr (kSplit) {
            load8(0, va);
            load4(0, vb);
        } else {
            // Packed staging needs no arithmetic: one bulk copy per token row and segment, all in flight at once
            // (16 rows of a 14336-wide layer are 129 KB), issued by the lanes of the last warp; the threads only
            // write the zeros behind the rows and the zero row.
            // Copy i of the 2 T copies (token i / 2, INT8 segment when i is even) is issued by lane i / kWarps of
            // warp i % kWarps: a warp's copies complete on its own barrier, and no warp issues more than four.
            {
                const int mine = (2 * p.T - warp + kWarps - 1) / kWarps;  // copies i = warp + kWarps * l, l < mine
                if (lane == 0) {
                    uint32_t bytes = 0;
                    for (int l = 0; l < mine; ++l) {
                        const int i = warp + kWarps * l;
                        bytes += (i & 1) ? static_cast<uint32_t>(p.row4) : static_cast<uint32_t>(p.r);
                    }
                    mbar_init(&ctl->act_bar[warp], 1);
                    fence_mbar_init();
                    mbar_arrive_expect_tx(&ctl->act_bar[warp], bytes);
                }
                __syncwarp();
                if (lane < mine) {
                    const int i = warp + kWarps * lane, t = i >> 1;
                    if ((i & 1) == 0) {
                        if (p.r > 0) bulk_load(act8 + static_cast<size_t>(t) * p.pitch8, p.x8 + static_cast<size_t>(t) * p.r, p.r, &ctl->act_bar[warp]);
                    } else {
                        bulk_load(act4 + static_cast<size_t>(t) * p.pitch4, p.x4 + static_cast<size_t>(t) * p.row4, p.row4, &ctl->act_bar[warp]);
                    }
                }
            }
            const int pv8 = v8 - r8, pv = pv8 + v4 - r4;  // vectors behind the data of a row: INT8, both segments
            const uint4 z = make_uint4(0, 0, 0, 0);
            for (int i = threadIdx.x; i < p.T * pv; i += kThreads) {
                const int t = i / pv, o = i - t * pv;
                if (o < pv8) *reinterpret_cast<uint4*>(act8 + static_cast<size_t>(t) * p.pitch8 + ((r8 + o) << 4)) = z;
                else *reinterpret_cast<uint4*>(act4 + static_cast<size_t>(t) * p.pitch4 + ((r4 + o - pv8) << 4)) = z;
            }
            if (TR > p.T)
                for (int i = threadIdx.x; i < v8 + v4; i += kThreads) {
                    if (i < v8) *reinterpret_cast<uint4*>(act8 + static_cast<size_t>(p.T) * p.pitch8 + (i << 4)) = z;
                    else *reinterpret_cast<uint4*>(act4 + static_cast<size_t>(p.T) * p.pitch4 + ((i - v8) << 4)) = z;
                }
        }
        // Sum of the even-position INT4 codes per token, from the global rows (up to four vectors in flight per lane).
        constexpr int kTokIters = (8 * TT + kWarps - 1) / kWarps;
        int se[kTokIters];
#pragma unroll
        for (int tt = 0; tt < kTokIters; ++tt) {
            const int t = warp + kWarps * tt;
            se[tt] = 0;
            if (t < p.T) {
                const uint4* row = reinterpret_cast<const uint4*>(p.x4 + static_cast<size_t>(t) * p.row4);
                for (int i0 = 0; i0 < r4; i0 += 128) {
                    uint4 v[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int i = i0 + 32 * k + lane;
                        v[k] = i < r4 ? __ldg(row + i) : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 q = v[k];
                        if (ASYM) q = make_uint4(q.x & kLo, q.y & kLo, q.z & kLo, q.w & kLo);
                        else q = make_uint4((q.x << 4) & kHi, (q.y << 4) & kHi, (q.z << 4) & kHi, (q.w << 4) & kHi);
                        se[tt] = __dp4a(static_cast<int>(q.x), 0x01010101, se[tt]);  // the lanes are < 128 when unsigned
                        se[tt] = __dp4a(static_cast<int>(q.y), 0x01010101, se[tt]);
                        se[tt] = __dp4a(static_cast<int>(q.z), 0x01010101, se[tt]);
                        se[tt] = __dp4a(static_cast<int>(q.w), 0x01010101, se[tt]);
                    }
                }
            }
        }
        if (lane == 0) {
            // Part of the ring now, the rest once the activations are staged: a copy instruction waits for room in
            // the SM's copy queue, and a warp held there holds up the barrier below and with it the first product.
            const int now = first_burst < kEarlyStages ? first_burst : kEarlyStages;
            for (int s = issued; s < now; ++s) issue(s);
            if (issued < now) issued = now;
        }
        if constexpr (kSplit) {
            store8(0, va);
            store4(0, vb);
            for (int base = kBatch * kThreads; base < n8; base += kBatch * kThreads) {
                load8(base, va);
                store8(base, va);
            }
            for (int base = kBatch * kThreads; base < n4; base += kBatch * kThreads) {
                load4(base, vb);
                store4(base, vb);
            }
        }
#pragma unroll
        for (int tt = 0; tt < kTokIters; ++tt) {
            int v = se[tt];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0 && warp + kWarps * tt < p.T) ctl->s_even[warp + kWarps * tt] = ASYM ? v : v >> 4;  // signed codes: the lanes held 16 x the codes
        }
    }
    __syncthreads();
    bool ok = true;
    if constexpr (!kSplit) {  // the staged rows have landed
#pragma unroll 1
        for (int w = 0; w < kWarps && ok; ++w) ok = mbar_wait(&ctl->act_bar[w], 0, abort_flag, p.status);
    }
    int sevt[TT][2];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt)
#pragma unroll
        for (int e = 0; e < 2; ++e) sevt[tt][e] = 8 * tt + 2 * tig + e < p.T ? ctl->s_even[8 * tt + 2 * tig + e] : 0;

    const uint8_t* a8row = act8 + static_cast<size_t>(a_ok ? g : p.T) * p.pitch8 + 16 * tig;
    const uint8_t* a4row = act4 + static_cast<size_t>(a_ok ? g : p.T) * p.pitch4 + 16 * tig;
    const uint8_t* b8row = act8 + static_cast<size_t>(b_ok ? g + 8 : p.T) * p.pitch8 + 16 * tig;
    const uint8_t* b4row = act4 + static_cast<size_t>(b_ok ? g + 8 : p.T) * p.pitch4 + 16 * tig;
    const size_t odd_ofs = static_cast<size_t>(TR) * p.pitch4;  // kSplit: the odd codes follow the even ones
    const int wofs = g * kChunkBytes + 16 * tig;

    int stage = 0;
    uint32_t phase = 0;
    int consumed = 0;
    int iss_stage = issued == p.nstages ? 0 : issued;  // the stage the next copy goes into (lane 0)
    int idx = cb, item = pb >> 16, c = pb & 0xFFFF;
    while (idx < ce && ok) {
        // One segment: this warp's part of `item` (all of it, or a slice of its chunks).
        const int seg_begin = idx;
        const int ub = u0 + 2 * item;
        const int halves = u1 - ub >= 2 ? 2 : 1;
        const int n0 = ub * kUnitRows + g;  // this thread's channel in unit 0 of the item (unit 1: + 8)
        // Channel scales, fetched now and used after the reduction.
        uint32_t rw8[2], rw4[2];
        int ws8[2] = {}, ws4[2] = {};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = h < halves ? n0 + 8 * h : n0;
            rw8[h] = load_scale_raw(p.s_w8, n, p.w_fp16);
            rw4[h] = load_scale_raw(p.s_w4, n, p.w_fp16);
            if (ASYM) {
                ws8[h] = __ldg(p.wsum8 + n);
                ws4[h] = __ldg(p.wsum4 + n);
            }
        }
        // Sums of this warp's part of the item: element i of group tt is unit i >> 1 (channel n0 + 8 (i >> 1)),
        // token 8 tt + 2 tig + (i & 1).
        // With one token group a step issues two products per accumulator, each waiting for the one before: the two
        // halves of a step then go to accumulators of their own (kAcc = 2), which halves the dependent chain.
        constexpr int kAcc = TT == 1 ? 2 : 1;
        int acc8[TT][kAcc][4], accO[TT][kAcc][4], accE[TT][kAcc][4];
#pragma unroll
        for (int tt = 0; tt < TT; ++tt)
#pragma unroll
            for (int a = 0; a < kAcc; ++a)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc8[tt][a][i] = accO[tt][a][i] = accE[tt][a][i] = 0;

        for (; c < nchunks && idx < ce; ++c, ++idx) {
            if (!mbar_wait(&full[stage], phase, abort_flag, p.status)) { ok = false; break; }
            const uint8_t* w0 = ring + static_cast<size_t>(stage) * kStageBytes + wofs;
            const uint8_t* w1 = w0 + 8 * kChunkBytes;  // a single unit: stale rows, their sums are never used
            if (c < p.c8) {
                const int co = c * kChunkBytes;
#pragma unroll
                for (int s = 0; s < CS; ++s) {
                    const uint4 wa = *reinterpret_cast<const uint4*>(w0 + 64 * s);
                    const uint4 wb = *reinterpret_cast<const uint4*>(w1 + 64 * s);
                    const uint4 x = *reinterpret_cast<const uint4*>(a8row + co + 64 * s);
                    mma_s8<ASYM>(acc8[0][0], wa.x, wb.x, wa.y, wb.y, x.x, x.y);
                    mma_s8<ASYM>(acc8[0][kAcc - 1], wa.z, wb.z, wa.w, wb.w, x.z, x.w);
                    if (TT == 2) {
                        const uint4 y = *reinterpret_cast<const uint4*>(b8row + co + 64 * s);
                        mma_s8<ASYM>(acc8[TT - 1][0], wa.x, wb.x, wa.y, wb.y, y.x, y.y);
                        mma_s8<ASYM>(acc8[TT - 1][0], wa.z, wb.z, wa.w, wb.w, y.z, y.w);
                    }
                }
            } else {
                const int co = (c - p.c8) * kChunkBytes;
#pragma unroll
                for (int s = 0; s < CS; ++s) {
                    const uint4 wa = *reinterpret_cast<const uint4*>(w0 + 64 * s);
                    const uint4 wb = *reinterpret_cast<const uint4*>(w1 + 64 * s);
                    // odd codes times 16 / even codes plus 8 of the two units' rows: the A fragments of two products
                    const uint32_t ao[8] = {wa.x & kHi, wb.x & kHi, wa.y & kHi, wb.y & kHi, wa.z & kHi, wb.z & kHi, wa.w & kHi, wb.w & kHi};
                    const uint32_t ae[8] = {even_codes(wa.x), even_codes(wb.x), even_codes(wa.y), even_codes(wb.y),
                                            even_codes(wa.z), even_codes(wb.z), even_codes(wa.w), even_codes(wb.w)};
#pragma unroll
                    for (int tt = 0; tt < TT; ++tt) {
                        const uint8_t* row = tt == 0 ? a4row : b4row;
                        uint32_t xe[4], xo[4];
                        if (kSplit) {
                            const uint4 e = *reinterpret_cast<const uint4*>(row + co + 64 * s);
                            const uint4 o = *reinterpret_cast<const uint4*>(row + odd_ofs + co + 64 * s);
                            xe[0] = e.x; xe[1] = e.y; xe[2] = e.z; xe[3] = e.w;
                            xo[0] = o.x; xo[1] = o.y; xo[2] = o.z; xo[3] = o.w;
                        } else {
                            const uint4 x = *reinterpret_cast<const uint4*>(row + co + 64 * s);
                            const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (ASYM) { xe[j] = xs[j] & kLo; xo[j] = (xs[j] >> 4) & kLo; }
                                else { xe[j] = (xs[j] << 4) & kHi; xo[j] = xs[j] & kHi; }
                            }
                        }
                        mma_s8<ASYM>(accO[tt][0], ao[0], ao[1], ao[2], ao[3], xo[0], xo[1]);
                        mma_s8<ASYM>(accE[tt][0], ae[0], ae[1], ae[2], ae[3], xe[0], xe[1]);
                        mma_s8<ASYM>(accO[tt][kAcc - 1], ao[4], ao[5], ao[6], ao[7], xo[2], xo[3]);
                        mma_s8<ASYM>(accE[tt][kAcc - 1], ae[4], ae[5], ae[6], ae[7], xe[2], xe[3]);
                    }
                }
            }
            ++consumed;
            __syncwarp();
            if (lane == 0) {
                // Copies go into the ring's stages in order.  One per chunk read keeps a full ring full; until the
                // ring is as deep as it gets, two per chunk read: it deepens while the first chunks are consumed
                // instead of holding up the first product.
                for (int k = 0; k < 2 && is_idx < ce && issued - consumed < p.nstages; ++k) {
                    issue(iss_stage);
                    if (++iss_stage == p.nstages) iss_stage = 0;
                    ++issued;
                }
            }
            if (++stage == p.nstages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;

        // This warp's sums of the segment: acc8 and acc4 + 8 * S_even's share (every shift exact).
        int part[TT][2][4];
#pragma unroll
        for (int tt = 0; tt < TT; ++tt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int s8 = acc8[tt][0][i] + (kAcc == 2 ? acc8[tt][kAcc - 1][i] : 0);
                const int sO = accO[tt][0][i] + (kAcc == 2 ? accO[tt][kAcc - 1][i] : 0);
                const int sE = accE[tt][0][i] + (kAcc == 2 ? accE[tt][kAcc - 1][i] : 0);
                part[tt][0][i] = s8;
                part[tt][1][i] = ASYM ? (sO >> 4) + sE : (sO >> 8) + (sE >> 4);
            }
        const int item_begin = item * nchunks, item_end = item_begin + nchunks;
        bool finish = true;
        if (seg_begin != item_begin || idx != item_end) {
            // Shared item: its slot belongs to the first warp whose run touches it.
            int first = kWarps, touching = 0;
            for (int w = 0; w < kWarps; ++w) {
                const int b = linear(tab[w]), e = linear(tab[w + 1]);
                if (b < e && b < item_end && e > item_begin) {
                    if (first == kWarps) first = w;
                    ++touching;
                }
            }
            int* slot = slots + first * kSlotInts + lane * 4;
#pragma unroll
            for (int tt = 0; tt < TT; ++tt)
#pragma unroll
                for (int a = 0; a < 2; ++a)
#pragma unroll
                    for (int i = 0; i < 4; ++i) atomicAdd(slot + (tt * 2 + a) * 128 + i, part[tt][a][i]);
            __threadfence_block();
            __syncwarp();
            int prev = 0;
            if (lane == 0) prev = atomicAdd(&ctl->arrived[first], 1);
            prev = __shfl_sync(0xffffffffu, prev, 0);
            finish = prev == touching - 1;
            if (finish) {
                __threadfence_block();
                const volatile int* vs = slot;
#pragma unroll
                for (int tt = 0; tt < TT; ++tt)
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int i = 0; i < 4; ++i) part[tt][a][i] = vs[(tt * 2 + a) * 128 + i];
            }
        }
        if (finish) {
            // Epilogue on the fragment this thread holds.
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h >= halves) break;
                const float sw8h = scale_value(rw8[h], p.w_fp16), sw4h = scale_value(rw4[h], p.w_fp16);
                const int n = n0 + 8 * h;
#pragma unroll
                for (int tt = 0; tt < TT; ++tt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int t = 8 * tt + 2 * tig + e;
                        if (t >= p.T) continue;
                        const int a8v = part[tt][0][2 * h + e];
                        const int a4v = part[tt][1][2 * h + e] - 8 * sevt[tt][e];
                        float y = static_cast<float>(a8v) * (sx8t[tt][e] * sw8h) + static_cast<float>(a4v) * (sx4t[tt][e] * sw4h);
                        if (ASYM)
                            y += zx8t[tt][e] * (static_cast<float>(ws8[h]) * sw8h) + zx4t[tt][e] * (static_cast<float>(ws4[h]) * sw4h);
                        const size_t o = static_cast<size_t>(t) * p.N + n;
                        if (p.y_dtype == RESQ_Y_BF16) reinterpret_cast<__nv_bfloat16*>(p.Y)[o] = __float2bfloat16_rn(y);
                        else reinterpret_cast<float*>(p.Y)[o] = y;
                        if (p.dbg8) {
                            p.dbg8[o] = a8v;
                            p.dbg4[o] = a4v;
                        }
                    }
            }
        }
        c = 0;
        ++item;
    }

    if (!ok && lane == 0) {
        // Let the copies already in flight land before the CTA gives up its shared memory.
        const int pending = issued - consumed;
        for (int k = 0; k < pending; ++k) {
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(&full[stage], phase) && global_timer_ns() - t0 < 100000000ull) {}
            if (++stage == p.nstages) { stage = 0; phase ^= 1; }
        }
    }
    if (!kSplit && !ok && threadIdx.x == kThreads - 32) {
        const uint64_t t0 = global_timer_ns();
        for (int w = 0; w < kWarps; ++w)
            while (!mbar_try_wait(&ctl->act_bar[w], 0) && global_timer_ns() - t0 < 100000000ull) {}
    }
    __syncthreads();
    if (threadIdx.x == 0 && ctl->abort_flag) atomicOr(p.status, kStatusBitTimeout);
}

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][row_bytes] matrix seen as 32-bit elements; box = chunk_bytes x box_rows rows (16 for an item, 8 for a
// single unit), dense in shared memory (no swizzle), zero fill out of range.
bool make_map_rows(CUtensorMap* m, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t chunk_bytes,
                   uint32_t box_rows = kItemRows) {
    EncodeFn enc = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!enc) return false;
    cuuint64_t dims[2] = {row_bytes / 4, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {chunk_bytes / 4, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int TT, int CS, bool SPLIT, bool ASYM>
cudaError_t launch_variant(const CUtensorMap (&tm)[4], const Params& p, int grid, size_t smem, cudaStream_t st) {
    auto kern = mixed_gemm_stream_kernel<TT, CS, SPLIT, ASYM>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.early_weights ? 1 : 0;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], p);
}

// How a launch cuts its work and its shared memory: chunk width, staging form, ring depth, grid.
struct Plan {
    int TT, TR, cs, split, nstages, c8, c4, pitch8, pitch4, units, grid;
    size_t fixed, smem;
    bool ok;
};

Plan make_plan(int T, int N, int K, int r, int sms) {
    Plan pl = {};
    const int row4 = (K - r) / 2;
    pl.units = N / kUnitRows;
    if (pl.units >= (1 << 24)) return pl;  // the kernel's 32-bit unit arithmetic
    pl.TT = T <= 8 ? 1 : 2;
    pl.TR = T % 8 == 0 ? T : T + 1;  // a zero row for the token columns beyond T
    // Configurations in order of preference: split staging of the INT4 activations before packed for T <= 8 and the
    // reverse above, the larger chunk (5 steps) before the smaller (3 steps); the first that leaves every warp four
    // stages wins, else the last one tried that leaves two.
    for (int pass = 0; pass < 2 && !pl.ok; ++pass) {
        const int need = pass == 0 ? 4 : kMinStages;
        for (int k = 0; k < 2 && !pl.ok; ++k) {
            const int sp = pl.TT == 1 ? 1 - k : k;  // measured: split staging pays for T <= 8 only
            for (int c : {5, 3}) {
                const int chunk = 64 * c;
                pl.c8 = (r + chunk - 1) / chunk;
                pl.c4 = (row4 + chunk - 1) / chunk;
                pl.pitch8 = round_up(pl.c8 * chunk, 128) + 64;
                pl.pitch4 = round_up(pl.c4 * chunk, 128) + 64;
                pl.fixed = static_cast<size_t>(round_up(static_cast<int>(kControlBytes + kSlotBytes + static_cast<size_t>(pl.TR) * pl.pitch8 +
                                                                         static_cast<size_t>(sp ? 2 : 1) * pl.TR * pl.pitch4), 128));
                pl.cs = c;
                pl.split = sp;
                pl.nstages = pl.fixed < static_cast<size_t>(kSmemLimit)
                                 ? static_cast<int>((kSmemLimit - pl.fixed) / kWarps / (static_cast<size_t>(kItemRows) * chunk))
                                 : 0;
                if (pl.nstages >= need) { pl.ok = true; break; }
            }
        }
    }
    if (!pl.ok) return pl;
    if (pl.nstages > kMaxStages) pl.nstages = kMaxStages;
    pl.smem = pl.fixed + static_cast<size_t>(kWarps) * pl.nstages * kItemRows * 64 * pl.cs;
    pl.grid = pl.units < sms ? pl.units : sms;
    return pl;
}

// Units per CTA (`urem` CTAs, spread evenly over the grid, own one more) and the warps' run boundaries for the two CTA sizes.
void fill_split(const Plan& pl, int& uq, int& urem, int (&tab)[2][kWarps + 1]) {
    uq = pl.units / pl.grid;
    urem = pl.units % pl.grid;
    for (int k = 0; k < 2; ++k)
        for (int w = 0; w <= kWarps; ++w) tab[k][w] = run_boundary(w, (uq + 1 - k + 1) >> 1, pl.c8, pl.c4);
}

}  // namespace

static int g_early_weights = 0;
void set_decode_early_weights(int on) { g_early_weights = on < 0 ? 0 : (on > 2 ? 2 : on); }

// Returns cudaErrorNotSupported (nothing launched) when the staged activations leave no room for the rings.
cudaError_t launch_mixed_gemm_stream(int T, int N, int K, int r, const int8_t* x8, const uint8_t* x4,
                                     const float* s_x8, const float* s_x4, const int8_t* w8, const uint8_t* w4,
                                     const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                     int32_t* dbg8, int32_t* dbg4, cudaStream_t st, const float* z_x8,
                                     const float* z_x4, const int32_t* wsum8, const int32_t* wsum4) {
    const bool asym = z_x8 != nullptr;  // then x8 / x4 hold unsigned codes
    int dev = 0, sms = 148;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const Plan pl = make_plan(T, N, K, r, sms);
    if (!pl.ok) return cudaErrorNotSupported;
    Params p;
    p.T = T; p.N = N; p.r = r; p.row4 = (K - r) / 2;
    p.TR = pl.TR;
    fill_split(pl, p.uq, p.urem, p.tab);
    p.c8 = pl.c8; p.c4 = pl.c4; p.pitch8 = pl.pitch8; p.pitch4 = pl.pitch4;
    p.nstages = pl.nstages;
    p.ring_ofs = static_cast<int>(pl.fixed);
    p.early_weights = g_early_weights;
    p.x8 = x8; p.x4 = x4; p.s_x8 = s_x8; p.s_x4 = s_x4; p.s_w8 = s_w8; p.s_w4 = s_w4;
    p.w_fp16 = w_scale_fp16 ? 1 : 0;
    p.z_x8 = z_x8; p.z_x4 = z_x4; p.wsum8 = wsum8; p.wsum4 = wsum4;
    p.Y = Y; p.y_dtype = y_dtype; p.dbg8 = dbg8; p.dbg4 = dbg8 ? dbg4 : nullptr;
    p.status = device_status_ptr();

    // Maps: [0], [1] INT8 / INT4 weights with the 16-row box of an item, [2], [3] the same with the 8-row box of a
    // single unit.
    CUtensorMap tm[4];
    CUtensorMap &t8 = tm[0], &t4 = tm[1];
    if (!make_map_rows(&t4, w4, N, p.row4, 64 * pl.cs) || !make_map_rows(&tm[3], w4, N, p.row4, 64 * pl.cs, kUnitRows))
        return cudaErrorInvalidValue;
    if (r > 0) {
        if (!make_map_rows(&t8, w8, N, r, 64 * pl.cs) || !make_map_rows(&tm[2], w8, N, r, 64 * pl.cs, kUnitRows))
            return cudaErrorInvalidValue;
    } else {
        t8 = t4;  // uniform INT4: no INT8 chunks are ever requested
        tm[2] = tm[3];
    }
    const int variant = (pl.TT == 2 ? 4 : 0) + (pl.cs == 5 ? 2 : 0) + pl.split;
#define RESQ_STREAM_CASE(v, tt, c, sp)                                                               \
    case v:                                                                                          \
        return asym ? launch_variant<tt, c, sp, true>(tm, p, pl.grid, pl.smem, st)       \
                    : launch_variant<tt, c, sp, false>(tm, p, pl.grid, pl.smem, st);
    switch (variant) {
        RESQ_STREAM_CASE(0, 1, 3, false)
        RESQ_STREAM_CASE(1, 1, 3, true)
        RESQ_STREAM_CASE(2, 1, 5, false)
        RESQ_STREAM_CASE(3, 1, 5, true)
        RESQ_STREAM_CASE(4, 2, 3, false)
        RESQ_STREAM_CASE(5, 2, 3, true)
        RESQ_STREAM_CASE(6, 2, 5, false)
        default:
            return asym ? launch_variant<2, 5, true, true>(tm, p, pl.grid, pl.smem, st)
                        : launch_variant<2, 5, true, false>(tm, p, pl.grid, pl.smem, st);
    }
#undef RESQ_STREAM_CASE
}

}  // namespace resq
