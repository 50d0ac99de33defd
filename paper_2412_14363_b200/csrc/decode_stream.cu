// Few-token (T <= 16) mixed-precision GEMM, streaming form: Eq. 4 and its dequantizing epilogue for a
// memory-bound step, where the only cost that matters is reading the packed weights once at HBM rate.
//
// Work split.  The weight rows are cut into units of 8 output channels; CTA b of a persistent grid
// (one CTA per SM) owns a contiguous, balanced range of units.  Inside the CTA the work is the
// sequence of (item, chunk) pairs -- an item is a pair of units (16 channels), a chunk a slice of
// its reduction dimension -- cut into eight equal runs, one per warp.  A warp that holds a whole item
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
// Arithmetic.  mma.sync.m16n8k32 (s8) with the tokens as the 16-row operand (shared by the item's
// two units) and a unit's 8 channels as the 8-column operand; the reduction index may be permuted
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
constexpr int kSmemLimit = 227 * 1024;
constexpr int kControlBytes = 1024;
constexpr int kSlotInts = 2 * 2 * 128;  // [half][acc8 | acc4][fragment element]: one shared item
constexpr int kSlotBytes = kWarps * kSlotInts * 4;
constexpr uint32_t kHi = 0xF0F0F0F0u, kLo = 0x0F0F0F0Fu, kFlip = 0x08080808u;

struct Params {
    int T, N, r, row4;     // row4 = (K - r) / 2: bytes of a packed INT4 weight row
    int c8, c4;            // chunks per row in the INT8 / INT4 segment
    int units;             // N / 8
    int pitch8, pitch4;    // bytes per token of the staged activations (zero padded to whole chunks)
    int nstages;           // stages per warp
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
};

struct __align__(16) Control {
    uint64_t full[kWarps][kMaxStages];
    int s_even[16];  // per token: sum of the even-position INT4 activation codes
    int arrived[kWarps];  // per slot: warps that have added their part
    int abort_flag;
};
static_assert(sizeof(Control) <= kControlBytes, "control block");

// AU: the 16-row operand (the tokens) holds unsigned bytes.
template <bool AU>
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    if constexpr (AU)
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
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

// Two consecutive per-channel scales (channels n, n + 1; n even).
__device__ __forceinline__ float2 load_scale2(const void* p, int n, int fp16) {
    if (fp16) return __half22float2(*reinterpret_cast<const __half2*>(reinterpret_cast<const __half*>(p) + n));
    return *reinterpret_cast<const float2*>(reinterpret_cast<const float*>(p) + n);
}

// TT:     1 for T <= 8 (token rows 8..15 of the 16-row operand are zero and are not staged), 2 for T <= 16.
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
                         const Params p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int TP = TT * 8;
    constexpr int kChunkBytes = CS * 64;
    constexpr int kStageBytes = kItemRows * kChunkBytes;
    Control* ctl = reinterpret_cast<Control*>(smem);
    int* slots = reinterpret_cast<int*>(smem + kControlBytes);                        // [kWarps][kSlotInts]
    uint8_t* act8 = smem + kControlBytes + kSlotBytes;                                // [TP][pitch8]
    uint8_t* act4 = act8 + static_cast<size_t>(TP) * p.pitch8;                        // kSplit: even [TP][pitch4], odd [TP][pitch4]; else packed [TP][pitch4]
    uint8_t* rings = act4 + static_cast<size_t>(kSplit ? 2 : 1) * TP * p.pitch4;      // [kWarps][nstages][16][chunk]
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int u0 = static_cast<int>(static_cast<long long>(p.units) * blockIdx.x / gridDim.x);
    const int u1 = static_cast<int>(static_cast<long long>(p.units) * (blockIdx.x + 1) / gridDim.x);
    const int cta_items = (u1 - u0 + 1) >> 1;
    const int nchunks = p.c8 + p.c4;
    const int cta_chunks = cta_items * nchunks;
    auto run_begin = [&](int w) { return static_cast<int>(static_cast<long long>(cta_chunks) * w / kWarps); };
    const int cb = run_begin(warp), ce = run_begin(warp + 1);  // this warp's run of (item, chunk) pairs
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
    // Issue cursor of this warp (only lane 0 uses it): next (item, chunk) to copy.
    int is_idx = cb, is_item = cb / nchunks, is_chunk = cb - (cb / nchunks) * nchunks;
    auto issue = [&](int stage) {
        const int ub = u0 + 2 * is_item;
        const bool seg8 = is_chunk < p.c8;
        const int x = (seg8 ? is_chunk : is_chunk - p.c8) * (kChunkBytes / 4);  // in 32-bit elements: a multiple of 16
        mbar_arrive_expect_tx(&full[stage], kStageBytes);
        tma_load_2d_hint(ring + static_cast<size_t>(stage) * kStageBytes, seg8 ? &tmW8 : &tmW4, &full[stage], x, ub * kUnitRows,
                         stream_policy);
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
    }
    for (int i = threadIdx.x; i < kWarps * kSlotInts; i += kThreads) slots[i] = 0;
    if (threadIdx.x < kWarps) ctl->arrived[threadIdx.x] = 0;
    if (threadIdx.x == 0) ctl->abort_flag = 0;
    if (p.early_weights) griddep_wait();

    // Token scales of the two accumulator rows this thread holds.
    const float sx8a = g < p.T ? p.s_x8[g] : 0.f, sx4a = g < p.T ? p.s_x4[g] : 0.f;
    const float sx8b = g + 8 < p.T ? p.s_x8[g + 8] : 0.f, sx4b = g + 8 < p.T ? p.s_x4[g + 8] : 0.f;
    const float zx8a = ASYM && g < p.T ? p.z_x8[g] : 0.f, zx4a = ASYM && g < p.T ? p.z_x4[g] : 0.f;
    const float zx8b = ASYM && g + 8 < p.T ? p.z_x8[g + 8] : 0.f, zx4b = ASYM && g + 8 < p.T ? p.z_x4[g + 8] : 0.f;
    // Stage the activation codes: zero padded to the pitch, zero rows for tokens >= T.  The first
    // batch of INT8 and of INT4 vectors is loaded before anything is stored (one round trip to L2 for
    // the usual sizes); the rest of the ring goes out right behind those loads.
    {
        const int v8 = p.pitch8 >> 4, v4 = p.pitch4 >> 4;  // 16-byte vectors per token
        const int r8 = p.r >> 4, r4 = p.row4 >> 4;         // ... that hold data
        const int n8 = TP * v8, n4 = TP * v4;
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
                    *reinterpret_cast<uint4*>(dst + static_cast<size_t>(TP) * p.pitch4) =
                        make_uint4((v[b].x >> 4) & kLo, (v[b].y >> 4) & kLo, (v[b].z >> 4) & kLo, (v[b].w >> 4) & kLo);
                } else if (kSplit) {
                    *reinterpret_cast<uint4*>(dst) =
                        make_uint4((v[b].x << 4) & kHi, (v[b].y << 4) & kHi, (v[b].z << 4) & kHi, (v[b].w << 4) & kHi);
                    *reinterpret_cast<uint4*>(dst + static_cast<size_t>(TP) * p.pitch4) =
                        make_uint4(v[b].x & kHi, v[b].y & kHi, v[b].z & kHi, v[b].w & kHi);
                } else {
                    *reinterpret_cast<uint4*>(dst) = v[b];
                }
            }
        };
        uint4 va[kBatch], vb[kBatch];
        load8(0, va);
        load4(0, vb);
        if (lane == 0) {
            for (int s = issued; s < first_burst; ++s) issue(s);
            issued = first_burst;
        }
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
    __syncthreads();
    // Sum of the even-position INT4 codes per token (warp w: tokens w and w + 8), from the staged rows.
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) {
        const int t = warp + 8 * tt;
        int se = 0;
        if (t < p.T) {
            const uint8_t* row = act4 + static_cast<size_t>(t) * p.pitch4;
            for (int i = lane; i < (p.pitch4 >> 4); i += 32) {
                uint4 v = *reinterpret_cast<const uint4*>(row + (i << 4));
                if (!kSplit) {
                    if (ASYM) v = make_uint4(v.x & kLo, v.y & kLo, v.z & kLo, v.w & kLo);
                    else v = make_uint4((v.x << 4) & kHi, (v.y << 4) & kHi, (v.z << 4) & kHi, (v.w << 4) & kHi);
                }
                se = __dp4a(static_cast<int>(v.x), 0x01010101, se);  // the lanes are < 128 when unsigned
                se = __dp4a(static_cast<int>(v.y), 0x01010101, se);
                se = __dp4a(static_cast<int>(v.z), 0x01010101, se);
                se = __dp4a(static_cast<int>(v.w), 0x01010101, se);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        if (lane == 0) ctl->s_even[t] = ASYM ? se : se >> 4;  // signed codes: the lanes held 16 x the codes
    }
    __syncthreads();
    const int sev_a = ctl->s_even[g], sev_b = TT == 2 ? ctl->s_even[g + 8] : 0;

    const uint8_t* a8row = act8 + static_cast<size_t>(g) * p.pitch8 + 16 * tig;
    const uint8_t* a4row = act4 + static_cast<size_t>(g) * p.pitch4 + 16 * tig;
    const int wofs = g * kChunkBytes + 16 * tig;

    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int consumed = 0;
    int idx = cb, item = cb / nchunks, c = cb - (cb / nchunks) * nchunks;
    while (idx < ce && ok) {
        // One segment: this warp's part of `item` (all of it, or a slice of its chunks).
        const int seg_begin = idx;
        const int ub = u0 + 2 * item;
        const int halves = u1 - ub >= 2 ? 2 : 1;
        const int n0 = ub * kUnitRows + 2 * tig;  // first of this thread's two channels in half 0
        // Channel scales, fetched now and used after the reduction.
        float2 sw8[2], sw4[2];
        int2 ws8[2] = {}, ws4[2] = {};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = h < halves ? n0 + 8 * h : n0;
            sw8[h] = load_scale2(p.s_w8, n, p.w_fp16);
            sw4[h] = load_scale2(p.s_w4, n, p.w_fp16);
            if (ASYM) {
                ws8[h] = *reinterpret_cast<const int2*>(p.wsum8 + n);
                ws4[h] = *reinterpret_cast<const int2*>(p.wsum4 + n);
            }
        }
        int acc8[2][4], accO[2][4], accE[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc8[h][i] = accO[h][i] = accE[h][i] = 0;

        for (; c < nchunks && idx < ce; ++c, ++idx) {
            if (!mbar_wait(&full[stage], phase, abort_flag, p.status)) { ok = false; break; }
            const uint8_t* w0 = ring + static_cast<size_t>(stage) * kStageBytes + wofs;
            const uint8_t* w1 = w0 + 8 * kChunkBytes;
            if (c < p.c8) {
                const uint8_t* xa = a8row + c * kChunkBytes;
#pragma unroll
                for (int s = 0; s < CS; ++s) {
                    const uint4 x = *reinterpret_cast<const uint4*>(xa + 64 * s);
                    uint4 y = make_uint4(0, 0, 0, 0);
                    if (TT == 2) y = *reinterpret_cast<const uint4*>(xa + 8 * p.pitch8 + 64 * s);
                    const uint4 wa = *reinterpret_cast<const uint4*>(w0 + 64 * s);
                    const uint4 wb = *reinterpret_cast<const uint4*>(w1 + 64 * s);
                    mma_s8<ASYM>(acc8[0], x.x, y.x, x.y, y.y, wa.x, wa.y);
                    mma_s8<ASYM>(acc8[1], x.x, y.x, x.y, y.y, wb.x, wb.y);
                    mma_s8<ASYM>(acc8[0], x.z, y.z, x.w, y.w, wa.z, wa.w);
                    mma_s8<ASYM>(acc8[1], x.z, y.z, x.w, y.w, wb.z, wb.w);
                }
            } else {
                const uint8_t* xa = a4row + (c - p.c8) * kChunkBytes;
#pragma unroll
                for (int s = 0; s < CS; ++s) {
                    uint32_t xe[4], xo[4], ye[4], yo[4];
                    if (kSplit) {
                        const uint8_t* xod = xa + static_cast<size_t>(TP) * p.pitch4;
                        const uint4 e = *reinterpret_cast<const uint4*>(xa + 64 * s);
                        const uint4 o = *reinterpret_cast<const uint4*>(xod + 64 * s);
                        xe[0] = e.x; xe[1] = e.y; xe[2] = e.z; xe[3] = e.w;
                        xo[0] = o.x; xo[1] = o.y; xo[2] = o.z; xo[3] = o.w;
                        uint4 e2 = make_uint4(0, 0, 0, 0), o2 = e2;
                        if (TT == 2) {
                            e2 = *reinterpret_cast<const uint4*>(xa + 8 * p.pitch4 + 64 * s);
                            o2 = *reinterpret_cast<const uint4*>(xod + 8 * p.pitch4 + 64 * s);
                        }
                        ye[0] = e2.x; ye[1] = e2.y; ye[2] = e2.z; ye[3] = e2.w;
                        yo[0] = o2.x; yo[1] = o2.y; yo[2] = o2.z; yo[3] = o2.w;
                    } else {
                        const uint4 x = *reinterpret_cast<const uint4*>(xa + 64 * s);
                        uint4 y = make_uint4(0, 0, 0, 0);
                        if (TT == 2) y = *reinterpret_cast<const uint4*>(xa + 8 * p.pitch4 + 64 * s);
                        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (ASYM) {
                                xe[j] = xs[j] & kLo; xo[j] = (xs[j] >> 4) & kLo;
                                ye[j] = ys[j] & kLo; yo[j] = (ys[j] >> 4) & kLo;
                            } else {
                                xe[j] = (xs[j] << 4) & kHi; xo[j] = xs[j] & kHi;
                                ye[j] = (ys[j] << 4) & kHi; yo[j] = ys[j] & kHi;
                            }
                        }
                    }
                    const uint4 wa = *reinterpret_cast<const uint4*>(w0 + 64 * s);
                    const uint4 wb = *reinterpret_cast<const uint4*>(w1 + 64 * s);
                    const uint32_t was[4] = {wa.x, wa.y, wa.z, wa.w}, wbs[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                    for (int j = 0; j < 4; j += 2) {
                        mma_s8<ASYM>(accO[0], xo[j], yo[j], xo[j + 1], yo[j + 1], was[j] & kHi, was[j + 1] & kHi);
                        mma_s8<ASYM>(accE[0], xe[j], ye[j], xe[j + 1], ye[j + 1], even_codes(was[j]), even_codes(was[j + 1]));
                        mma_s8<ASYM>(accO[1], xo[j], yo[j], xo[j + 1], yo[j + 1], wbs[j] & kHi, wbs[j + 1] & kHi);
                        mma_s8<ASYM>(accE[1], xe[j], ye[j], xe[j + 1], ye[j + 1], even_codes(wbs[j]), even_codes(wbs[j + 1]));
                    }
                }
            }
            ++consumed;
            __syncwarp();
            if (lane == 0 && is_idx < ce) {
                ++issued;
                issue(stage);  // refill the stage just read
            }
            if (++stage == p.nstages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;

        // This warp's sums of the segment: acc8 and acc4 + 8 * S_even's share (every shift exact).
        int part[2][2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                part[h][0][i] = acc8[h][i];
                part[h][1][i] = ASYM ? (accO[h][i] >> 4) + accE[h][i] : (accO[h][i] >> 8) + (accE[h][i] >> 4);
            }
        const int item_begin = item * nchunks, item_end = item_begin + nchunks;
        bool finish = true;
        if (seg_begin != item_begin || idx != item_end) {
            // Shared item: its slot belongs to the first warp whose run touches it.
            int first = kWarps, touching = 0;
            for (int w = 0; w < kWarps; ++w) {
                const int b = run_begin(w), e = run_begin(w + 1);
                if (b < e && b < item_end && e > item_begin) {
                    if (first == kWarps) first = w;
                    ++touching;
                }
            }
            int* slot = slots + first * kSlotInts + lane * 4;
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int a = 0; a < 2; ++a)
#pragma unroll
                    for (int i = 0; i < 4; ++i) atomicAdd(slot + (h * 2 + a) * 128 + i, part[h][a][i]);
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
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int i = 0; i < 4; ++i) part[h][a][i] = vs[(h * 2 + a) * 128 + i];
            }
        }
        if (finish) {
            // Epilogue on the fragment this thread holds: element i of half h is token g + 8 * (i >> 1),
            // channel n0 + 8 * h + (i & 1).
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h >= halves) break;
#pragma unroll
                for (int tr = 0; tr < TT; ++tr) {
                    const int t = g + 8 * tr;
                    if (t >= p.T) continue;
                    const float sx8 = tr ? sx8b : sx8a, sx4 = tr ? sx4b : sx4a;
                    const int sev = 8 * (tr ? sev_b : sev_a);
                    const int a8x = part[h][0][2 * tr], a8y = part[h][0][2 * tr + 1];
                    const int a4x = part[h][1][2 * tr] - sev, a4y = part[h][1][2 * tr + 1] - sev;
                    float yx = static_cast<float>(a8x) * (sx8 * sw8[h].x) + static_cast<float>(a4x) * (sx4 * sw4[h].x);
                    float yy = static_cast<float>(a8y) * (sx8 * sw8[h].y) + static_cast<float>(a4y) * (sx4 * sw4[h].y);
                    if (ASYM) {
                        const float zx8 = tr ? zx8b : zx8a, zx4 = tr ? zx4b : zx4a;
                        yx += zx8 * (static_cast<float>(ws8[h].x) * sw8[h].x) + zx4 * (static_cast<float>(ws4[h].x) * sw4[h].x);
                        yy += zx8 * (static_cast<float>(ws8[h].y) * sw8[h].y) + zx4 * (static_cast<float>(ws4[h].y) * sw4[h].y);
                    }
                    const size_t o = static_cast<size_t>(t) * p.N + n0 + 8 * h;
                    if (p.y_dtype == RESQ_Y_BF16)
                        *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(p.Y) + o) = __floats2bfloat162_rn(yx, yy);
                    else
                        *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.Y) + o) = make_float2(yx, yy);
                    if (p.dbg8) {
                        *reinterpret_cast<int2*>(p.dbg8 + o) = make_int2(a8x, a8y);
                        *reinterpret_cast<int2*>(p.dbg4 + o) = make_int2(a4x, a4y);
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
    __syncthreads();
    if (threadIdx.x == 0 && ctl->abort_flag) atomicOr(p.status, kStatusBitTimeout);
}

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][row_bytes] matrix seen as 32-bit elements; box = chunk_bytes x 16 rows, dense in shared
// memory (no swizzle), zero fill out of range.
bool make_map_rows(CUtensorMap* m, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t chunk_bytes) {
    EncodeFn enc = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!enc) return false;
    cuuint64_t dims[2] = {row_bytes / 4, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {chunk_bytes / 4, static_cast<cuuint32_t>(kItemRows)};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int TT, int CS, bool SPLIT, bool ASYM>
cudaError_t launch_variant(const CUtensorMap& t8, const CUtensorMap& t4, const Params& p, int grid, size_t smem,
                           cudaStream_t st) {
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
    return cudaLaunchKernelEx(&cfg, kern, t8, t4, p);
}

}  // namespace

static int g_early_weights = 0;
void set_decode_early_weights(int on) { g_early_weights = on ? 1 : 0; }

// Returns cudaErrorNotSupported (nothing launched) when the staged activations leave no room for the rings.
cudaError_t launch_mixed_gemm_stream(int T, int N, int K, int r, const int8_t* x8, const uint8_t* x4,
                                     const float* s_x8, const float* s_x4, const int8_t* w8, const uint8_t* w4,
                                     const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                     int32_t* dbg8, int32_t* dbg4, cudaStream_t st, const float* z_x8,
                                     const float* z_x4, const int32_t* wsum8, const int32_t* wsum4) {
    const bool asym = z_x8 != nullptr;  // then x8 / x4 hold unsigned codes
    Params p;
    p.T = T; p.N = N; p.r = r; p.row4 = (K - r) / 2;
    p.units = N / kUnitRows;
    const int TT = T <= 8 ? 1 : 2, TP = 8 * TT;
    // Configurations in order of preference: split staging of the INT4 activations before packed
    // for T <= 8 and the reverse above, the
    // larger chunk (5 steps) before the smaller (3 steps); the first that leaves every warp four
    // stages wins, else the last one tried that leaves two.
    int cs = 0, nstages = 0, split = 0;
    size_t fixed = 0;
    bool found = false;
    for (int pass = 0; pass < 2 && !found; ++pass) {
        const int need = pass == 0 ? 4 : kMinStages;
        for (int k = 0; k < 2; ++k) {
            const int sp = TT == 1 ? 1 - k : k;  // measured: split staging pays for T <= 8 only
            for (int c : {5, 3}) {
                const int chunk = 64 * c;
                p.c8 = (r + chunk - 1) / chunk;
                p.c4 = (p.row4 + chunk - 1) / chunk;
                p.pitch8 = round_up(p.c8 * chunk, 128) + 64;
                p.pitch4 = round_up(p.c4 * chunk, 128) + 64;
                fixed = kControlBytes + kSlotBytes + static_cast<size_t>(TP) * p.pitch8 +
                        static_cast<size_t>(sp ? 2 : 1) * TP * p.pitch4;
                cs = c;
                split = sp;
                nstages = fixed < static_cast<size_t>(kSmemLimit)
                              ? static_cast<int>((kSmemLimit - fixed) / kWarps / (static_cast<size_t>(kItemRows) * chunk))
                              : 0;
                if (nstages >= need) { found = true; break; }
            }
            if (found) break;
        }
    }
    if (!found) return cudaErrorNotSupported;
    if (nstages > kMaxStages) nstages = kMaxStages;
    p.nstages = nstages;
    p.early_weights = g_early_weights;
    p.x8 = x8; p.x4 = x4; p.s_x8 = s_x8; p.s_x4 = s_x4; p.s_w8 = s_w8; p.s_w4 = s_w4;
    p.w_fp16 = w_scale_fp16 ? 1 : 0;
    p.z_x8 = z_x8; p.z_x4 = z_x4; p.wsum8 = wsum8; p.wsum4 = wsum4;
    p.Y = Y; p.y_dtype = y_dtype; p.dbg8 = dbg8; p.dbg4 = dbg8 ? dbg4 : nullptr;
    p.status = device_status_ptr();
    const size_t smem = fixed + static_cast<size_t>(kWarps) * nstages * kItemRows * 64 * cs;

    CUtensorMap t8, t4;
    if (!make_map_rows(&t4, w4, N, p.row4, 64 * cs)) return cudaErrorInvalidValue;
    if (r > 0) {
        if (!make_map_rows(&t8, w8, N, r, 64 * cs)) return cudaErrorInvalidValue;
    } else {
        t8 = t4;  // uniform INT4: no INT8 chunks are ever requested
    }
    int dev = 0, sms = 148;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = p.units < sms ? p.units : sms;
    const int variant = (TT == 2 ? 4 : 0) + (cs == 5 ? 2 : 0) + split;
#define RESQ_STREAM_CASE(v, tt, c, sp)                                                               \
    case v:                                                                                          \
        return asym ? launch_variant<tt, c, sp, true>(t8, t4, p, grid, smem, st)                     \
                    : launch_variant<tt, c, sp, false>(t8, t4, p, grid, smem, st);
    switch (variant) {
        RESQ_STREAM_CASE(0, 1, 3, false)
        RESQ_STREAM_CASE(1, 1, 3, true)
        RESQ_STREAM_CASE(2, 1, 5, false)
        RESQ_STREAM_CASE(3, 1, 5, true)
        RESQ_STREAM_CASE(4, 2, 3, false)
        RESQ_STREAM_CASE(5, 2, 3, true)
        RESQ_STREAM_CASE(6, 2, 5, false)
        default:
            return asym ? launch_variant<2, 5, true, true>(t8, t4, p, grid, smem, st)
                        : launch_variant<2, 5, true, false>(t8, t4, p, grid, smem, st);
    }
#undef RESQ_STREAM_CASE
}

}  // namespace resq
