// Single-query attention over the mixed-precision KV cache (Section 4.3, Eq. 8; Section 5.1).  HBM-bound: every
// 5632-byte cache block (32 positions of one KV head: key and value codes, scales, zero-points) is read once.
//
// Work.  Blocks are numbered in (sequence, KV head, block) order; the 148 x 12 warps of the persistent grid
// each take an equal contiguous run of that list.  A warp owns a ring of three block-sized stages filled by
// bulk copies that its lane 0 issues (one copy per block, completion on the warp's own mbarriers), so no
// CTA-wide barrier exists after start-up.  Whenever the run leaves a (sequence, head) the warp writes one
// partial record (running maximum, sum of weights, unnormalised output) for the query heads of that KV head;
// a second small kernel merges the records of each (sequence, query head).
//
// Arithmetic.  The codes never become dequantized values.  With q8/q4 the two segments of a query head,
//     q . k_hat = s8 (q8 . c8) + z8 sum(q8) + s4 (q4 . c4) + z4 sum(q4),
//     sum_j p_j v_hat_j = sum_j (p_j s_j) c_j + sum_j p_j z_j          (per segment),
// so both products contract fp16 queries / weights with integer codes on mma.sync m16n8k16 (codes are exact
// in half: 1024 + c and 64 + c are built with one logic op on the packed bytes or nibbles; the offsets are
// removed from the fp32 sums afterwards).  Positions are the M rows of the score product (8 query heads of a group as N) and the
// K rows of the output product (16 coefficients as M), so the score accumulators only need an 8x8 transpose
// (movmatrix) to become the second product's B fragments.  Scores, the running softmax and all sums are
// fp32; the weights p_j s_j are scaled by a power of two taken from the value scales so that they stay in
// half's range whatever the magnitude of V.
#include <cuda_fp16.h>

#include "internal.h"
#include "ptx.cuh"
#include "../../include/resq_kv.h"

namespace resq {
namespace {

constexpr int kD = 128;
constexpr int kWarps = 12;
constexpr int kStages = 3;
constexpr int kBlk = RESQ_KV_BLOCK_BYTES;
constexpr int kOffK8 = 0, kOffK4 = 512, kOffKM = 2304, kOffV8 = 2816, kOffV4 = 3328, kOffVM = 5120;
constexpr int kNumWarps = 148 * kWarps;  // the grid is always 148 CTAs
constexpr int kRecFloats = 8 * (kD + 2);  // per query head of the group: m, l, 128 outputs
constexpr float kLog2eOverSqrtD = 0.12751743f;  // log2(e) / sqrt(128)

struct AttnParams {
    const uint8_t* cache;
    const __half* q;
    const int32_t* seq_lens;
    const int32_t* seq_map;  // NULL: query row b reads cache sequence b; else the cache sequence of query row b
    float* partial;
    float* out;
    int* status;
    int n_seqs, n_kv_heads, group, capacity;  // n_seqs: query rows (= cache sequences when seq_map is NULL)
    int n_cache_seqs;
};

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ int clamped_len(const int32_t* seq_lens, int b, int capacity) {
    const int len = seq_lens[b];
    return len < 0 ? 0 : (len > capacity ? capacity : len);
}

// Whole warp: returns the number of blocks per head summed over all sequences.  If target >= 0, also finds the
// sequence that holds global block `target` (the list has n_kv_heads times the per-head blocks of each
// sequence) and the per-head blocks of all sequences before it.
__device__ __forceinline__ long long scan_blocks(const AttnParams& p, int lane, long long target, int* b_out,
                                                 long long* before_out) {
    long long base = 0;
    bool found = false;
    for (int b0 = 0; b0 < p.n_seqs; b0 += 32) {
        const int b = b0 + lane;
        const int t = b < p.n_seqs ? (clamped_len(p.seq_lens, b, p.capacity) + 31) >> 5 : 0;
        int incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (target >= 0 && !found) {
            const unsigned m = __ballot_sync(0xffffffffu, (base + incl) * p.n_kv_heads > target);
            if (m) {
                const int l = __ffs(m) - 1;
                *b_out = b0 + l;
                *before_out = base + __shfl_sync(0xffffffffu, incl - t, l);
                found = true;
            }
        }
        base += __shfl_sync(0xffffffffu, incl, 31);
    }
    return base;
}

struct Cursor {  // one block of the global list
    int b, h, blk, nblk, len;
};
__device__ __forceinline__ void advance(Cursor& cu, const AttnParams& p) {
    if (++cu.blk < cu.nblk) return;
    cu.blk = 0;
    if (++cu.h < p.n_kv_heads) return;
    cu.h = 0;
    do {
        if (++cu.b >= p.n_seqs) { cu.nblk = 0; cu.len = 0; return; }
        cu.len = clamped_len(p.seq_lens, cu.b, p.capacity);
        cu.nblk = (cu.len + 31) >> 5;
    } while (cu.nblk == 0);
}

// Codes as half2 operands WITH an offset: one logic op puts a code into the mantissa of 1024.0 (ulp 1) or of
// 64.0 (ulp 1/16, for a nibble sitting in bits 4-7), giving 1024 + c or 64 + c exactly.  The offsets are not
// subtracted per element: they add offset * sum(other operand) to a product, which is removed once per
// position (scores) or once per record (outputs, via a product with an all-ones operand).
constexpr float kOffLo = 1024.f, kOffHi = 64.f;
constexpr float kMid8 = 128.f, kMid4 = 8.f;  // centres of the code ranges
constexpr float kSlack = 8.f;  // log2 of the largest softmax weight before the reference is raised
// Two codes held in bits 0-3 / 16-19 (lo) or 4-7 / 20-23 (hi) of w: (w & mask) | exponent as ONE three-input
// logic op.  That needs mask and exponent in registers (the instruction takes a single immediate, and with two
// compile-time constants the assembler emits an AND and an OR), so the kernel derives the four words from a
// run-time value once and passes them around in this struct.
struct NibbleConsts {
    uint32_t mask_lo, exp_lo, mask_hi, exp_hi;
};
__device__ __forceinline__ uint32_t and_or(uint32_t w, uint32_t mask, uint32_t bits) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(w), "r"(mask), "r"(bits));  // (w & mask) | bits
    return d;
}
#define nib_lo(w) and_or((w), nc.mask_lo, nc.exp_lo)
#define nib_hi(w) and_or((w), nc.mask_hi, nc.exp_hi)
// Two bytes of w (picked by SEL), each with 0x64 as the upper byte of its half: 1024 + c.
template <uint32_t SEL>
__device__ __forceinline__ uint32_t bytes_h2(uint32_t w) { return __byte_perm(w, 0x64646464u, SEL); }

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(x));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t lds32(const uint8_t* p) { return *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ uint32_t lds16(const uint8_t* p) { return *reinterpret_cast<const uint16_t*>(p); }

// Coefficient index behind entry e (k = 2c, 2c + 1, 2c + 8, 2c + 9) of contraction step j of the score product,
// as the key-side extraction delivers them: step 0 is the 8-bit segment (bytes 4c..4c+3 of the position's 16),
// steps 1-6 take two steps per 32-bit word c + 4i of the 4-bit codes (nibbles (0,4),(1,5) then (2,6),(3,7)),
// step 7 the nibbles (0,2),(1,3) of half-word 24 + c.
__device__ __forceinline__ int kdim(int j, int c, int e) {
    if (j == 0) return 4 * c + e;
    if (j == 7) return 112 + 4 * c + ((e & 1) << 1) + (e >> 1);
    const int i = (j - 1) >> 1, sub = (j - 1) & 1;
    return 16 + 8 * (c + 4 * i) + 2 * sub + ((e & 1) << 2) + (e >> 1);
}

struct ValueScale {  // per position: value scales times 2^-E (E: the block's exponent), zero-points
    float sn8, sn4, z8, z4;
};
__device__ __forceinline__ ValueScale value_scale(const uint8_t* vm, int tok, float i2e) {
    const float4 m = *reinterpret_cast<const float4*>(vm + tok * 16);
    ValueScale v;
    v.sn8 = m.x * i2e;
    v.sn4 = m.z * i2e;
    v.z8 = m.y;
    v.z4 = m.w;
    return v;
}
// First product of a chain: C = 0.
__device__ __forceinline__ void mma_f16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

__global__ void __launch_bounds__(kWarps * 32, 1) attention_decode_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t rings[];
    __shared__ uint64_t full_s[kWarps][kStages];
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    uint8_t* ring = rings + static_cast<size_t>(warp) * kStages * kBlk;
    uint64_t* full = full_s[warp];
    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
        fence_mbar_init();
    }
    if (threadIdx.x == 0) abort_flag = 0;
    __syncthreads();
    griddep_launch_dependents();  // the merge kernel may be scheduled as SMs free up; it waits for this grid itself

    // ---- this warp's run of the global block list
    const long long wg = static_cast<long long>(blockIdx.x) * kWarps + warp;
    int b_first = 0;
    long long before = 0;
    const long long total = scan_blocks(p, lane, -1, &b_first, &before) * p.n_kv_heads;
    const long long start = total * wg / kNumWarps, end = total * (wg + 1) / kNumWarps, n = end - start;
    if (n <= 0) return;
    scan_blocks(p, lane, start, &b_first, &before);
    Cursor cons;
    cons.b = b_first;
    cons.len = clamped_len(p.seq_lens, b_first, p.capacity);
    cons.nblk = (cons.len + 31) >> 5;
    {
        const long long local = start - before * p.n_kv_heads;
        cons.h = static_cast<int>(local / cons.nblk);
        cons.blk = static_cast<int>(local - static_cast<long long>(cons.h) * cons.nblk);
    }
    Cursor prod = cons;
    const int blocks_cap = p.capacity / RESQ_KV_BLOCK;
    auto issue = [&](int stage) {  // lane 0 copies the producer cursor's block; every lane moves the cursor
        if (lane == 0) {
            int cb = prod.b;
            if (p.seq_map) {
                cb = p.seq_map[prod.b];
                if (cb < 0 || cb >= p.n_cache_seqs) {  // reported by the merge kernel; read a valid block meanwhile
                    cb = 0;
                }
            }
            const uint8_t* src = p.cache + ((static_cast<long long>(cb) * p.n_kv_heads + prod.h) * blocks_cap + prod.blk) * kBlk;
            mbar_arrive_expect_tx(&full[stage], kBlk);
            bulk_load(ring + stage * kBlk, src, kBlk, &full[stage]);
        }
        advance(prod, p);
    };
    long long issued = 0;
    for (; issued < n && issued < kStages; ++issued) issue(static_cast<int>(issued));

    // capacity is positive; the compiler cannot know, so the four words stay in registers (see NibbleConsts)
    const uint32_t never = p.capacity < 0 ? 1u : 0u;
    const NibbleConsts nc{0x000F000Fu ^ never, 0x64006400u ^ never, 0x00F000F0u ^ never, 0x54005400u ^ never};
    uint32_t qf[8][2];
    float kq8[2], kq4[2], ko8[2], ko4[2], m_run[2], l[2], z8[2], z4[2], acc[8][4], ones8[4], ones4[4], wx8[2], wx4[2];
    bool fresh = true, ok = true;
    int rec_blk0 = 0;  // block of the (sequence, head) at which the current record began
    long long i = 0;
    int stage = 0;
    uint32_t phase = 0;
    for (; i < n; ++i) {
        if (fresh) {  // a new (sequence, KV head): query fragments of its group, empty running state
            fresh = false;
            rec_blk0 = cons.blk;
            const __half* qrow = p.q + (static_cast<long long>(cons.b) * p.n_kv_heads * p.group + cons.h * p.group + g) * kD;
            float s8 = 0.f, s4 = 0.f, o4 = 0.f;  // sums of q over the segments; offset-weighted sum of the 4-bit part
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    __half2 v = __floats2half2_rn(0.f, 0.f);
                    if (g < p.group) v = __halves2half2(qrow[kdim(j, c, 2 * hf)], qrow[kdim(j, c, 2 * hf + 1)]);
                    qf[j][hf] = *reinterpret_cast<const uint32_t*>(&v);
                    const float2 f = __half22float2(v);
                    if (j == 0) s8 += f.x + f.y;
                    else { s4 += f.x + f.y; o4 += (hf == 0 ? kOffLo : kOffHi) * (f.x + f.y); }  // entries 0-1 lo, 2-3 hi
                }
            s8 += __shfl_xor_sync(0xffffffffu, s8, 1); s8 += __shfl_xor_sync(0xffffffffu, s8, 2);
            s4 += __shfl_xor_sync(0xffffffffu, s4, 1); s4 += __shfl_xor_sync(0xffffffffu, s4, 2);
            o4 += __shfl_xor_sync(0xffffffffu, o4, 1); o4 += __shfl_xor_sync(0xffffffffu, o4, 2);
#pragma unroll
            for (int e = 0; e < 2; ++e) {  // the score fragment's columns are heads 2c, 2c + 1
                kq8[e] = kLog2eOverSqrtD * __shfl_sync(0xffffffffu, s8, 4 * (2 * c + e));
                kq4[e] = kLog2eOverSqrtD * __shfl_sync(0xffffffffu, s4, 4 * (2 * c + e));
                ko8[e] = kOffLo * kq8[e];
                ko4[e] = kLog2eOverSqrtD * __shfl_sync(0xffffffffu, o4, 4 * (2 * c + e));
                m_run[e] = -INFINITY; l[e] = z8[e] = z4[e] = ones8[e] = ones4[e] = ones8[2 + e] = ones4[2 + e] = wx8[e] = wx4[e] = 0.f;
            }
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
        }
        if (!mbar_wait(&full[stage], phase, &abort_flag, p.status)) { ok = false; break; }
        const uint8_t* st = ring + stage * kBlk;
        const int valid = min(RESQ_KV_BLOCK, cons.len - RESQ_KV_BLOCK * cons.blk);
        if (valid < RESQ_KV_BLOCK) {  // last block of a sequence: the unused slots hold anything -- zero their value scales
            if (lane >= valid) *reinterpret_cast<float4*>(ring + stage * kBlk + kOffVM + lane * 16) = make_float4(0.f, 0.f, 0.f, 0.f);
            __syncwarp();
        }
        // ---- the block's exponent: E from the largest value scale, clamped to 2^-64 .. 2^64 (0 scales included)
        float e_blk, i2e;
        {
            const float4 vm = *reinterpret_cast<const float4*>(st + kOffVM + lane * 16);
            uint32_t eb = __reduce_max_sync(0xffffffffu, __float_as_uint(fmaxf(fmaxf(vm.x, vm.z), 0.f))) & 0x7F800000u;
            eb = min(max(eb, 63u << 23), 191u << 23);
            i2e = __uint_as_float((254u << 23) - eb);
            e_blk = static_cast<float>(static_cast<int>(eb >> 23) - 127);
        }

        // ---- scores of the 32 positions (two 16-row products), in log2 units, plus the block's exponent
        float sc[2][4];
        ValueScale vs[2][2];
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const int tokA = 16 * m + 2 * g, tokB = tokA + 1;  // rows g and g + 8 of the product
            float d8[4], d4[4], d4b[4];  // two chains for the 4-bit steps
            {
                const uint32_t wa = lds32(st + kOffK8 + tokA * 16 + 4 * c), wb = lds32(st + kOffK8 + tokB * 16 + 4 * c);
                mma_f16_first(d8, bytes_h2<0x4140>(wa), bytes_h2<0x4140>(wb), bytes_h2<0x4342>(wa), bytes_h2<0x4342>(wb),
                              qf[0][0], qf[0][1]);
            }
#pragma unroll
            for (int i3 = 0; i3 < 3; ++i3) {
                uint32_t wa = lds32(st + kOffK4 + tokA * 56 + 4 * (c + 4 * i3)), wb = lds32(st + kOffK4 + tokB * 56 + 4 * (c + 4 * i3));
                if (i3 == 0) mma_f16_first(d4, nib_lo(wa), nib_lo(wb), nib_hi(wa), nib_hi(wb), qf[1][0], qf[1][1]);
                else mma_f16(d4, nib_lo(wa), nib_lo(wb), nib_hi(wa), nib_hi(wb), qf[1 + 2 * i3][0], qf[1 + 2 * i3][1]);
                wa >>= 8; wb >>= 8;
                if (i3 == 0) mma_f16_first(d4b, nib_lo(wa), nib_lo(wb), nib_hi(wa), nib_hi(wb), qf[2][0], qf[2][1]);
                else mma_f16(d4b, nib_lo(wa), nib_lo(wb), nib_hi(wa), nib_hi(wb), qf[2 + 2 * i3][0], qf[2 + 2 * i3][1]);
            }
            {
                uint32_t xa = lds16(st + kOffK4 + tokA * 56 + 48 + 2 * c), xb = lds16(st + kOffK4 + tokB * 56 + 48 + 2 * c);
                xa = __byte_perm(xa, 0u, 0x4110); xb = __byte_perm(xb, 0u, 0x4110);  // nibbles 2, 3 up to bits 16-23
                mma_f16(d4b, nib_lo(xa), nib_lo(xb), nib_hi(xa), nib_hi(xb), qf[7][0], qf[7][1]);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) d4[e] += d4b[e];
            const float4 kmA = *reinterpret_cast<const float4*>(st + kOffKM + tokA * 16);
            const float4 kmB = *reinterpret_cast<const float4*>(st + kOffKM + tokB * 16);
            vs[m][0] = value_scale(st + kOffVM, tokA, i2e);
            vs[m][1] = value_scale(st + kOffVM, tokB, i2e);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                // d8, d4 carry the code offsets: remove offset * sum(q) (ko8, ko4) before the key scales apply
                const float sA = kmA.x * fmaf(kLog2eOverSqrtD, d8[e], -ko8[e]) + kmA.z * fmaf(kLog2eOverSqrtD, d4[e], -ko4[e]) +
                                 kmA.y * kq8[e] + kmA.w * kq4[e] + e_blk;
                const float sB = kmB.x * fmaf(kLog2eOverSqrtD, d8[2 + e], -ko8[e]) + kmB.z * fmaf(kLog2eOverSqrtD, d4[2 + e], -ko4[e]) +
                                 kmB.y * kq8[e] + kmB.w * kq4[e] + e_blk;
                sc[m][e] = sA;
                sc[m][2 + e] = sB;
            }
        }
        if (valid < RESQ_KV_BLOCK) {  // unused slots of a sequence's last block take no weight
#pragma unroll
            for (int m = 0; m < 2; ++m)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (16 * m + 2 * g >= valid) sc[m][e] = -INFINITY;
                    if (16 * m + 2 * g + 1 >= valid) sc[m][2 + e] = -INFINITY;
                }
        }
        // ---- reference exponent per head (columns 2c, 2c + 1), shared by the 8 lanes with this c.  It is raised to
        // the running maximum only when some score exceeds it by more than kSlack (and at a record's first block,
        // where it is -inf), so the usual block needs one vote instead of a shuffle reduction; meanwhile weights reach
        // at most 2^kSlack, far inside half's range.
        {
            const float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][2]), fmaxf(sc[1][0], sc[1][2]));
            const float mx1 = fmaxf(fmaxf(sc[0][1], sc[0][3]), fmaxf(sc[1][1], sc[1][3]));
            if (__any_sync(0xffffffffu, mx0 > m_run[0] + kSlack || mx1 > m_run[1] + kSlack)) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float mx = e == 0 ? mx0 : mx1;
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                    const float mn = fmaxf(m_run[e], mx);
                    const float a = ex2(m_run[e] - mn);
                    l[e] *= a; z8[e] *= a; z4[e] *= a; ones8[e] *= a; ones4[e] *= a; ones8[2 + e] *= a; ones4[2 + e] *= a;
                    wx8[e] *= a; wx4[e] *= a;
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) { acc[mt][e] *= a; acc[mt][2 + e] *= a; }
                    m_run[e] = mn;
                }
            }
        }
        // ---- weights, their transposes as B fragments, and the output products
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            float p8[2][2], p4[2][2];
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const ValueScale& v = vs[m][t];
                    const float pw = ex2(sc[m][2 * t + e] - m_run[e]);
                    const float w = pw * i2e;
                    l[e] += w; z8[e] = fmaf(w, v.z8, z8[e]); z4[e] = fmaf(w, v.z4, z4[e]);
                    p8[t][e] = pw * v.sn8; p4[t][e] = pw * v.sn4;
                    wx8[e] += p8[t][e]; wx4[e] += p4[t][e];  // the unrounded weights, for the centring below
                }
            const uint32_t b80 = movmatrix_trans(pack_h2(p8[0][0], p8[0][1])), b81 = movmatrix_trans(pack_h2(p8[1][0], p8[1][1]));
            const uint32_t b40 = movmatrix_trans(pack_h2(p4[0][0], p4[0][1])), b41 = movmatrix_trans(pack_h2(p4[1][0], p4[1][1]));
            {   // sum of the (rounded) weights per head, for the code offsets: a product with an all-ones operand
                mma_f16(ones8, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, b80, b81);  // all 16 rows alike
                mma_f16(ones4, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, b40, b41);
            }
            const int t0 = 16 * m + 4 * c;  // contraction entries 2c, 2c+1, 2c+8, 2c+9 are positions t0, t0+2, t0+1, t0+3
            {
                const uint8_t* v8 = st + kOffV8 + t0 * 16 + 2 * g;
                const uint32_t w02 = __byte_perm(lds16(v8), lds16(v8 + 32), 0x5410), w13 = __byte_perm(lds16(v8 + 16), lds16(v8 + 48), 0x5410);
                mma_f16(acc[0], bytes_h2<0x4240>(w02), bytes_h2<0x4341>(w02), bytes_h2<0x4240>(w13), bytes_h2<0x4341>(w13), b80, b81);
            }
#pragma unroll
            for (int i3 = 0; i3 < 3; ++i3) {
                const uint8_t* v4 = st + kOffV4 + t0 * 56 + 2 * (g + 8 * i3);
                uint32_t w02 = __byte_perm(lds16(v4), lds16(v4 + 112), 0x5410), w13 = __byte_perm(lds16(v4 + 56), lds16(v4 + 168), 0x5410);
                mma_f16(acc[1 + 2 * i3], nib_lo(w02), nib_hi(w02), nib_lo(w13), nib_hi(w13), b40, b41);
                w02 >>= 8; w13 >>= 8;
                mma_f16(acc[2 + 2 * i3], nib_lo(w02), nib_hi(w02), nib_lo(w13), nib_hi(w13), b40, b41);
            }
            {
                const uint8_t* v4 = st + kOffV4 + t0 * 56 + 48 + g;
                const uint32_t w02 = __byte_perm(v4[0], v4[112], 0x5410), w13 = __byte_perm(v4[56], v4[168], 0x5410);
                mma_f16(acc[7], nib_lo(w02), nib_hi(w02), nib_lo(w13), nib_hi(w13), b40, b41);
            }
        }
        __syncwarp();
        if (issued < n) {  // refill the stage just read
            issue(stage);
            ++issued;
        }
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
        // ---- leaving this (sequence, head), or the run: one partial record
        if (cons.blk == cons.nblk - 1 || i == n - 1) {
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    l[e] += __shfl_xor_sync(0xffffffffu, l[e], o);
                    z8[e] += __shfl_xor_sync(0xffffffffu, z8[e], o);
                    z4[e] += __shfl_xor_sync(0xffffffffu, z4[e], o);
                    wx8[e] += __shfl_xor_sync(0xffffffffu, wx8[e], o);
                    wx4[e] += __shfl_xor_sync(0xffffffffu, wx4[e], o);
                }
            // A warp that saw every block of the (sequence, head) writes the final output itself (the merge kernel
            // finds a single owner by the same run arithmetic and leaves at once); otherwise a partial record.
            const bool sole = rec_blk0 == 0 && cons.blk == cons.nblk - 1;
            float* rec = p.partial + (wg + static_cast<long long>(cons.b) * p.n_kv_heads + cons.h) * kRecFloats;
            float* fin = p.out + (static_cast<long long>(cons.b) * p.n_kv_heads + cons.h) * p.group * kD;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (2 * c + e >= p.group) continue;
                float* r = sole ? fin + (2 * c + e) * kD : rec + (2 * c + e) * (kD + 2) + 2;
                const float nrm = sole ? 1.f / l[e] : 1.f;
                if (!sole && g == 0) { r[-2] = m_run[e]; r[-1] = l[e]; }
                // Rows g of the output products carry offset kOffLo, rows g + 8 kOffLo (8-bit) or kOffHi (4-bit).  The
                // codes are also centred: sum w^ (c - mid) + mid * sum w with w^ the half-rounded and w the exact
                // weights (ones: sum w^, wx: sum w), which halves the effect of the rounding (|c - mid| <= range / 2).
                const float f8 = z8[e] - (kOffLo + kMid8) * ones8[e] + kMid8 * wx8[e];
                const float f4lo = z4[e] - (kOffLo + kMid4) * ones4[e] + kMid4 * wx4[e];
                const float f4hi = z4[e] - (kOffHi + kMid4) * ones4[e] + kMid4 * wx4[e];
                r[2 * g] = (acc[0][e] + f8) * nrm;
                r[2 * g + 1] = (acc[0][2 + e] + f8) * nrm;
#pragma unroll
                for (int i3 = 0; i3 < 3; ++i3) {
                    const int d0 = 16 + 4 * (g + 8 * i3);
                    r[d0] = (acc[1 + 2 * i3][e] + f4lo) * nrm;
                    r[d0 + 1] = (acc[1 + 2 * i3][2 + e] + f4hi) * nrm;
                    r[d0 + 2] = (acc[2 + 2 * i3][e] + f4lo) * nrm;
                    r[d0 + 3] = (acc[2 + 2 * i3][2 + e] + f4hi) * nrm;
                }
                r[112 + 2 * g] = (acc[7][e] + f4lo) * nrm;
                r[113 + 2 * g] = (acc[7][2 + e] + f4hi) * nrm;
            }
            fresh = true;
        }
        advance(cons, p);
    }
    if (!ok) {  // a wait ran out: let this warp's copies in flight land (bounded), then report
        for (long long k = i; k < issued; ++k) {
            const int stage = static_cast<int>(k % kStages);
            const uint32_t phase = static_cast<uint32_t>(k / kStages) & 1u;
            for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&full[stage], phase); ++spin) {}
        }
        if (lane == 0) atomicOr(p.status, kStatusBitTimeout);
    }
}

// Merges the partial records of one (sequence, query head): out = sum_i 2^(m_i - M) o_i / sum_i 2^(m_i - M) l_i.
// The warps that hold a record of this (sequence, KV head) are those whose runs meet its range of the block
// list.  The CTA has 128 x G threads: candidates are taken blockDim at a time (thread t reads (m, l) of candidate
// t, the block agrees on the maximum), then group g adds the weighted records g, g + G, ... eight at a time, one
// output coefficient per thread, and the G partial sums are added in group order.  G = 4 when few (sequence, head)
// pairs share the grid's warps (long contexts: hundreds of records each), else 1.  Launched so that it may start
// while the attention kernel drains: everything before griddepcontrol.wait reads only the sequence lengths.
constexpr int kMaxGroups = 4;
__global__ void __launch_bounds__(kD * kMaxGroups) attention_combine_kernel(const AttnParams p) {
    __shared__ long long red[2][kD * kMaxGroups / 32];
    __shared__ float redf[2][kD * kMaxGroups / 32];
    extern __shared__ __align__(16) uint8_t merge_smem[];  // rec_s [nthr] long long, f_s [nthr] float, num_s [groups][128] float
    const int n_q_heads = p.n_kv_heads * p.group;
    const int b = blockIdx.x / n_q_heads, hq = blockIdx.x - b * n_q_heads;
    const int hk = hq / p.group, hg = hq - hk * p.group;
    const int tid = threadIdx.x, nthr = blockDim.x, nwarp = nthr >> 5, warp = tid >> 5;
    const int d = tid & (kD - 1), grp = tid >> 7, groups = nthr >> 7;
    long long* rec_s = reinterpret_cast<long long*>(merge_smem);
    float* f_s = reinterpret_cast<float*>(rec_s + nthr);
    float* num_s = f_s + nthr;
    long long before = 0, total = 0;
    for (int i = tid; i < p.n_seqs; i += nthr) {
        const int len = p.seq_lens[i];
        if (blockIdx.x == 0 && (len < 0 || len > p.capacity)) atomicOr(p.status, kStatusBitIndex);
        if (blockIdx.x == 0 && p.seq_map && (p.seq_map[i] < 0 || p.seq_map[i] >= p.n_cache_seqs)) atomicOr(p.status, kStatusBitIndex);
        const int t = ((len < 0 ? 0 : (len > p.capacity ? p.capacity : len)) + 31) >> 5;
        total += t;
        if (i < b) before += t;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if ((tid & 31) == 0) { red[0][warp] = before; red[1][warp] = total; }
    __syncthreads();
    before = total = 0;
    for (int w = 0; w < nwarp; ++w) { before += red[0][w]; total += red[1][w]; }
    total *= p.n_kv_heads;
    float* out = p.out + (static_cast<long long>(b) * n_q_heads + hq) * kD;
    const int nblk = (clamped_len(p.seq_lens, b, p.capacity) + 31) >> 5;
    // Every CTA waits for the attention grid before it returns, also those with nothing to merge: this grid was
    // launched as a programmatic dependent, so the next kernel of the stream is ordered against THIS grid only,
    // and it must not retire while the attention grid is still writing `out`.
    griddep_wait();
    if (nblk == 0) {  // empty sequence
        if (grp == 0) out[d] = 0.f;
        return;
    }
    const long long lo = before * p.n_kv_heads + static_cast<long long>(hk) * nblk, hi = lo + nblk;  // [lo, hi)
    constexpr long long nw = kNumWarps;
    const int w_first = static_cast<int>(((lo + 1) * nw - 1) / total), w_last = static_cast<int>((hi * nw - 1) / total);
    if (w_first == w_last) return;  // one warp saw the whole (sequence, head) and wrote the output itself
    const long long s = static_cast<long long>(b) * p.n_kv_heads + hk;
    float M = -INFINITY, num = 0.f, den = 0.f;  // num: this group's share; den: a per-thread partial until the end
    for (int w0 = w_first; w0 <= w_last; w0 += nthr) {
        const int w = w0 + tid;
        bool have = false;
        if (w <= w_last) {  // a non-empty run that meets [lo, hi)
            const long long rs = total * w / nw, re = total * (w + 1) / nw;
            have = re > rs && re > lo && rs < hi;
        }
        const long long off = (w + s) * kRecFloats + hg * (kD + 2);
        float m = -INFINITY, lw = 0.f;
        if (have) { m = __ldcg(p.partial + off); lw = __ldcg(p.partial + off + 1); }
        float mx = m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        __syncthreads();  // the previous chunk's f_s / rec_s / redf are no longer read
        if ((tid & 31) == 0) redf[0][warp] = mx;
        __syncthreads();
        float Mn = M;
        for (int k = 0; k < nwarp; ++k) Mn = fmaxf(Mn, redf[0][k]);
        const float resc = ex2(M - Mn);  // 0 on the first chunk
        M = Mn;
        const float f = have ? ex2(m - M) : 0.f;
        f_s[tid] = f;
        rec_s[tid] = have ? off + 2 : -1;
        num *= resc;
        den = fmaf(f, lw, den * resc);
        __syncthreads();
        const int cnt = min(nthr, w_last - w0 + 1);
        for (int i0 = 8 * grp; i0 < cnt; i0 += 8 * groups) {
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const long long r = i0 + k < cnt ? rec_s[i0 + k] : -1;
                v[k] = r >= 0 ? __ldcg(p.partial + r + d) : 0.f;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) num = fmaf(i0 + k < cnt ? f_s[i0 + k] : 0.f, v[k], num);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    __syncthreads();
    if ((tid & 31) == 0) redf[1][warp] = den;
    num_s[grp * kD + d] = num;
    __syncthreads();
    if (grp == 0) {
        float dsum = 0.f, nsum = 0.f;
        for (int k = 0; k < nwarp; ++k) dsum += redf[1][k];
        for (int g = 0; g < groups; ++g) nsum += num_s[g * kD + d];
        out[d] = nsum / dsum;
    }
}

}  // namespace

size_t attention_scratch_bytes(int n_seqs, int n_kv_heads) {
    return (static_cast<size_t>(kNumWarps) + static_cast<size_t>(n_seqs) * n_kv_heads) * kRecFloats * sizeof(float);
}

cudaError_t launch_attention_decode(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, const int32_t* seq_lens,
                                    float* out, void* scratch, cudaStream_t st, int n_rows, const int32_t* seq_map) {
    if (n_rows < 0) n_rows = cache.n_seqs;  // single-query form: one query row per cache sequence
    static bool configured[64] = {};
    int dev = 0;
    if (cudaError_t e = cudaGetDevice(&dev); e != cudaSuccess) return e;
    constexpr int kSmem = kWarps * kStages * kBlk;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaError_t e = cudaFuncSetAttribute(attention_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
            e != cudaSuccess)
            return e;
        configured[dev] = true;
    }
    AttnParams p{};
    p.cache = static_cast<const uint8_t*>(cache.data);
    p.q = static_cast<const __half*>(q16);
    p.seq_lens = seq_lens;
    p.partial = static_cast<float*>(scratch);
    p.out = out;
    p.status = device_status_ptr();
    p.seq_map = seq_map;
    p.n_seqs = n_rows;
    p.n_cache_seqs = cache.n_seqs;
    p.n_kv_heads = cache.n_kv_heads;
    p.group = n_q_heads / cache.n_kv_heads;
    p.capacity = cache.capacity;
    count_launch(2);
    attention_decode_kernel<<<148, kWarps * 32, kSmem, st>>>(p);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_rows * n_q_heads, 1, 1);
    // few (sequence, head) pairs share the grid's warps: each has many records, so four groups of threads add them
    const int merge_threads = n_rows * cache.n_kv_heads <= 64 ? kD * kMaxGroups : kD;
    cfg.blockDim = dim3(merge_threads, 1, 1);
    cfg.dynamicSmemBytes = static_cast<size_t>(merge_threads) * (sizeof(long long) + sizeof(float)) + (merge_threads / kD) * kD * sizeof(float);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, attention_combine_kernel, p);
}

}  // namespace resq
