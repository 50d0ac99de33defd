// Few-token (T <= 16) mixed-precision GEMM, streaming form: Eq. 4 and its dequantizing epilogue for a
// memory-bound step, where the only cost that matters is reading the packed weights once at HBM rate.
//
// Work split.  The weight rows are cut into units of 8 output channels; CTA b of a persistent grid
// (one CTA per SM) owns a contiguous, balanced range of units and walks through it alone, so there
// is no reduction across CTAs, no scratch and no atomics, and the result does not depend on the grid.
//
// Data path.  A producer thread streams each unit through a ring of shared-memory stages with bulk
// copies (8 rows x up to 2048 bytes per stage, completion counted on an mbarrier), first the INT8
// columns, then the packed INT4 columns.  The ring is as deep as shared memory allows, so the bytes
// in flight per SM do not depend on how fast the consumers run.  Eight consumer warps share every
// stage (warp w takes the 64-byte steps w, w+8, ...) and feed mma.sync.m16n8k32 with the tokens as
// the 16-row operand and the unit's 8 channels as the 8-column operand; the reduction index may be
// permuted freely as long as both operands use the same permutation, so each thread simply takes 16
// contiguous bytes of its row.  An INT4 byte pair is never sign-extended arithmetically:
// (w << 4) & 0xF0F0F0F0 and w & 0xF0F0F0F0 are the even / odd codes times 16 as int8 lanes, the
// activations get the same treatment, and the INT4 accumulator therefore holds 256 x the true sum
// (|256 * 7 * 7 * (K - r)| < 2^31 for K - r < 171k), shifted back exactly in the epilogue.
// Per unit the eight warps' partial sums meet in shared memory and 128 threads apply the scales.
//
// Overlap with the preceding kernel.  The weights do not depend on it, so with the launch attribute
// for programmatic stream serialization the producer starts filling the ring at once while the
// consumers wait (griddepcontrol.wait) for the activations.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"
#include "ptx.cuh"

namespace resq {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + the producer warp
constexpr int kUnitRows = 8;
constexpr int kChunk = 2048;                 // bytes of one weight row per stage
constexpr int kRowPitch = kChunk + 64;       // = 64 mod 128: two rows' 64-byte pieces cover all banks
constexpr int kStageBytes = kUnitRows * kRowPitch;
constexpr int kMaxStages = 8;
constexpr int kMinStages = 3;
constexpr int kRedInts = kConsumerWarps * 256;  // per buffer: warp x {acc8[128], acc4[128]}
constexpr int kSmemLimit = 227 * 1024;

struct Params {
    int T, N, r, row4;     // row4 = (K - r) / 2: bytes of a packed INT4 weight row
    int c8, c4;            // chunks per row in the INT8 / INT4 segment
    int units;             // N / 8
    int pitch8, pitch4;    // bytes per token of the staged activations (zero padded)
    int nstages;
    int early_weights;     // the launch allows an early start: only the consumers wait for the upstream kernel
    const int8_t* x8;
    const uint8_t* x4;
    const float* s_x8;
    const float* s_x4;
    const uint8_t* w8;
    const uint8_t* w4;
    const void* s_w8;
    const void* s_w4;
    int w_fp16;
    void* Y;
    int y_dtype;
    int32_t* dbg8;
    int32_t* dbg4;
    int* status;
};

struct __align__(16) Control {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    float sx8[16];
    float sx4[16];
    int abort_flag;
};

__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void consumer_barrier() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float load_scale(const void* p, int i, int fp16) {
    return fp16 ? __half2float(reinterpret_cast<const __half*>(p)[i]) : reinterpret_cast<const float*>(p)[i];
}

constexpr uint32_t kHi = 0xF0F0F0F0u;

// TT = 1: T <= 8 (token rows 8..15 of the 16-row operand are zero and are not staged); TT = 2: T <= 16.
template <int TT>
__global__ void __launch_bounds__(kThreads, 1)
mixed_gemm_stream_kernel(const Params p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int TP = TT * 8;
    Control* ctl = reinterpret_cast<Control*>(smem);
    int* red = reinterpret_cast<int*>(smem + 512);                       // [2][kRedInts]
    uint8_t* act8 = smem + 512 + 2 * kRedInts * 4;                       // [TP][pitch8]
    uint8_t* act4 = act8 + static_cast<size_t>(TP) * p.pitch8;           // [TP][pitch4]
    uint8_t* ring = act4 + static_cast<size_t>(TP) * p.pitch4;           // [nstages][8][kRowPitch]
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int u0 = static_cast<int>(static_cast<long long>(p.units) * blockIdx.x / gridDim.x);
    const int u1 = static_cast<int>(static_cast<long long>(p.units) * (blockIdx.x + 1) / gridDim.x);
    const int nchunks = p.c8 + p.c4;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.nstages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kConsumerWarps);
        }
        ctl->abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    griddep_launch_dependents();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            if (!p.early_weights) griddep_wait();
            int stage = 0, issued = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u) {
                for (int c = 0; c < nchunks; ++c) {
                    const bool seg8 = c < p.c8;
                    const int rowbytes = seg8 ? p.r : p.row4;
                    const int off = (seg8 ? c : c - p.c8) * kChunk;
                    const int bytes = rowbytes - off < kChunk ? rowbytes - off : kChunk;
                    const uint8_t* src = (seg8 ? p.w8 : p.w4) + static_cast<size_t>(u) * kUnitRows * rowbytes + off;
                    if (!mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(&ctl->full[stage], static_cast<uint32_t>(kUnitRows * bytes));
                    uint8_t* dst = ring + static_cast<size_t>(stage) * kStageBytes;
#pragma unroll
                    for (int i = 0; i < kUnitRows; ++i)
                        bulk_load(dst + i * kRowPitch, src + static_cast<size_t>(i) * rowbytes, static_cast<uint32_t>(bytes),
                                  &ctl->full[stage]);
                    ++issued;
                    if (++stage == p.nstages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // Let the copies already in flight land before the CTA gives up its shared memory.
                int n = issued < p.nstages ? issued : p.nstages;
                for (int i = 0; i < n; ++i) {
                    if (stage == 0) { stage = p.nstages; phase ^= 1; }
                    --stage;
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(&ctl->full[stage], phase) && global_timer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int tid = threadIdx.x;
        const int g = lane >> 2, tig = lane & 3;
        griddep_wait();
        // Stage the activation codes (zero padded to the pitch, zero rows for tokens >= T).
        {
            const int v8 = p.pitch8 >> 4, v4 = p.pitch4 >> 4;  // 16-byte vectors per token
            for (int i = tid; i < TP * v8; i += kConsumerThreads) {
                const int t = i / v8, o = (i - t * v8) << 4;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (t < p.T && o < p.r) v = *reinterpret_cast<const uint4*>(p.x8 + static_cast<size_t>(t) * p.r + o);
                *reinterpret_cast<uint4*>(act8 + static_cast<size_t>(t) * p.pitch8 + o) = v;
            }
            for (int i = tid; i < TP * v4; i += kConsumerThreads) {
                const int t = i / v4, o = (i - t * v4) << 4;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (t < p.T && o < p.row4) v = *reinterpret_cast<const uint4*>(p.x4 + static_cast<size_t>(t) * p.row4 + o);
                *reinterpret_cast<uint4*>(act4 + static_cast<size_t>(t) * p.pitch4 + o) = v;
            }
            if (tid < 16) {
                ctl->sx8[tid] = tid < p.T ? p.s_x8[tid] : 0.f;
                ctl->sx4[tid] = tid < p.T ? p.s_x4[tid] : 0.f;
            }
        }
        consumer_barrier();

        int stage = 0, buf = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int u = u0; u < u1; ++u) {
            int acc8[4] = {0, 0, 0, 0}, acc4a[4] = {0, 0, 0, 0}, acc4b[4] = {0, 0, 0, 0};
            for (int c = 0; c < nchunks; ++c) {
                const bool seg8 = c < p.c8;
                const int rowbytes = seg8 ? p.r : p.row4;
                const int off = (seg8 ? c : c - p.c8) * kChunk;
                const int bytes = rowbytes - off < kChunk ? rowbytes - off : kChunk;
                const int nsteps = (bytes + 63) >> 6;
                if (ok && !mbar_wait(&ctl->full[stage], phase, abort_flag)) ok = false;
                if (ok) {
                    const uint8_t* wrow = ring + static_cast<size_t>(stage) * kStageBytes + g * kRowPitch + 16 * tig;
                    if (seg8) {
                        const uint8_t* xa = act8 + static_cast<size_t>(g) * p.pitch8 + off + 16 * tig;
                        for (int s = warp; s < nsteps; s += kConsumerWarps) {
                            const uint4 w = *reinterpret_cast<const uint4*>(wrow + 64 * s);
                            const uint4 x = *reinterpret_cast<const uint4*>(xa + 64 * s);
                            uint4 y = make_uint4(0, 0, 0, 0);
                            if (TT == 2) y = *reinterpret_cast<const uint4*>(xa + 8 * p.pitch8 + 64 * s);
                            mma_s8(acc8, x.x, y.x, x.y, y.y, w.x, w.y);
                            mma_s8(acc8, x.z, y.z, x.w, y.w, w.z, w.w);
                        }
                    } else {
                        const uint8_t* xa = act4 + static_cast<size_t>(g) * p.pitch4 + off + 16 * tig;
                        for (int s = warp; s < nsteps; s += kConsumerWarps) {
                            const uint4 w = *reinterpret_cast<const uint4*>(wrow + 64 * s);
                            const uint4 x = *reinterpret_cast<const uint4*>(xa + 64 * s);
                            uint4 y = make_uint4(0, 0, 0, 0);
                            if (TT == 2) y = *reinterpret_cast<const uint4*>(xa + 8 * p.pitch4 + 64 * s);
                            mma_s8(acc4a, (x.x << 4) & kHi, (y.x << 4) & kHi, x.x & kHi, y.x & kHi, (w.x << 4) & kHi, w.x & kHi);
                            mma_s8(acc4b, (x.y << 4) & kHi, (y.y << 4) & kHi, x.y & kHi, y.y & kHi, (w.y << 4) & kHi, w.y & kHi);
                            mma_s8(acc4a, (x.z << 4) & kHi, (y.z << 4) & kHi, x.z & kHi, y.z & kHi, (w.z << 4) & kHi, w.z & kHi);
                            mma_s8(acc4b, (x.w << 4) & kHi, (y.w << 4) & kHi, x.w & kHi, y.w & kHi, (w.w << 4) & kHi, w.w & kHi);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                }
                if (++stage == p.nstages) { stage = 0; phase ^= 1; }
            }
            // The eight warps' partial sums of this unit meet in shared memory.
            int* my = red + buf * kRedInts + warp * 256 + lane * 4;
            *reinterpret_cast<int4*>(my) = make_int4(acc8[0], acc8[1], acc8[2], acc8[3]);
            *reinterpret_cast<int4*>(my + 128) =
                make_int4(acc4a[0] + acc4b[0], acc4a[1] + acc4b[1], acc4a[2] + acc4b[2], acc4a[3] + acc4b[3]);
            consumer_barrier();
            if (tid < 128 && !*abort_flag) {
                // element e = lane * 4 + i of the accumulator fragment: token g + 8 * (i >> 1), channel 2 * tig + (i & 1)
                const int* src = red + buf * kRedInts + tid;
                int a8 = 0, a4 = 0;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    a8 += src[w * 256];
                    a4 += src[w * 256 + 128];
                }
                a4 >>= 8;  // exact: the sum is a multiple of 256
                const int el = tid >> 2, i = tid & 3;
                const int t = (el >> 2) + 8 * (i >> 1);
                const int n = u * kUnitRows + 2 * (el & 3) + (i & 1);
                if (t < p.T) {
                    const float t8 = static_cast<float>(a8) * (ctl->sx8[t] * load_scale(p.s_w8, n, p.w_fp16));
                    const float t4 = static_cast<float>(a4) * (ctl->sx4[t] * load_scale(p.s_w4, n, p.w_fp16));
                    const float y = t8 + t4;
                    const size_t o = static_cast<size_t>(t) * p.N + n;
                    if (p.y_dtype == RESQ_Y_BF16) reinterpret_cast<__nv_bfloat16*>(p.Y)[o] = __float2bfloat16_rn(y);
                    else reinterpret_cast<float*>(p.Y)[o] = y;
                    if (p.dbg8) {
                        p.dbg8[o] = a8;
                        p.dbg4[o] = a4;
                    }
                }
            }
            buf ^= 1;
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && ctl->abort_flag) atomicOr(p.status, RESQ_ERR_TIMEOUT);
}

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

}  // namespace

static int g_early_weights = 0;
void set_decode_early_weights(int on) { g_early_weights = on ? 1 : 0; }

// Returns cudaErrorNotSupported (nothing launched) when the staged activations leave no room for the ring.
cudaError_t launch_mixed_gemm_stream(int T, int N, int K, int r, const int8_t* x8, const uint8_t* x4,
                                     const float* s_x8, const float* s_x4, const int8_t* w8, const uint8_t* w4,
                                     const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                     int32_t* dbg8, int32_t* dbg4, cudaStream_t st) {
    Params p;
    p.T = T; p.N = N; p.r = r; p.row4 = (K - r) / 2;
    p.c8 = (r + kChunk - 1) / kChunk;
    p.c4 = (p.row4 + kChunk - 1) / kChunk;
    p.units = N / kUnitRows;
    p.pitch8 = round_up(r, 128) + 64;
    p.pitch4 = round_up(p.row4, 128) + 64;
    const int TP = T <= 8 ? 8 : 16;
    const size_t fixed = 512 + 2 * kRedInts * 4 + static_cast<size_t>(TP) * (p.pitch8 + p.pitch4);
    if (fixed + static_cast<size_t>(kMinStages) * kStageBytes > static_cast<size_t>(kSmemLimit)) return cudaErrorNotSupported;
    int nstages = static_cast<int>((kSmemLimit - fixed) / kStageBytes);
    if (nstages > kMaxStages) nstages = kMaxStages;
    p.nstages = nstages;
    p.early_weights = g_early_weights;
    p.x8 = x8; p.x4 = x4; p.s_x8 = s_x8; p.s_x4 = s_x4;
    p.w8 = reinterpret_cast<const uint8_t*>(w8); p.w4 = w4; p.s_w8 = s_w8; p.s_w4 = s_w4;
    p.w_fp16 = w_scale_fp16 ? 1 : 0;
    p.Y = Y; p.y_dtype = y_dtype; p.dbg8 = dbg8; p.dbg4 = dbg8 ? dbg4 : nullptr;
    p.status = device_status_ptr();
    const size_t smem = fixed + static_cast<size_t>(nstages) * kStageBytes;

    auto kern = T <= 8 ? mixed_gemm_stream_kernel<1> : mixed_gemm_stream_kernel<2>;
    static bool attr_set[2][64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[T <= 8][dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set[T <= 8][dev] = true;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.units < sms ? p.units : sms, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.early_weights ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace resq
