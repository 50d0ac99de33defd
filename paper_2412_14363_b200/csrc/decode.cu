// Few-token (T <= 16) mixed-precision GEMM: memory-bound, streams the packed weights once at HBM rate.
//
// Layout of the work
//   grid = (ceil(N / 64), ksplit); the ksplit CTAs of one 64-channel block form a thread-block
//   cluster and split the reduction dimension; their int32 partial sums meet in the leader CTA's
//   shared memory (distributed shared memory), so there are no global atomics, no scratch buffer and
//   the result is bit-exact whatever the split.
//   A CTA has 8 warps = 4 row groups of 16 channels x 2 interleaved K halves.
// Data path
//   Weights go global -> registers directly, 16 bytes per thread and row, already in the operand
//   order of mma.sync.m16n8k32 (weights are the 16-row A operand, tokens the 8-column B operand);
//   the reduction index may be permuted freely as long as both operands use the same permutation.
//   An INT4 byte pair is never sign-extended arithmetically: (w << 4) & 0xF0F0F0F0 and
//   w & 0xF0F0F0F0 are the even / odd codes times 16 as int8 lanes.  The activations get the same
//   treatment when they are staged in shared memory, so the INT4 accumulator holds 256 x the true sum
//   (|256 * 7 * 7 * (K - r)| < 2^31 for K - r < 171k) and is shifted back exactly in the epilogue.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"

namespace resq {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 64;
constexpr int kTokStride = 144;  // bytes per token per step in shared memory (128 + 16 pad: conflict-free LDS.128)
constexpr int kUnroll = 4;       // steps whose weight loads are in flight per thread

struct Params {
    int T, N, r, K4;
    int S8, S4;          // 64-byte steps of a weight row in the INT8 / INT4 segment
    int steps_per_cta;
    const int8_t* x8;
    const uint8_t* x4;
    const float* s_x8;
    const float* s_x4;
    const int8_t* w8;
    const uint8_t* w4;
    const void* s_w8;
    const void* s_w4;
    int w_fp16;
    void* Y;
    int y_dtype;
    int32_t* dbg8;
    int32_t* dbg4;
};

__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t local_smem_addr, uint32_t rank, int4 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(rank));
    asm volatile("st.shared::cluster.v4.s32 [%0], {%1,%2,%3,%4};" ::"r"(remote), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

__device__ __forceinline__ float load_scale(const void* p, int i, int fp16) {
    return fp16 ? __half2float(reinterpret_cast<const __half*>(p)[i]) : reinterpret_cast<const float*>(p)[i];
}

// TT = number of 8-token column tiles (1: T <= 8, 2: T <= 16).
template <int TT>
__global__ void __launch_bounds__(kThreads)
mixed_gemm_decode_kernel(const Params p) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TP = TT * 8;  // padded token count
    const int ksplit = gridDim.y;
    const int crank = ksplit > 1 ? static_cast<int>(cluster_ctarank()) : 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int rg = warp & 3, kh = warp >> 2;
    const int n0 = blockIdx.x * kRowsPerCta + rg * 16;

    const int S = p.S8 + p.S4;
    const int s_begin = crank * p.steps_per_cta;
    const int s_end = min(S, s_begin + p.steps_per_cta);

    uint8_t* xs = smem;                                                   // [steps_per_cta][TP][kTokStride]
    int* red = reinterpret_cast<int*>(smem + static_cast<size_t>(p.steps_per_cta) * TP * kTokStride);  // [4][32][16]
    int* slots = red + 4 * 32 * 16;                                       // [ksplit-1][4][32][16] (leader only)

    // Weight rows of this thread (clamped: out-of-range rows are computed on row N-1 and never stored).
    const int rowA = min(n0 + g, p.N - 1), rowB = min(n0 + g + 8, p.N - 1);
    const uint8_t* w8a = reinterpret_cast<const uint8_t*>(p.w8) + static_cast<size_t>(rowA) * p.r + 16 * tig;
    const uint8_t* w8b = reinterpret_cast<const uint8_t*>(p.w8) + static_cast<size_t>(rowB) * p.r + 16 * tig;
    const int row4 = p.K4 >> 1;
    const uint8_t* w4a = p.w4 + static_cast<size_t>(rowA) * row4 + 16 * tig;
    const uint8_t* w4b = p.w4 + static_cast<size_t>(rowB) * row4 + 16 * tig;

    auto load_step = [&](int s, uint4& a, uint4& b) {
        a = make_uint4(0, 0, 0, 0);
        b = a;
        if (s >= s_end) return;
        if (s < p.S8) {
            if (64 * s + 16 * tig < p.r) {
                a = ldg_stream(w8a + 64 * s);
                b = ldg_stream(w8b + 64 * s);
            }
        } else {
            const int o = 64 * (s - p.S8);
            if (o + 16 * tig < row4) {
                a = ldg_stream(w4a + o);
                b = ldg_stream(w4b + o);
            }
        }
    };

    // First batch of weight loads goes out before the activations are staged.
    const int s_first = s_begin + kh;
    uint4 wa[kUnroll], wb[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) load_step(s_first + 2 * u, wa[u], wb[u]);

    // ---- stage this CTA's slice of the activations: 16 source bytes per thread and iteration
    {
        const int nsteps = s_end - s_begin;
        const int items = nsteps * TP * 4;  // (step, token, quarter of the step's 64 source bytes)
        for (int it = threadIdx.x; it < items; it += kThreads) {
            const int q = it & 3, t = (it >> 2) % TP, ls = (it >> 2) / TP;
            const int s = s_begin + ls;
            uint8_t* dst = xs + (static_cast<size_t>(ls) * TP + t) * kTokStride;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (s < p.S8) {
                const int off = 64 * s + 16 * q;
                if (t < p.T && off < p.r) v = *reinterpret_cast<const uint4*>(p.x8 + static_cast<size_t>(t) * p.r + off);
                *reinterpret_cast<uint4*>(dst + 16 * q) = v;
            } else {
                const int off = 64 * (s - p.S8) + 16 * q;
                if (t < p.T && off < row4) v = *reinterpret_cast<const uint4*>(p.x4 + static_cast<size_t>(t) * row4 + off);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    o[2 * i] = (w[i] << 4) & 0xF0F0F0F0u;   // even codes x 16
                    o[2 * i + 1] = w[i] & 0xF0F0F0F0u;      // odd codes x 16
                }
                *reinterpret_cast<uint4*>(dst + 32 * q) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(dst + 32 * q + 16) = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
    }
    __syncthreads();

    int acc8[TT][4], acc4[TT][4];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc8[tt][i] = acc4[tt][i] = 0;

    for (int sb = s_first; sb < s_end; sb += 2 * kUnroll) {
        uint4 na[kUnroll], nb[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) load_step(sb + 2 * kUnroll + 2 * u, na[u], nb[u]);  // next batch
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int s = sb + 2 * u;
            if (s < s_end) {
                const uint8_t* xrow = xs + static_cast<size_t>(s - s_begin) * TP * kTokStride + g * kTokStride;
                const uint32_t qa[4] = {wa[u].x, wa[u].y, wa[u].z, wa[u].w};
                const uint32_t qb[4] = {wb[u].x, wb[u].y, wb[u].z, wb[u].w};
                if (s < p.S8) {
#pragma unroll
                    for (int tt = 0; tt < TT; ++tt) {
                        const uint4 xb = *reinterpret_cast<const uint4*>(xrow + tt * 8 * kTokStride + 16 * tig);
                        const uint32_t a0[4] = {qa[0], qb[0], qa[1], qb[1]};
                        const uint32_t a1[4] = {qa[2], qb[2], qa[3], qb[3]};
                        mma_s8(acc8[tt], a0, xb.x, xb.y);
                        mma_s8(acc8[tt], a1, xb.z, xb.w);
                    }
                } else {
#pragma unroll
                    for (int tt = 0; tt < TT; ++tt) {
                        const uint4 x0 = *reinterpret_cast<const uint4*>(xrow + tt * 8 * kTokStride + 32 * tig);
                        const uint4 x1 = *reinterpret_cast<const uint4*>(xrow + tt * 8 * kTokStride + 32 * tig + 16);
                        const uint32_t xl[4] = {x0.x, x0.z, x1.x, x1.z};
                        const uint32_t xh[4] = {x0.y, x0.w, x1.y, x1.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t a[4] = {(qa[j] << 4) & 0xF0F0F0F0u, (qb[j] << 4) & 0xF0F0F0F0u,
                                                   qa[j] & 0xF0F0F0F0u, qb[j] & 0xF0F0F0F0u};
                            mma_s8(acc4[tt], a, xl[j], xh[j]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            wa[u] = na[u];
            wb[u] = nb[u];
        }
    }

    // ---- reduce the two K halves inside the CTA
    int* my = red + (rg * 32 + lane) * 16;
    if (kh == 1) {
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) {
            *reinterpret_cast<int4*>(my + tt * 8) = make_int4(acc8[tt][0], acc8[tt][1], acc8[tt][2], acc8[tt][3]);
            *reinterpret_cast<int4*>(my + tt * 8 + 4) = make_int4(acc4[tt][0], acc4[tt][1], acc4[tt][2], acc4[tt][3]);
        }
    }
    __syncthreads();
    if (kh == 0) {
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) {
            const int4 a = *reinterpret_cast<const int4*>(my + tt * 8), b = *reinterpret_cast<const int4*>(my + tt * 8 + 4);
            acc8[tt][0] += a.x; acc8[tt][1] += a.y; acc8[tt][2] += a.z; acc8[tt][3] += a.w;
            acc4[tt][0] += b.x; acc4[tt][1] += b.y; acc4[tt][2] += b.z; acc4[tt][3] += b.w;
        }
    }

    // ---- reduce across the cluster: every non-leader CTA writes into its slot of the leader's shared memory
    if (ksplit > 1) {
        if (crank != 0 && kh == 0) {
            const uint32_t base = static_cast<uint32_t>(__cvta_generic_to_shared(slots)) +
                                  static_cast<uint32_t>((((crank - 1) * 4 + rg) * 32 + lane) * 16 * 4);
#pragma unroll
            for (int tt = 0; tt < TT; ++tt) {
                st_cluster_v4(base + tt * 32, 0, make_int4(acc8[tt][0], acc8[tt][1], acc8[tt][2], acc8[tt][3]));
                st_cluster_v4(base + tt * 32 + 16, 0, make_int4(acc4[tt][0], acc4[tt][1], acc4[tt][2], acc4[tt][3]));
            }
        }
        cluster_sync_all();
        if (crank != 0) return;
        if (kh == 0) {
            for (int c = 0; c < ksplit - 1; ++c) {
                const int* sl = slots + ((c * 4 + rg) * 32 + lane) * 16;
#pragma unroll
                for (int tt = 0; tt < TT; ++tt) {
                    const int4 a = *reinterpret_cast<const int4*>(sl + tt * 8), b = *reinterpret_cast<const int4*>(sl + tt * 8 + 4);
                    acc8[tt][0] += a.x; acc8[tt][1] += a.y; acc8[tt][2] += a.z; acc8[tt][3] += a.w;
                    acc4[tt][0] += b.x; acc4[tt][1] += b.y; acc4[tt][2] += b.z; acc4[tt][3] += b.w;
                }
            }
        }
    }
    if (kh != 0) return;

    // ---- epilogue: fragment element i of tile tt is (channel n0 + g + 8*(i>>1), token tt*8 + 2*tig + (i&1))
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int n = n0 + g + 8 * (i >> 1), t = tt * 8 + 2 * tig + (i & 1);
            if (n < p.N && t < p.T) {
                const int a8 = acc8[tt][i], a4 = acc4[tt][i] >> 8;  // exact: acc4 is a multiple of 256
                const float t8 = static_cast<float>(a8) * (p.s_x8[t] * load_scale(p.s_w8, n, p.w_fp16));
                const float t4 = static_cast<float>(a4) * (p.s_x4[t] * load_scale(p.s_w4, n, p.w_fp16));
                const float y = t8 + t4;
                const size_t off = static_cast<size_t>(t) * p.N + n;
                if (p.y_dtype == RESQ_Y_BF16) reinterpret_cast<__nv_bfloat16*>(p.Y)[off] = __float2bfloat16_rn(y);
                else reinterpret_cast<float*>(p.Y)[off] = y;
                if (p.dbg8) {
                    p.dbg8[off] = a8;
                    p.dbg4[off] = a4;
                }
            }
        }
    }
}

}  // namespace

size_t decode_scratch_bytes(int, int) { return 0; }  // partial sums meet in distributed shared memory

cudaError_t launch_mixed_gemm_decode(int T, int N, int K, int r, const int8_t* x8, const uint8_t* x4,
                                     const float* s_x8, const float* s_x4, const int8_t* w8, const uint8_t* w4,
                                     const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                     int32_t* dbg8, int32_t* dbg4, void* /*scratch*/, cudaStream_t st) {
    Params p;
    p.T = T; p.N = N; p.r = r; p.K4 = K - r;
    p.S8 = (r + 63) / 64;
    p.S4 = (p.K4 / 2 + 63) / 64;
    p.x8 = x8; p.x4 = x4; p.s_x8 = s_x8; p.s_x4 = s_x4; p.w8 = w8; p.w4 = w4; p.s_w8 = s_w8; p.s_w4 = s_w4;
    p.w_fp16 = w_scale_fp16 ? 1 : 0;
    p.Y = Y; p.y_dtype = y_dtype; p.dbg8 = dbg8; p.dbg4 = dbg8 ? dbg4 : nullptr;
    const int S = p.S8 + p.S4;
    const int n_blocks = (N + kRowsPerCta - 1) / kRowsPerCta;
    const int TP = T <= 8 ? 8 : 16;
    // Split K over a cluster until about two CTAs per SM are in flight, keeping >= 4 steps per CTA
    // and the staged activations within shared memory.
    int ksplit = 1;
    while (ksplit < 8 && n_blocks * ksplit < 2 * 148 && S / (ksplit * 2) >= 4) ksplit *= 2;
    auto smem_for = [&](int ks) {
        const int spc = (S + ks - 1) / ks;
        return static_cast<size_t>(spc) * TP * kTokStride + 4 * 32 * 16 * 4 + static_cast<size_t>(ks - 1) * 4 * 32 * 16 * 4;
    };
    while (ksplit < 8 && smem_for(ksplit) > 200 * 1024) ksplit *= 2;
    if (smem_for(ksplit) > 227 * 1024) return cudaErrorInvalidConfiguration;
    p.steps_per_cta = (S + ksplit - 1) / ksplit;
    const size_t smem = smem_for(ksplit);

    auto kern = T <= 8 ? mixed_gemm_decode_kernel<1> : mixed_gemm_decode_kernel<2>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_blocks, ksplit, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = ksplit;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace resq
