/*
 * resq.h -- C ABI of the ResQ mixed-precision linear layer for NVIDIA B200 (sm_100a).
 *
 * The layer (paper, Section 4.1): activations are expressed in an orthogonal basis U = P·R
 * (Eq. 5); the first r coefficients of every token are quantized to symmetric per-token INT8,
 * the remaining K - r to symmetric per-token INT4 (Eq. 1, Eq. 2); the weights, projected offline
 * by U^T, are quantized the same way per output channel (Eq. 3); the output is the sum of the
 * two same-precision integer products, each rescaled by its token scale and channel scale (Eq. 4):
 *
 *     Y[t][n] = s_x8[t]·s_w8[n]·sum_{j<r}  x8[t][j]·w8[n][j]
 *             + s_x4[t]·s_w4[n]·sum_{j<K-r} x4[t][j]·w4[n][j]
 *
 * Conventions shared by every entry point
 *  - All data pointers are DEVICE pointers to caller-owned memory unless a parameter says "host".
 *    The library allocates no device memory, keeps no reference to any buffer after the call
 *    returns, and never synchronizes the stream: work is enqueued on `stream` (a cudaStream_t
 *    passed as void*, NULL = default stream).
 *  - Descriptor structs are read on the host during the call.
 *  - Matrices are row-major with the K (reduction) dimension contiguous.  The high-precision
 *    coefficients come first in a row: columns [0, r) are the INT8 segment, [r, K) the INT4 one.
 *  - INT4 packing: byte i of a row holds code 2i in bits 0..3 and code 2i+1 in bits 4..7, two's
 *    complement.  Codes produced here lie in [-127,127] and [-7,7]; consumers accept the full
 *    [-128,127] and [-8,7].
 *  - Quantizer arithmetic (fixed so that results are reproducible bit for bit): absmax a over the
 *    segment; s = a / qmax as an IEEE fp32 division (qmax = 127 or 7); if the scale is stored as
 *    fp16 it is rounded to fp16 first and the rounded value is the one used; code =
 *    clamp(round-half-even(x / s)) with an IEEE fp32 division; a == 0 gives s = 0 and codes 0.
 *  - Shape rules: r % 32 == 0, (K - r) % 32 == 0, 0 <= r < K (r = 0: uniform INT4), n_out % 8 == 0, T >= 1.
 *    Data pointers must be 16-byte aligned.
 *  - Every function returns a resq_status_t (0 = success).  Arguments are validated on the host
 *    before the first launch: RESQ_ERR_NULL / _SHAPE / _ALIGN / _WORKSPACE / _ARCH mean that nothing was
 *    enqueued.  RESQ_ERR_CUDA can also come from a later launch of a call that enqueues several kernels.  Waits inside the
 *    kernels are bounded; a wait that runs out sets a device status word (see resq_device_status)
 *    and the kernel drains and returns.
 *  - Inputs must be finite; NaN/Inf are not checked.
 */
#ifndef RESQ_H_
#define RESQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum resq_status {
    RESQ_OK = 0,
    RESQ_ERR_NULL = 1,       /* a required pointer is NULL */
    RESQ_ERR_SHAPE = 2,      /* a shape rule above is violated */
    RESQ_ERR_ALIGN = 3,      /* a pointer is not 16-byte aligned */
    RESQ_ERR_WORKSPACE = 4,  /* workspace missing or smaller than resq_workspace_bytes() */
    RESQ_ERR_ARCH = 5,       /* current device is not compute capability 10.x */
    RESQ_ERR_CUDA = 6,       /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
    RESQ_ERR_TIMEOUT = 7,    /* reported by resq_device_status: a bounded device wait ran out */
    RESQ_ERR_INDEX = 8       /* reported by resq_device_status: an index read on the device (cache slot, sequence
                                length) was out of range; the element was skipped or clamped (resq_kv.h) */
} resq_status_t;

/* Weight-scale storage type. */
enum { RESQ_SCALE_FP32 = 0, RESQ_SCALE_FP16 = 1 };
/* Output type of Y. */
enum { RESQ_Y_BF16 = 0, RESQ_Y_FP32 = 1 };

/* One linear layer: K input features (coefficients), n_out output channels, r high-precision
 * coefficients (the paper uses r = K/8, Section 4.1). */
typedef struct resq_layer_desc {
    int32_t K;
    int32_t n_out;
    int32_t r;
    int32_t w_scale_dtype; /* RESQ_SCALE_FP32 or RESQ_SCALE_FP16 */
} resq_layer_desc_t;

/* Quantized weights of one layer, as written by resq_pack_weights (Eq. 3). */
typedef struct resq_weights {
    const int8_t* w8;    /* [n_out][r]        INT8 codes                                   */
    const uint8_t* w4;   /* [n_out][(K-r)/2]  INT4 codes, packed                            */
    const void* s_w8;    /* [n_out]           fp32 or fp16 per w_scale_dtype                */
    const void* s_w4;    /* [n_out]                                                          */
    const int8_t* w4_i8; /* [n_out][K-r] optional: the INT4 codes one per byte (sign-extended),
                            a layout for the compute-bound many-token kernel; NULL = absent, the
                            kernel then expands `w4` itself into the workspace */
} resq_weights_t;

/* Byte sizes of the packed buffers of a layer. */
size_t resq_w8_bytes(const resq_layer_desc_t* desc);    /* n_out * r          */
size_t resq_w4_bytes(const resq_layer_desc_t* desc);    /* n_out * (K-r) / 2  */
size_t resq_w4_i8_bytes(const resq_layer_desc_t* desc); /* n_out * (K-r)      */
size_t resq_scale_bytes(const resq_layer_desc_t* desc); /* n_out * 4 or * 2   */

/* Scratch bytes that resq_project_quantize / resq_mixed_gemm / resq_linear need for T tokens.
 * has_P != 0: the online projection is used.  has_w4_i8 != 0: weights carry the w4_i8 layout.
 * Returns 0 on an invalid descriptor. */
size_t resq_workspace_bytes(const resq_layer_desc_t* desc, int T, int has_P, int has_w4_i8);

/*
 * Eq. 3: quantize projected weights.  W_proj is (U^T W)^T as fp32 [n_out][K]; each output channel is
 * split at r and quantized per segment (round to nearest; the paper's experiments use GPTQ instead,
 * which is out of scope).  Outputs w8, w4, s_w8, s_w4 as in resq_weights_t; w4_i8 may be NULL.
 */
int resq_pack_weights(const resq_layer_desc_t* desc, const float* W_proj, int8_t* w8, uint8_t* w4,
                      void* s_w8, void* s_w4, int8_t* w4_i8, void* stream);

/*
 * Eq. 3 with the rounding of the paper's experiments (Section 5.1: "apply GPTQ for weight quantization"; Frantar et
 * al., 2022) instead of round-to-nearest.  W_proj as for resq_pack_weights.  U_inv: fp32 [K][K], the upper triangular
 * Cholesky factor of the inverse of the layer's damped input Hessian H = (2/n) X^T X + 0.01 mean(diag) I, X being
 * calibration inputs of the layer in the projected basis (H^-1 = U_inv^T U_inv; the factorisation is the caller's:
 * any LAPACK, offline).  dead_cols: optional bytes [K], non-zero where H had a zero diagonal entry (an input that was
 * never active): those weights are set to 0.  Per output channel: the scales are those of resq_pack_weights on the
 * rows as given; columns are visited in order, column j is rounded to code_j = clamp(round-half-even(w_j / s)), and
 * (w_j - code_j s) / U_inv[j][j] times U_inv[j][j+1:] is subtracted from the columns not yet visited.  All of it in
 * fp64, one rounding per operation in this order, so the codes are reproducible bit for bit.  An offline step: the
 * sweep is a chain of K dependent steps per row.  K * 9 bytes (a row in shared memory) must not exceed 200 KB, else
 * RESQ_ERR_SHAPE.  Outputs as resq_pack_weights.
 */
int resq_pack_weights_gptq(const resq_layer_desc_t* desc, const float* W_proj, const float* U_inv,
                           const uint8_t* dead_cols, int8_t* w8, uint8_t* w4, void* s_w8, void* s_w4, int8_t* w4_i8,
                           void* stream);

/*
 * Eq. 3 with the projection done here (Section 4.3: the bases are multiplied into the weights offline): W_raw is
 * the unprojected weight as bf16 [n_out][K] (row n = the K input weights of output channel n), U the basis as
 * bf16 [K][K] (row i = input feature, column j = coefficient, as P of resq_project_quantize).  Forms
 * W_proj = W_raw·U = (U^T W)^T in fp32 on the tensor cores (bf16 products, fp32 accumulation), in panels of
 * rows staged in the workspace, and quantizes it like resq_pack_weights (round to nearest; GPTQ is not built).
 * Codes can differ by one step from those of an fp64 projection on a small fraction of elements, like the
 * online activation path.  Workspace: resq_pack_projected_workspace_bytes(desc) bytes.
 */
size_t resq_pack_projected_workspace_bytes(const resq_layer_desc_t* desc);
int resq_pack_weights_projected(const resq_layer_desc_t* desc, const void* W_raw, const void* U, int8_t* w8,
                                uint8_t* w4, void* s_w8, void* s_w4, int8_t* w4_i8, void* workspace,
                                size_t workspace_bytes, void* stream);

/*
 * Eq. 2: per-token split quantization of the coefficients.
 *   P == NULL: the rows of X (bf16 [T][K]) already are the coefficients -- the projection was
 *              folded into the preceding layer's weights (Section 4.3, U_A/U_B).
 *   P != NULL: bf16 [K][K], row i = input feature, column j = coefficient; C = X·P is formed online
 *              on the tensor cores with fp32 accumulation (Section 4.3, U_D for the down_proj input)
 *              and quantized from fp32 without an intermediate bf16 rounding.  Needs workspace
 *              (the fp32 panel; what resq_workspace_bytes adds beyond it is the projection GEMM's
 *              scratch, see resq_project -- a workspace that only holds the panel is accepted too).
 * Outputs: x8 int8 [T][r]; x4 packed uint8 [T][(K-r)/2]; s_x8, s_x4 fp32 [T].
 * x4_i8 (optional, may be NULL): the INT4 codes one per byte, int8 [T][K-r].
 */
int resq_project_quantize(const void* X, const void* P, int T, int K, int r, int8_t* x8, uint8_t* x4,
                          float* s_x8, float* s_x4, int8_t* x4_i8, void* workspace,
                          size_t workspace_bytes, void* stream);

/*
 * The paper's own down_proj input path (Section 4.3): U_D is a Hadamard matrix, so the projection that cannot
 * be folded is a fast transform, and the down_proj weights and activations are quantized uniformly to 4 bits
 * (r = 0; a mixed split r > 0 is accepted as well).  C = X·H_K / sqrt(K) is formed in fp32 per token in shared
 * memory and quantized at once (Eq. 1, Eq. 2) without ever being written out.  H_K = Sylvester(2^k) (x) H_m with
 * coefficient index a·m + b; m = 1, or m = 12 / 28 by Paley's second construction (q = 5 / 13) -- the paper
 * names no construction; K = 8192, 14336 and 28672 are covered.  Other K, or K·4 bytes > 200 KB, give
 * RESQ_ERR_SHAPE.  Outputs as resq_project_quantize (x8 may be NULL when r = 0).  The weights to pair with it are
 * resq_pack_weights of (H_K^T W / sqrt(K))^T.  Every entry point accepts r = 0 (then w8 / x8 may be NULL).
 * The first call on each device sets kernel attributes: make it outside any stream capture.
 */
int resq_hadamard_quantize(const void* X, int T, int K, int r, int8_t* x8, uint8_t* x4, float* s_x8, float* s_x4,
                           int8_t* x4_i8, void* stream);

/*
 * The online projection alone (Section 4.3, U_D): C = X·P with X bf16 [T][K], P bf16 [K][K] (row i =
 * input feature, column j = coefficient), C fp32 [T][K], bf16 products accumulated in fp32 on the
 * tensor cores.  This is the first half of resq_project_quantize with P != NULL, exposed so that the
 * coefficients can be inspected and the GEMM timed on its own.  K % 8 == 0.
 * workspace (optional, may be NULL): resq_project_workspace_bytes() bytes of scratch.  With it, when the
 * last round of 256 x 256 output tiles would occupy less than half of the GPU, those tiles are cut along K
 * into partial tiles that a second kernel adds up in a fixed order (deterministic; the fp32 sums are then
 * formed in that order instead of one run over K).  resq_workspace_bytes() with has_P includes this scratch.
 */
size_t resq_project_workspace_bytes(void);
int resq_project(const void* X, const void* P, int T, int K, float* C, void* workspace, size_t workspace_bytes,
                 void* stream);

/*
 * Eq. 4 with the dequantizing epilogue: Y = diag(s_x8)(x8·w8^T)diag(s_w8) + diag(s_x4)(x4·w4^T)diag(s_w4).
 * Integer products accumulate exactly in int32; the epilogue is fp32:
 *     y = (float)acc8 * (s_x8[t] * s_w8[n]) + (float)acc4 * (s_x4[t] * s_w4[n])
 * rounded to bf16 (nearest even) when y_dtype == RESQ_Y_BF16.  Y is [T][n_out].
 * T <= 16 runs a weight-streaming kernel (exact integer sums whatever its work split), larger T the
 * tensor-core tile kernel.
 * The INT4 activation codes come packed (x4, uint8 [T][(K-r)/2]) and/or one per byte (x4_i8, int8
 * [T][K-r], as resq_project_quantize can emit them).  The streaming kernel reads x4, so x4 is
 * required when T <= 16; the tile kernel reads x4_i8 and, if only x4 is given, first expands it
 * into the workspace.  At least one of the two must be non-NULL.
 * dbg_acc8 / dbg_acc4: optional int32 [T][n_out] dumps of the two accumulators (NULL = off).
 */
int resq_mixed_gemm(const resq_layer_desc_t* desc, int T, const int8_t* x8, const uint8_t* x4,
                    const int8_t* x4_i8, const float* s_x8, const float* s_x4, const resq_weights_t* W,
                    void* Y, int y_dtype,
                    int32_t* dbg_acc8, int32_t* dbg_acc4, void* workspace, size_t workspace_bytes,
                    void* stream);

/*
 * The whole layer: resq_project_quantize followed by resq_mixed_gemm, with the quantized
 * activations held in the workspace.  X bf16 [T][K]; P bf16 [K][K] or NULL; Y [T][n_out].
 */
int resq_linear(const resq_layer_desc_t* desc, int T, const void* X, const void* P,
                const resq_weights_t* W, void* Y, int y_dtype, void* workspace, size_t workspace_bytes,
                void* stream);

/*
 * ---- Asymmetric per-token activations (Eq. 1, second form; the activation setting of the paper's
 * experiments, Section 5.1), symmetric per-channel weights as before. ----
 * Per token and segment: z = min, s = (max - min) / (2^N - 1), code = round-half-even((x - z) / s) in
 * [0, 2^N - 1] (fp32 subtraction and divisions in this order; a constant segment gives s = 0, codes 0),
 * dequantized value code * s + z.  Expanding Eq. 4 with these activations gives, per segment, the integer
 * product of the unsigned codes with the weight codes plus a rank-one term:
 *     Y[t][n] = s_x8[t]*s_w8[n]*sum_j u8[t][j]*w8[n][j] + z_x8[t]*s_w8[n]*wsum8[n]
 *             + s_x4[t]*s_w4[n]*sum_j u4[t][j]*w4[n][j] + z_x4[t]*s_w4[n]*wsum4[n],
 * wsum8[n] = sum_j w8[n][j] and wsum4[n] = sum_j w4[n][j] being the integer row sums of the weight codes
 * (computed once per layer by resq_weight_row_sums).  The products run as u8 x s8: on the weight-streaming
 * kernel for T <= 16 when the packed codes u4 are given, on the tensor-core tile kernel otherwise.  Unsigned INT4 codes pack like the signed ones (code 2i in the low nibble).
 * The epilogue is fp32: (float)acc*(s_x*s_w) per segment plus z_x*((float)wsum*s_w) per segment.
 * K * 4 bytes (a staged fp32 row) must not exceed 200 KB, else RESQ_ERR_SHAPE.
 */
int resq_weight_row_sums(const resq_layer_desc_t* desc, const resq_weights_t* W, int32_t* wsum8, int32_t* wsum4,
                         void* stream);
/* As resq_project_quantize; u8 uint8 [T][r], u4 packed uint8 [T][(K-r)/2] and/or u4_u8 uint8 [T][K-r] (one code
 * per byte), scales s_x8/s_x4 and zero-points z_x8/z_x4 fp32 [T]. */
int resq_project_quantize_asym(const void* X, const void* P, int T, int K, int r, uint8_t* u8, uint8_t* u4,
                               float* s_x8, float* s_x4, float* z_x8, float* z_x4, uint8_t* u4_u8, void* workspace,
                               size_t workspace_bytes, void* stream);
/* As resq_mixed_gemm, with unsigned activation codes, zero-points and the weight row sums. */
int resq_mixed_gemm_asym(const resq_layer_desc_t* desc, int T, const uint8_t* u8, const uint8_t* u4,
                         const uint8_t* u4_u8, const float* s_x8, const float* s_x4, const float* z_x8,
                         const float* z_x4, const resq_weights_t* W, const int32_t* wsum8, const int32_t* wsum4,
                         void* Y, int y_dtype, int32_t* dbg_acc8, int32_t* dbg_acc4, void* workspace,
                         size_t workspace_bytes, void* stream);
/* As resq_linear. */
int resq_linear_asym(const resq_layer_desc_t* desc, int T, const void* X, const void* P, const resq_weights_t* W,
                     const int32_t* wsum8, const int32_t* wsum4, void* Y, int y_dtype, void* workspace,
                     size_t workspace_bytes, void* stream);
/* Scratch bytes the three calls above need (0 on an invalid descriptor). */
size_t resq_workspace_bytes_asym(const resq_layer_desc_t* desc, int T, int has_P, int has_w4_i8);

/*
 * (No counterpart in the paper: a deployment aid.)  resq_project_quantize with P != NULL for callers that
 * cannot allocate device memory at all -- a server whose start-up code gave the whole GPU to its own pool, a
 * plug-in living inside another program's memory plan, a real-time loop that cannot afford cudaMalloc's
 * device-wide synchronisation.  The fp32 staging panel that the regular call takes from the caller's workspace
 * is instead a fixed array of RESQ_STATIC_SCRATCH_BYTES built into the library (each GPU that loads the library
 * holds it until the process exits).  The call allocates nothing, frees nothing and takes no workspace argument;
 * inputs and outputs are still the caller's buffers, with the meanings and layouts of resq_project_quantize
 * (r = 0 and a NULL x8 included).
 *  - Result: the same kernels as the regular call, run without the projection GEMM's split scratch.  The
 *    output is therefore identical, bit for bit, to resq_project_quantize given a workspace that holds only
 *    the panel (T * K * 4 bytes, rounded up to 256).  Against the regular call with the full
 *    resq_workspace_bytes() workspace it is identical wherever that call does not cut tiles along K; where
 *    it does -- every call with T <= 64, and larger T whose last round of tiles is thin -- the fp32 sums are
 *    formed in another order, and codes can differ by one step on a small fraction of elements (both stay
 *    within the online path's tolerance against exact sums).  Without the split a T <= 64 call also keeps
 *    only K/256 of the 74 SM pairs busy: at K = 14336 it is about a third slower than the regular call.
 *  - Limit: T * K * 4 bytes must not exceed RESQ_STATIC_SCRATCH_BYTES (K = 4096: T <= 512; K = 14336:
 *    T <= 146; K = 28672: T <= 73); beyond it the call returns RESQ_ERR_WORKSPACE and launches nothing.
 *    P must be non-NULL (without a projection no scratch is needed: use resq_project_quantize).
 *  - The first call on each device looks up the array's device address (and sets a kernel
 *    attribute); make that first call outside any stream capture, with that device current.
 *  - All calls on a device share the one array, and it keeps whatever the previous call wrote.  Nothing
 *    in it needs clearing (each call overwrites every element it later reads), but two calls that
 *    overlap on the GPU -- different streams, no ordering between them -- race on it: order them.
 */
#define RESQ_STATIC_SCRATCH_BYTES (8u << 20)
int resq_project_quantize_static(const void* X, const void* P, int T, int K, int r, int8_t* x8, uint8_t* x4,
                                 float* s_x8, float* s_x4, int8_t* x4_i8, void* stream);

/*
 * Process-wide options (host state of the library; not thread-safe against concurrent calls).
 *  RESQ_OPT_DECODE_EARLY_WEIGHTS (default 0): when 1, the few-token kernel (T <= 16) is launched so
 *    that it may begin while the preceding kernel of the stream is still running; it then streams its
 *    packed weights into shared memory at once and only waits for that kernel before it reads the
 *    activation codes and scales.  Generation is memory-bound (paper, Introduction), and this hides
 *    the ramp of each short kernel behind the tail of the previous one.  The caller promises that the
 *    packed weights and their scales were complete before the preceding kernel was enqueued (true
 *    for weights packed at load time; false if resq_pack_weights is the preceding kernel).
 *  RESQ_OPT_WAIT_LIMIT_US (default 2 000 000): wall-clock limit, in microseconds, of a single wait inside a
 *    kernel (for a copy to land, for a pipeline stage to be released).  Stored on the CURRENT device with a
 *    blocking copy; kernels enqueued afterwards on that device use it.  value >= 1; the kernels look at the
 *    limit only once a wait has lasted 100 us, so smaller values act as 100.
 * Returns RESQ_ERR_SHAPE for an unknown option or value.
 */
enum { RESQ_OPT_DECODE_EARLY_WEIGHTS = 1, RESQ_OPT_WAIT_LIMIT_US = 2 };
int resq_set_option(int option, int value);

/* Inverse of the INT4 packing, for inspection: packed [rows][cols/2] -> int8 [rows][cols]. */
int resq_unpack_int4(const uint8_t* packed, int8_t* out, size_t rows, size_t cols, void* stream);

/* Synchronizes `stream`, then reads and clears the device status word of the current device:
 * RESQ_OK, RESQ_ERR_TIMEOUT, RESQ_ERR_INDEX (a timeout wins if both happened), or RESQ_ERR_CUDA if the stream
 * reported an error. */
int resq_device_status(void* stream);

/* Self-test of the failure path (no counterpart in the paper).  Every wait inside the kernels of this library is
 * bounded (Conventions above).  This call enqueues one small kernel whose only CTA waits for a barrier phase
 * that nothing completes: the wait runs out after the limit of RESQ_OPT_WAIT_LIMIT_US, the kernel records the
 * condition and returns by itself -- nothing traps, the context stays usable -- and the next resq_device_status
 * returns RESQ_ERR_TIMEOUT (and RESQ_OK again after that).  Set a short limit first (say 1000 us) and restore it
 * afterwards; with the default limit the kernel runs for two seconds. */
int resq_selftest_wait_runs_out(void* stream);

/* Number of kernels that the entry points of this library have enqueued in this process so far (host state; the
 * attention call counts its two kernels).  For accounting: a benchmark reads it before and after a timed region. */
unsigned long long resq_launch_count(void);

/* The CUDA runtime's description of the error behind the latest RESQ_ERR_CUDA that any entry point of
 * this process returned ("no error" if there was none).  Host state, for diagnostics. */
const char* resq_last_cuda_error(void);

/* Static, human-readable name of a status code. */
const char* resq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* RESQ_H_ */
