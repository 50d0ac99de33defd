/*
 * CPU oracle for the ResQ mixed-precision linear layer.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct restatement of the paper's definitions, used by the tests, the
 * smoke check and the benchmark's CPU-baseline leg to judge the CUDA path.  It shares no code with
 * the CUDA library and the product never calls it.
 *
 *   Eq. 1 (Section 3)   symmetric N-bit quantizer: s = max|x| / (2^(N-1) - 1), code = round(x / s), clipped
 *   Eq. 2 (Section 4.1) activation coefficients X·U: r of them at H = 8 bits, the other d - r at L = 4 bits
 *   Eq. 3 (Section 4.1) projected weights U^T·W quantized the same way, one scale per output channel and segment
 *   Eq. 4 (Section 4.1) layer output = low-precision product + high-precision product (no cross terms)
 * and, further down, the asymmetric form of Eq. 1 for the activations (Section 5.1) with its epilogue.
 *
 * Readings where the paper is silent: rounding is to nearest, ties to even, in fp32 (rintf under the
 * default rounding mode); s and x/s are IEEE fp32 divisions; a zero segment gets s = 0 and codes 0;
 * codes are clipped to [-2^(N-1), 2^(N-1) - 1]; the high-precision coefficients come FIRST in a row;
 * one scale per (row, segment).
 *
 * Every pin lives in tests/test_oracle_*.py (brute force with exact rationals, closed forms,
 * invariants, library routines).  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------- format helpers (bf16 / fp16 are storage formats, widened exactly) ---------- */
static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bf16, round to nearest, ties to even (finite inputs). */
static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t keep = u >> 16, rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1;
    return (uint16_t)keep;
}

void oracle_bf16_to_f32(const uint16_t* in, long n, float* out) {
    for (long i = 0; i < n; ++i) out[i] = bf16_to_f32(in[i]);
}
void oracle_f32_to_bf16(const float* in, long n, uint16_t* out) {
    for (long i = 0; i < n; ++i) out[i] = f32_to_bf16(in[i]);
}

/* ---------- Eq. 1: symmetric quantizer on one vector ---------- */
/* bits = 8 or 4.  scale_fp16 != 0: the scale is stored as fp16, and codes are taken against the
 * stored value.  Returns the scale; writes n codes. */
float oracle_quantize_vector(const float* x, long n, int bits, int scale_fp16, int8_t* code) {
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const float lo = -(float)(1 << (bits - 1)), hi = qmax;
    float a = 0.0f;
    for (long j = 0; j < n; ++j) {
        float v = fabsf(x[j]);
        if (v > a) a = v;
    }
    float s = a / qmax;
    if (scale_fp16) s = (float)(_Float16)s;
    if (!(s > 0.0f)) {
        for (long j = 0; j < n; ++j) code[j] = 0;
        return 0.0f;
    }
    for (long j = 0; j < n; ++j) {
        float q = rintf(x[j] / s);
        if (q < lo) q = lo;
        if (q > hi) q = hi;
        code[j] = (int8_t)q;
    }
    return s;
}

/* ---------- Eq. 2 / Eq. 3: split quantization of the rows of a [rows][K] fp32 matrix ---------- */
/* q8 [rows][r], q4 [rows][K-r] (one code per byte), s8/s4 [rows]. */
void oracle_split_quantize(const float* C, long rows, int K, int r, int scale_fp16,
                           int8_t* q8, int8_t* q4, float* s8, float* s4) {
    const int K4 = K - r;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < rows; ++t) {
        s8[t] = oracle_quantize_vector(C + t * K, r, 8, scale_fp16, q8 + t * r);
        s4[t] = oracle_quantize_vector(C + t * K + r, K4, 4, scale_fp16, q4 + t * K4);
    }
}

/* Uniform-precision form of Eq. 1 on every row of a [rows][n] matrix (one scale per row). */
void oracle_quantize_rows(const float* x, long rows, int n, int bits, int8_t* code, float* s) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < rows; ++t) s[t] = oracle_quantize_vector(x + t * n, n, bits, 0, code + t * n);
}

/* Canonical nibble packing: byte i holds code 2i in bits 0..3 and code 2i+1 in bits 4..7, two's complement. */
void oracle_pack_nibbles(const int8_t* code, long n, uint8_t* packed) {
    for (long i = 0; i < n / 2; ++i)
        packed[i] = (uint8_t)((code[2 * i] & 0x0F) | ((code[2 * i + 1] & 0x0F) << 4));
}
void oracle_unpack_nibbles(const uint8_t* packed, long n, int8_t* code) {
    for (long i = 0; i < n / 2; ++i) {
        int l = packed[i] & 0x0F, h = packed[i] >> 4;
        code[2 * i] = (int8_t)(l >= 8 ? l - 16 : l);
        code[2 * i + 1] = (int8_t)(h >= 8 ? h - 16 : h);
    }
}

/* ---------- online projection (Section 4.3, U_D): C = X·P, bf16 inputs widened exactly ---------- */
/* X [T][K] bf16, P [K][K] bf16 (row i = input feature, column j = coefficient).  Each coefficient is
 * summed in fp64 and rounded once to fp32; it is never rounded to bf16. */
void oracle_project(const uint16_t* X, const uint16_t* P, long T, int K, float* C) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        double* acc = (double*)calloc((size_t)K, sizeof(double));
        /* acc[j] = sum over i (ascending) of X[t][i] * P[i][j]; the i loop is outermost only so that
         * P is walked along its rows -- each coefficient's sum keeps its order. */
        for (int i = 0; i < K; ++i) {
            const double x = (double)bf16_to_f32(X[t * K + i]);
            const uint16_t* prow = P + (long)i * K;
            for (int j = 0; j < K; ++j) acc[j] += x * (double)bf16_to_f32(prow[j]);
        }
        for (int j = 0; j < K; ++j) C[t * K + j] = (float)acc[j];
        free(acc);
    }
}

/* ---------- Eq. 4: one same-precision integer product, acc[t][n] = sum_j x[t][j] * w[n][j] ---------- */
/* int64 accumulation; returns the number of outputs that would not fit int32 (must be 0). */
long oracle_int_gemm(const int8_t* x, const int8_t* w, long T, long N, int Kseg, int32_t* acc) {
    long overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (long t = 0; t < T; ++t) {
        for (long n = 0; n < N; ++n) {
            int64_t a = 0;
            for (int j = 0; j < Kseg; ++j) a += (int64_t)x[t * Kseg + j] * (int64_t)w[n * Kseg + j];
            if (a > INT32_MAX || a < INT32_MIN) overflow += 1;
            acc[t * N + n] = (int32_t)a;
        }
    }
    return overflow;
}

/* ---------- dequantizing epilogue of Eq. 4 ---------- */
/* y = acc8·s_x8[t]·s_w8[n] + acc4·s_x4[t]·s_w4[n], evaluated in fp64 from the stored fp32 scale
 * values, rounded once to fp32 (y32) and from there to bf16 (ybf). */
void oracle_epilogue(const int32_t* acc8, const int32_t* acc4, const float* s_x8, const float* s_x4,
                     const float* s_w8, const float* s_w4, long T, long N, float* y32, uint16_t* ybf) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        for (long n = 0; n < N; ++n) {
            double y = (double)acc8[t * N + n] * (double)s_x8[t] * (double)s_w8[n] +
                       (double)acc4[t * N + n] * (double)s_x4[t] * (double)s_w4[n];
            float yf = (float)y;
            y32[t * N + n] = yf;
            if (ybf) ybf[t * N + n] = f32_to_bf16(yf);
        }
    }
}

/* ====================================================================================================
 * Asymmetric per-token activations (Eq. 1, second form; the setting of the paper's experiments, Section 5.1):
 *     z = min(x),  s = (max(x) - min(x)) / (2^N - 1),  code = round((x - z) / s) clipped to [0, 2^N - 1],
 *     dequantized value = code * s + z.
 * Readings where the paper is silent: max - min, x - z and the two divisions are IEEE fp32 operations in this
 * order; rounding is to nearest, ties to even; a constant segment gets s = 0 and codes 0 (its dequantized value
 * is z exactly); the zero-point stays an fp32 number (it is not snapped to the integer grid).
 * With symmetric weights (Eq. 3) the layer output (Eq. 4) becomes, per segment,
 *     sum_j (code_j * s_x + z_x) * (w_j * s_w) = s_x * s_w * sum_j code_j * w_j  +  z_x * s_w * sum_j w_j,
 * i.e. the integer product plus a rank-one term with the integer row sums of the weight codes.
 * ==================================================================================================== */
void oracle_quantize_vector_asym(const float* x, long n, int bits, uint8_t* code, float* s_out, float* z_out) {
    const float qmax = (float)((1 << bits) - 1);
    if (n == 0) { /* an empty segment (r = 0): nothing to quantize, s = 0 and z = 0 */
        *s_out = 0.0f;
        *z_out = 0.0f;
        return;
    }
    float lo = x[0], hi = x[0];
    for (long j = 1; j < n; ++j) {
        if (x[j] < lo) lo = x[j];
        if (x[j] > hi) hi = x[j];
    }
    const float range = hi - lo;
    const float s = range / qmax;
    *z_out = lo;
    if (!(s > 0.0f)) {
        for (long j = 0; j < n; ++j) code[j] = 0;
        *s_out = 0.0f;
        return;
    }
    *s_out = s;
    for (long j = 0; j < n; ++j) {
        const float d = x[j] - lo;
        float q = rintf(d / s);
        if (q < 0.0f) q = 0.0f;
        if (q > qmax) q = qmax;
        code[j] = (uint8_t)q;
    }
}

/* u8 [rows][r], u4 [rows][K-r] (one code per byte), s8/s4/z8/z4 [rows]. */
void oracle_split_quantize_asym(const float* C, long rows, int K, int r, uint8_t* u8, uint8_t* u4,
                                float* s8, float* s4, float* z8, float* z4) {
    const int K4 = K - r;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < rows; ++t) {
        oracle_quantize_vector_asym(C + t * K, r, 8, u8 + t * r, s8 + t, z8 + t);
        oracle_quantize_vector_asym(C + t * K + r, K4, 4, u4 + t * K4, s4 + t, z4 + t);
    }
}

/* acc[t][n] = sum_j u[t][j] * w[n][j] with unsigned activation codes; int64, overflow count returned. */
long oracle_int_gemm_u8(const uint8_t* u, const int8_t* w, long T, long N, int Kseg, int32_t* acc) {
    long overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (long t = 0; t < T; ++t) {
        for (long n = 0; n < N; ++n) {
            int64_t a = 0;
            for (int j = 0; j < Kseg; ++j) a += (int64_t)u[t * Kseg + j] * (int64_t)w[n * Kseg + j];
            if (a > INT32_MAX || a < INT32_MIN) overflow += 1;
            acc[t * N + n] = (int32_t)a;
        }
    }
    return overflow;
}

/* Row sums of the weight codes: wsum[n] = sum_j w[n][j]. */
void oracle_weight_row_sums(const int8_t* w, long N, int Kseg, int32_t* wsum) {
    for (long n = 0; n < N; ++n) {
        int64_t a = 0;
        for (int j = 0; j < Kseg; ++j) a += w[n * Kseg + j];
        wsum[n] = (int32_t)a;
    }
}

/* y = acc8*s_x8*s_w8 + z_x8*s_w8*wsum8 + acc4*s_x4*s_w4 + z_x4*s_w4*wsum4 in fp64 from the stored fp32
 * values, rounded once to fp32 and from there to bf16. */
void oracle_epilogue_asym(const int32_t* acc8, const int32_t* acc4, const float* s_x8, const float* s_x4,
                          const float* z_x8, const float* z_x4, const float* s_w8, const float* s_w4,
                          const int32_t* wsum8, const int32_t* wsum4, long T, long N, float* y32, uint16_t* ybf) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        for (long n = 0; n < N; ++n) {
            double y = (double)acc8[t * N + n] * (double)s_x8[t] * (double)s_w8[n] +
                       (double)z_x8[t] * (double)s_w8[n] * (double)wsum8[n] +
                       (double)acc4[t * N + n] * (double)s_x4[t] * (double)s_w4[n] +
                       (double)z_x4[t] * (double)s_w4[n] * (double)wsum4[n];
            float yf = (float)y;
            y32[t * N + n] = yf;
            if (ybf) ybf[t * N + n] = f32_to_bf16(yf);
        }
    }
}

/* Number of threads the parallel loops use (for the benchmark's "cores" field). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif
