// Internal declarations shared by the translation units of the library (host side).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/resq.h"
#include "../../include/resq_kv.h"

namespace resq {

// Device status block (one per device that loaded the library): int word 0 collects the condition bits that
// kernels OR in (kStatusBitTimeout, kStatusBitIndex below), the 64-bit word at byte offset 8 holds the limit
// of one bounded wait in nanoseconds.
int* device_status_ptr();  // device address of the block of the current device, or nullptr
// Counts kernels enqueued by this process (resq_launch_count); called once per launch by the wrappers below.
void count_launch(int n = 1);
constexpr int kStatusBitTimeout = 1;  // a bounded wait ran out
constexpr int kStatusBitIndex = 2;    // an index read on the device was out of range

// ---- kernels (launch wrappers; return cudaGetLastError()) ----------------------------------
// Split quantization of the rows of a [rows][K] matrix (Eq. 2 for activations, Eq. 3 for weights).
//   in_is_f32: rows are fp32 (weights, projected coefficients) instead of bf16.
//   scale_fp16: scales are rounded to and stored as fp16 (weights only).
//   programmatic: enqueue with programmatic stream serialization (the kernel waits for the preceding grid itself,
//                 so its CTAs can be scheduled while that grid drains); only the whole-row kernel honours it.
cudaError_t launch_split_quantize(const void* in, bool in_is_f32, size_t rows, int K, int r, int8_t* q8,
                                  uint8_t* q4, void* s8, void* s4, bool scale_fp16, int8_t* q4_i8,
                                  size_t in_row_stride, cudaStream_t st, bool programmatic = false);

// GPTQ rounding of the rows of W [N][K] fp32 with the upper Cholesky factor U [K][K] fp32 of the inverse Hessian
// (Section 5.1); dead: optional [K] bytes, non-zero = the column's weights are zeroed.  Returns cudaErrorNotSupported
// when a row (9 bytes per weight) does not fit in shared memory.
cudaError_t launch_pack_gptq(const float* W, const float* U, const uint8_t* dead, int N, int K, int r, int8_t* w8,
                             uint8_t* w4, void* s8, void* s4, bool scale_fp16, int8_t* w4e, cudaStream_t st);

// Hadamard transform of the bf16 rows (H_K / sqrt(K), K = 2^k * {1, 12, 28}) fused with the split quantizer
// (r may be 0).  Returns cudaErrorNotSupported for other K or rows wider than 200 KB of fp32.
cudaError_t launch_hadamard_quantize(const void* X, size_t rows, int K, int r, int8_t* q8, uint8_t* q4, float* s8,
                                     float* s4, int8_t* q4_i8, cudaStream_t st);

// codes_unsigned: the nibbles are 0..15 (asymmetric activation codes) instead of two's complement.
cudaError_t launch_unpack_int4(const uint8_t* packed, int8_t* out, size_t rows, size_t cols, cudaStream_t st,
                               bool codes_unsigned = false);

// Many-token tile kernel on tcgen05 kind::i8.  x4e / w4e are the INT4 codes one per byte.
cudaError_t launch_mixed_gemm_tiles(int T, int N, int K, int r, const int8_t* x8, const int8_t* x4e,
                                    const float* s_x8, const float* s_x4, const int8_t* w8, const int8_t* w4e,
                                    const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                    int32_t* dbg8, int32_t* dbg4, cudaStream_t st, const float* z_x8 = nullptr,
                                    const float* z_x4 = nullptr, const int32_t* wsum8 = nullptr,
                                    const int32_t* wsum4 = nullptr);
// z_x8 != NULL selects asymmetric activations: x8 / x4e then hold UNSIGNED codes (0..255, 0..15) and the
// epilogue adds z_x8[t] * s_w8[n] * wsum8[n] + z_x4[t] * s_w4[n] * wsum4[n].

// Asymmetric split quantization (Eq. 1, second form) of the rows of a [rows][K] matrix.  Returns
// cudaErrorNotSupported for rows wider than 200 KB.
cudaError_t launch_split_quantize_asym(const void* in, bool in_is_f32, size_t rows, int K, int r, uint8_t* u8,
                                       uint8_t* u4, float* s8, float* s4, float* z8, float* z4, uint8_t* u4_u8,
                                       size_t in_row_stride_bytes, cudaStream_t st);
// wsum8[n] = sum_j w8[n][j], wsum4[n] = sum_j w4[n][j] (packed codes).
cudaError_t launch_weight_row_sums(const int8_t* w8, const uint8_t* w4, int N, int K, int r, int32_t* wsum8,
                                   int32_t* wsum4, cudaStream_t st);

// Few-token (T <= 16) streaming kernel (persistent grid, bulk-copy ring).  Returns cudaErrorNotSupported, with
// nothing launched, when the staged activations leave no room for the ring; the caller then splits the tokens
// over two launches.
cudaError_t launch_mixed_gemm_stream(int T, int N, int K, int r, const int8_t* x8, const uint8_t* x4,
                                     const float* s_x8, const float* s_x4, const int8_t* w8, const uint8_t* w4,
                                     const void* s_w8, const void* s_w4, bool w_scale_fp16, void* Y, int y_dtype,
                                     int32_t* dbg8, int32_t* dbg4, cudaStream_t st, const float* z_x8 = nullptr,
                                     const float* z_x4 = nullptr, const int32_t* wsum8 = nullptr,
                                     const int32_t* wsum4 = nullptr);  // z_x8 != NULL: asymmetric, unsigned codes
void set_decode_early_weights(int on);

// Online projection C = X·P (bf16 x bf16 -> fp32) on tcgen05 kind::f16, CTA pairs; writes fp32 C [T][K].
// scratch (optional, project_split_scratch_bytes() bytes): lets a thinly filled last round of tiles be cut along K.
size_t project_split_scratch_bytes();
cudaError_t launch_project_gemm(const void* X, const void* P, int T, int K, float* C, cudaStream_t st,
                                void* scratch = nullptr, size_t scratch_bytes = 0);

// ---- attention-block path (declared in resq_kv.h) ----
cudaError_t launch_uc_quantize(const float* W_C, int8_t* wq, float* s_u, cudaStream_t st);
// Query projection and / or cache update in one launch (either part may be absent: q == NULL, or k == NULL).
cudaError_t launch_qkv_project_append(const resq_kv_cache_t* cache, const void* q, long long q_rows, void* q_out,
                                      const void* k, const void* v, long long T, const int32_t* seq_ids,
                                      const int32_t* positions, const int8_t* wq, const float* s_u, cudaStream_t st);
size_t attention_scratch_bytes(int n_seqs, int n_kv_heads);
// n_rows >= 0 with seq_map: the many-query form -- q16 / out / seq_lens have n_rows rows and row i reads the first
// seq_lens[i] positions of cache sequence seq_map[i]; scratch: attention_scratch_bytes(n_rows, n_kv_heads).
cudaError_t launch_attention_decode(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, const int32_t* seq_lens,
                                    float* out, void* scratch, cudaStream_t st, int n_rows = -1,
                                    const int32_t* seq_map = nullptr);

// Causal attention of T new tokens of sequence `seq` (positions pos0 .. pos0 + T - 1) on the tensor cores.
cudaError_t launch_attention_prefill(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, int seq, int pos0,
                                     int T, float* out, cudaStream_t st);

// d_head = 64 (plain kernels, same arithmetic and cache format with every code array halved).
size_t kv64_block_bytes();
cudaError_t launch_uc_quantize64(const float* W_C, int8_t* wq, float* s_u, cudaStream_t st);
cudaError_t launch_qkv_project_append64(const resq_kv_cache_t* cache, const void* q, long long q_rows, void* q_out,
                                        const void* k, const void* v, long long T, const int32_t* seq_ids,
                                        const int32_t* positions, const int8_t* wq, const float* s_u, cudaStream_t st);
// Row i of q16 / out attends the first len_of_row[i] (null: len0 + i + 1) positions of sequence seq_of_row[i] (null:
// seq_const if >= 0, else i).
cudaError_t launch_attention64(const resq_kv_cache_t& cache, const void* q16, int n_q_heads, int rows,
                               const int32_t* seq_of_row, const int32_t* len_of_row, int seq_const, int len0, float* out,
                               cudaStream_t st);

// Driver entry point for tensor-map encoding (resolved once, without linking libcuda).
void* tensor_map_encode_fn();

}  // namespace resq
