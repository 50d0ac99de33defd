/*
 * resq_kv.h -- C ABI of the attention-block path of ResQ for NVIDIA B200 (sm_100a): the online U_C
 * projection of query and key, the mixed-precision KV cache and single-query attention on it.
 *
 * What the paper defines (Section 4.3 "Projections within the attention block", Eq. 8; Section 5.1 and the
 * appendix on implementation details):
 *  - The value basis U_B is multiplied into the v_proj / o_proj weights offline: no run-time step here.
 *  - Query and key are multiplied AFTER the rotary embedding by the same orthogonal d_head x d_head matrix
 *    U_C, which leaves q·K^T unchanged (Eq. 8).  The product is formed at run time with U_C and its input
 *    in 8 bits.
 *  - The KV cache is quantized per head, asymmetrically, to 4 bits with the first d_head/8 coefficients of
 *    each head vector in 8 bits; the query stays in 16 bits.
 *
 * Arithmetic taken here (the paper fixes no operation order):
 *  - U_C enters as the weight W_C = U_C^T, fp32 [d_head][d_head], row j = output coefficient j, one matrix
 *    per layer shared by its heads; symmetric per-row INT8 (s_u[j] = max_i|W_C[j][i]| / 127, codes
 *    round-half-even(W_C[j][i] / s_u[j]), IEEE fp32 divisions).
 *  - Each head vector x (bf16, d_head values of one token) gets a symmetric INT8 scale s_x = max|x| / 127
 *    and codes the same way; the contraction is exact in int32;
 *        y[j] = (float)acc[j] * (s_x * s_u[j])                       (fp32, this order).
 *  - Query: y is rounded to IEEE half (nearest even).
 *  - Key: y stays fp32 and goes straight into the cache quantizer.  Value: the bf16 head vector (already
 *    in the U_B basis) goes into the same quantizer.
 *  - Cache quantizer, per head vector and per segment ([0, d/8) in 8 bits, [d/8, d) in 4 bits): z = min,
 *    s = (max - min) / (2^N - 1), code = round-half-even((x - z) / s) in [0, 2^N - 1] (fp32 subtraction and
 *    divisions in this order; a constant segment gives s = 0 and codes 0); the dequantized value is
 *    code * s + z.  s and z are stored as fp32.
 *  - Attention: out[h] = softmax_j(q[h]·K_hat[j] / sqrt(d_head)) · V_hat over the positions j < seq_len of
 *    the KV head h / (n_q_heads / n_kv_heads); K_hat, V_hat are the dequantized vectors.  Scores and the
 *    softmax are fp32; the softmax weights times the value scales are rounded to half before the second
 *    product; accumulation is fp32.  An empty sequence gives out = 0.
 *
 * Cache layout (one buffer per layer, caller-owned, any initial content).  Positions are grouped in blocks
 * of RESQ_KV_BLOCK = 32; the block of (sequence b, KV head h, positions [32i, 32i + 32)) starts at byte
 *        ((b * n_kv_heads + h) * (capacity / 32) + i) * RESQ_KV_BLOCK_BYTES
 * and holds, for p = position % 32 (d_head = 128):
 *        offset    0  k8   [32][16]  uint8   8-bit codes of key coefficients [0, 16)
 *        offset  512  k4   [32][56]  uint8   4-bit codes of key coefficients [16, 128), code 2i in the low nibble
 *        offset 2304  km   [32][4]   fp32    s8, z8, s4, z4 of the key
 *        offset 2816  v8, offset 3328 v4, offset 5120 vm: the same for the value
 * so one block is one contiguous 5632-byte transfer.  88 bytes per head vector instead of 256 in bf16.
 * For d_head = 64 every code array is half as wide (k8 [32][8] at 0, k4 [32][28] at 256, km at 1152, the value
 * half at 1664: 3328 bytes per block, 52 per head vector); resq_kv_block_bytes() gives the block size of a geometry.
 *
 * Conventions are those of resq.h: device pointers unless marked host, caller-owned memory, no allocation,
 * no stream synchronisation, 16-byte aligned pointers, status codes of resq_status_t, arguments validated
 * on the host before anything is enqueued.  d_head must be 128 or 64; capacity % 32 == 0;
 * n_q_heads / n_kv_heads must be an integer between 1 and 8.  d_head = 128 runs on the tuned kernels (mma.sync
 * fragments for the projection and the single-query pass, tcgen05 tiles for the prefill form); d_head = 64 runs the
 * same arithmetic and cache format on plain kernels (one warp per head vector / per query head, fp32 attention), so
 * its outputs meet the same bit-exact and tolerance statements but not the same speed.  Indices that live on the device (seq_ids,
 * positions, seq_lens) are checked by the kernels: an out-of-range entry is skipped (a sequence length is
 * clamped to the capacity) and RESQ_ERR_INDEX is reported by resq_device_status.
 */
#ifndef RESQ_KV_H_
#define RESQ_KV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RESQ_KV_BLOCK 32
#define RESQ_KV_BLOCK_BYTES 5632

typedef struct resq_kv_cache {
    int32_t n_seqs;     /* sequences the buffer has room for                     */
    int32_t n_kv_heads; /* KV heads per token                                    */
    int32_t d_head;     /* 128 or 64                                             */
    int32_t capacity;   /* positions per sequence, a multiple of RESQ_KV_BLOCK   */
    void* data;         /* resq_kv_cache_bytes() bytes, layout above             */
} resq_kv_cache_t;

/* Bytes of one cache block (32 positions of one KV head, keys and values): 5632 for d_head = 128, 3328 for 64, else 0. */
size_t resq_kv_block_bytes(int d_head);

/* n_seqs * n_kv_heads * (capacity / 32) * resq_kv_block_bytes(d_head), or 0 for an invalid geometry. */
size_t resq_kv_cache_bytes(int n_seqs, int n_kv_heads, int d_head, int capacity);

/* Section 5.1 ("U_C ... quantized to 8-bit"): INT8 codes wq [d_head][d_head] and scales s_u [d_head] of
 * W_C = U_C^T (fp32 [d_head][d_head]). */
int resq_uc_quantize(const float* W_C, int d_head, int8_t* wq, float* s_u, void* stream);

/* Section 4.3, Eq. 8, query side: q bf16 [rows][d_head] (rows = tokens x query heads, after the rotary
 * embedding) -> q_out IEEE half [rows][d_head] = half(q U_C) through the 8-bit product above. */
int resq_query_project(const void* q, int64_t rows, int d_head, const int8_t* wq, const float* s_u, void* q_out,
                       void* stream);

/* Section 4.3 / Section 5.1, cache side: for each of the T tokens, every key head vector k[t][h] (bf16
 * [T][n_kv_heads][d_head], after the rotary embedding) is projected by U_C in 8 bits, quantized and
 * written, with the quantized value head vector v[t][h] (bf16, same shape), at position positions[t] of
 * sequence seq_ids[t] (int32 [T] each).  Tokens of one call must address distinct (sequence, position)
 * pairs.  wq / s_u as written by resq_uc_quantize. */
int resq_kv_append(const resq_kv_cache_t* cache, const void* k, const void* v, int64_t T, const int32_t* seq_ids,
                   const int32_t* positions, const int8_t* wq, const float* s_u, void* stream);

/* resq_query_project and resq_kv_append of the same T tokens in one launch (q bf16 [T][n_q_heads][d_head]): the
 * query, key and value head vectors are independent pieces of work, so a generation step's few of them run side
 * by side instead of as two short kernels one after the other. */
int resq_qkv_project_append(const resq_kv_cache_t* cache, const void* q, int n_q_heads, void* q_out, const void* k,
                            const void* v, int64_t T, const int32_t* seq_ids, const int32_t* positions,
                            const int8_t* wq, const float* s_u, void* stream);

/* Scratch bytes of resq_attention_decode (0 for an invalid geometry). */
size_t resq_attention_workspace_bytes(int n_seqs, int n_q_heads, int n_kv_heads, int d_head);

/* Single-query attention over the cache (generation; the paper's Introduction calls this stage memory-bound):
 * q16 half [n_seqs][n_q_heads][d_head] (resq_query_project's output), seq_lens int32 [n_seqs], out fp32
 * [n_seqs][n_q_heads][d_head] in the U_B basis (o_proj's weights carry U_B^T).  Every cache byte of the
 * live positions is read once. */
int resq_attention_decode(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, const int32_t* seq_lens,
                          float* out, void* workspace, size_t workspace_bytes, void* stream);

/* Many-query attention over the cache (prefill, chunked prefill, speculative steps; Section 4.3 Eq. 8 with the cache
 * of Section 5.1): query row i -- q16 half [n_queries][n_q_heads][d_head] -- attends the first q_len[i] positions of
 * cache sequence q_seq[i] (int32 [n_queries] each); out fp32 [n_queries][n_q_heads][d_head].  Causal attention of
 * tokens appended at positions p_i is q_len[i] = p_i + 1, after the tokens have been appended.  The arithmetic per
 * query row is that of resq_attention_decode (same kernels, same tolerance; the fp32 partial sums of a row are merged
 * in the order its cache blocks fall on the grid's warps): every row streams its own prefix of the cache (from L2
 * when rows share a sequence), so the cost grows with the sum of the q_len, not with the tile products of a
 * tensor-core prefill kernel.  An out-of-range q_seq[i] is reported as RESQ_ERR_INDEX by resq_device_status (the row's
 * output is then unspecified); q_len is clamped like seq_lens.  n_queries >= 1. */
size_t resq_attention_queries_workspace_bytes(int n_queries, int n_q_heads, int n_kv_heads, int d_head);
int resq_attention_queries(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, int n_queries,
                           const int32_t* q_seq, const int32_t* q_len, float* out, void* workspace,
                           size_t workspace_bytes, void* stream);

/* Causal attention of a run of T new tokens of ONE sequence over the cache, on the tensor cores (prefill and chunked
 * prefill; Section 4.3 Eq. 8 with the cache of Section 5.1): token t -- q16 half [T][n_q_heads][d_head], at position
 * pos0 + t of cache sequence `seq` -- attends positions 0 .. pos0 + t, which must have been appended (the T new
 * tokens included); out fp32 [T][n_q_heads][d_head].  seq, pos0 and T are host values: 0 <= seq < n_seqs, pos0 >= 0,
 * T >= 1, pos0 + T <= capacity, else RESQ_ERR_SHAPE.  No workspace.
 * The same definition as resq_attention_queries with q_seq[t] = seq, q_len[t] = pos0 + t + 1, evaluated tile-wise: 128
 * (token, query head) rows that share a KV head meet 64 cache positions at a time, every cache block is read once per
 * such tile.  The score products run on the integer codes held exactly in half (scales and zero-points applied in
 * fp32), the softmax is fp32 with the row maximum found in a first pass over the keys, the softmax weights times the
 * value scales are rounded to half before the second product, accumulation is fp32. */
int resq_attention_prefill(const resq_kv_cache_t* cache, const void* q16, int n_q_heads, int seq, int pos0, int T,
                           float* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RESQ_KV_H_ */
