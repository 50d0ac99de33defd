"""CPU oracle for the attention-block path of ResQ (Section 4.3, Eq. 8; Section 5.1) -- TEST INFRASTRUCTURE ONLY.

What the paper fixes: query and key are multiplied, after the rotary embedding, by the same orthogonal
d_head x d_head matrix U_C at run time, with U_C and the projection's input in 8-bit (Section 5.1); the
value basis U_B is folded into the neighbouring weights and has no run-time step; the KV cache is
quantized per head, asymmetrically, to 4 bits with the first 1/8 of each head's coefficients in 8 bits
(Section 5.1, Appendix "Additional implementation details"); the query stays in 16 bits.

Every function takes the steps in that order with numpy / the C quantizers of this package; nothing is
blocked or fused.  Attention itself is the textbook definition in fp64 on the dequantized cache.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import int_gemm, pack_nibbles_u, quantize_rows, split_quantize_asym


def quantize_uc(W_C):
    """W_C = U_C^T as a weight [d_out][d_in]: symmetric per-output-channel INT8 (Eq. 1, uniform 8-bit).
    Returns (codes int8 [d][d], s_u fp32 [d])."""
    W_C = np.ascontiguousarray(W_C, np.float32)
    assert W_C.ndim == 2 and W_C.shape[0] == W_C.shape[1]
    return quantize_rows(W_C, 8)


def project_int8(X, wq, s_u):
    """Online U_C projection in 8-bit (Section 4.3, Section 5.1): each row of X [rows][d] (one head vector of
    one token) gets a symmetric INT8 scale, the contraction is exact in integers, and
    y[t][j] = fl32(fl32(acc[t][j]) * fl32(s_x[t] * s_u[j])).  Returns (Y fp32, codes, s_x)."""
    X = np.ascontiguousarray(X, np.float32)
    xq, s_x = quantize_rows(X, 8)
    acc = int_gemm(xq, wq)
    scale = s_x[:, None].astype(np.float32) * np.asarray(s_u, np.float32)[None, :]
    Y = acc.astype(np.float32) * scale
    assert Y.dtype == np.float32
    return Y, xq, s_x


def query_fp16(Y):
    """The projected query is kept in 16 bits (Appendix): round-to-nearest-even to IEEE half."""
    return np.asarray(Y, np.float32).astype(np.float16)


@dataclass
class HeadCodes:
    """Mixed-precision codes of head vectors [rows][d]: the first d/8 coefficients in 8 bits, the rest in 4."""
    c8: np.ndarray    # uint8 [rows][d/8]
    u4: np.ndarray    # uint8 [rows][7d/8], one code per byte
    c4: np.ndarray    # uint8 [rows][7d/16], two codes per byte (code 2i in the low nibble)
    meta: np.ndarray  # fp32 [rows][4] = (s8, z8, s4, z4)


def kv_quantize(Y) -> HeadCodes:
    """Per-head asymmetric cache quantizer (Section 5.1): Eq. 1 with z = min and s = (max - min) / (2^N - 1) on
    the two segments of every head vector."""
    Y = np.ascontiguousarray(Y, np.float32)
    rows, d = Y.shape
    assert d % 16 == 0
    c8, u4, s8, s4, z8, z4 = split_quantize_asym(Y, d // 8)
    return HeadCodes(c8, u4, pack_nibbles_u(u4), np.stack([s8, z8, s4, z4], axis=1).astype(np.float32))


def kv_dequantize(h: HeadCodes):
    """x_hat = code * s + z per segment (Eq. 1), evaluated in fp64 from the stored fp32 scale and zero-point."""
    s8, z8, s4, z4 = (h.meta[:, i].astype(np.float64)[:, None] for i in range(4))
    return np.concatenate([h.c8.astype(np.float64) * s8 + z8, h.u4.astype(np.float64) * s4 + z4], axis=1)


def attention_decode(q16, K_hat, V_hat, seq_lens, n_q_heads: int, n_kv_heads: int):
    """Single-query attention on the dequantized cache, fp64.

    q16   [B][Hq][d]            projected queries (fp16 values)
    K_hat [B][Hkv][S][d] fp64   dequantized keys (projected by U_C), V_hat likewise (U_B basis)
    Query head h reads KV head h // (Hq / Hkv).  out[b][h] = softmax(q K^T / sqrt(d)) V over the first
    seq_lens[b] positions (Eq. 8 shows the scores equal those of the unprojected q and K)."""
    q = np.asarray(q16, np.float64)
    B, Hq, d = q.shape
    assert Hq == n_q_heads and Hq % n_kv_heads == 0
    g = Hq // n_kv_heads
    out = np.zeros((B, Hq, d), np.float64)
    for b in range(B):
        S = int(seq_lens[b])
        if S == 0:  # nothing to attend to: the output is defined as 0
            continue
        for h in range(Hq):
            K = K_hat[b][h // g][:S]
            V = V_hat[b][h // g][:S]
            sc = (K @ q[b, h]) / np.sqrt(float(d))
            p = np.exp(sc - sc.max())
            p /= p.sum()
            out[b, h] = p @ V
    return out


def attention_queries(q16, K_hat, V_hat, q_seq, q_len, n_q_heads: int, n_kv_heads: int):
    """Many-query attention on the dequantized cache, fp64: query row i attends the first q_len[i] positions of
    sequence q_seq[i] (causal attention of a token at position p is q_len = p + 1).  The textbook definition, one
    row at a time: out[i][h] = softmax(q[i][h] K^T / sqrt(d)) V over those positions; an empty prefix gives 0.

    q16 [n][Hq][d]; K_hat / V_hat [B][Hkv][S][d] fp64 (lists of arrays)."""
    q = np.asarray(q16, np.float64)
    n, Hq, d = q.shape
    assert Hq == n_q_heads and Hq % n_kv_heads == 0
    g = Hq // n_kv_heads
    out = np.zeros((n, Hq, d), np.float64)
    for i in range(n):
        b, L = int(q_seq[i]), int(q_len[i])
        if L == 0:
            continue
        for h in range(Hq):
            K = K_hat[b][h // g][:L]
            V = V_hat[b][h // g][:L]
            sc = (K @ q[i, h]) / np.sqrt(float(d))
            p = np.exp(sc - sc.max())
            out[i, h] = (p / p.sum()) @ V
    return out
