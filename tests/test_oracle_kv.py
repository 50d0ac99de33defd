"""Pins for the attention-block oracle (oracle/kv.py): Eq. 8, the 8-bit U_C projection, the per-head mixed
cache quantizer and single-query attention, each against something other than the oracle itself."""
import math

import numpy as np
import pytest

import oracle
from oracle import kv


def _orthogonal(d, seed):
    rng = np.random.default_rng(seed)
    q, r = np.linalg.qr(rng.standard_normal((d, d)))
    return q * np.sign(np.diag(r))


def _bf16(x):
    return oracle.bf16_bits_to_f32(oracle.f32_to_bf16_bits(np.asarray(x, np.float32)))


def test_eq8_scores_invariant_under_uc():
    """Eq. 8: (q U_C)(U_C^T K^T) = q K^T for orthogonal U_C, in fp64."""
    rng = np.random.default_rng(0)
    U = _orthogonal(128, 1)
    q, K = rng.standard_normal((4, 128)), rng.standard_normal((37, 128))
    assert np.abs((q @ U) @ (K @ U).T - q @ K.T).max() < 1e-12


def test_project_int8_orientation_and_error_bound():
    """project_int8(X, quantize_uc(U^T)) approximates X U (not X U^T) within the bound the two roundings allow:
    |y_j - (xU)_j| <= sum_i (|x_i| s_u[j]/2 + |U_ij| s_x/2 + s_x s_u[j]/4) (+ fp32 epilogue rounding)."""
    d = 128
    U = _orthogonal(d, 2)
    X = _bf16(np.random.default_rng(3).standard_normal((9, d)) * 3.0)
    wq, s_u = kv.quantize_uc(U.T.astype(np.float32))
    Y, xq, s_x = kv.project_int8(X, wq, s_u)
    exact = X.astype(np.float64) @ U.astype(np.float32).astype(np.float64)
    bound = (np.abs(X).sum(1)[:, None] * s_u[None, :] / 2 + (np.abs(U.astype(np.float32)).sum(0)[None, :]) * s_x[:, None] / 2
             + d * s_x[:, None] * s_u[None, :] / 4) * (1 + 1e-5)
    assert (np.abs(Y - exact) <= bound).all()
    assert np.abs(Y - exact).max() < 0.05 * np.abs(exact).max()
    wrong = X.astype(np.float64) @ U.T
    assert np.abs(Y - wrong).max() > 0.5 * np.abs(exact).max()


def test_project_int8_brute_force_tiny():
    """d = 16, 3 rows: products of dequantized codes summed in fp64 (Python loops) against the fp32 epilogue."""
    d = 16
    U = _orthogonal(d, 4).astype(np.float32)
    X = _bf16(np.random.default_rng(5).standard_normal((3, d)))
    wq, s_u = kv.quantize_uc(U.T.copy())
    Y, xq, s_x = kv.project_int8(X, wq, s_u)
    for t in range(3):
        a = float(np.abs(X[t]).max())
        assert s_x[t] == np.float32(a) / np.float32(127)
        for j in range(d):
            ref = sum((int(xq[t, i]) * float(s_x[t])) * (int(wq[j, i]) * float(s_u[j])) for i in range(d))
            assert abs(float(Y[t, j]) - ref) <= 3 * np.spacing(np.float32(abs(ref))) + 1e-30
    # codes of U^T are per OUTPUT coefficient j: row j of wq encodes column j of U_C
    for j in range(d):
        col = U[:, j]
        assert s_u[j] == np.float32(np.abs(col).max()) / np.float32(127)
        assert abs(int(wq[j, int(np.abs(col).argmax())])) == 127


def test_query_kept_in_half_precision():
    y = np.array([[1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 65504.0, 1e-8]], np.float32)
    h = kv.query_fp16(y)
    assert h.dtype == np.float16
    assert float(h[0, 0]) == 1.0 and float(h[0, 1]) == 1.0 + 2.0 ** -9 and float(h[0, 2]) == 65504.0  # ties to even


@pytest.mark.parametrize("d", [128, 64])
def test_kv_quantize_layout_and_bounds(d):
    """The first d/8 coefficients in 8 bits, the rest in 4 (d = 128 and the 64-wide heads of the small model)."""
    rng = np.random.default_rng(6)
    rows, r = 11, d // 8
    Y = (rng.standard_normal((rows, d)) * np.r_[np.full(r, 8.0), np.ones(d - r)] + 0.7).astype(np.float32)
    h = kv.kv_quantize(Y)
    assert h.c8.shape == (rows, r) and h.u4.shape == (rows, d - r) and h.c4.shape == (rows, (d - r) // 2) and h.meta.shape == (rows, 4)
    assert h.u4.max() == 15 and h.c8.max() == 255 and h.c8.min() == 0 and h.u4.min() == 0
    for t in range(rows):
        s8, z8, s4, z4 = (np.float32(v) for v in h.meta[t])
        assert z8 == Y[t, :r].min() and z4 == Y[t, r:].min()
        assert s8 == (Y[t, :r].max() - Y[t, :r].min()) / np.float32(255)
        assert s4 == (Y[t, r:].max() - Y[t, r:].min()) / np.float32(15)
        assert h.c8[t, Y[t, :r].argmax()] == 255 and h.u4[t, Y[t, r:].argmin()] == 0
    xh = kv.kv_dequantize(h)
    err = np.abs(xh - Y)
    assert (err[:, :r] <= h.meta[:, 0:1] / 2 * (1 + 1e-4)).all() and (err[:, r:] <= h.meta[:, 2:3] / 2 * (1 + 1e-4)).all()
    # two codes per byte, code 2i in the low nibble
    assert (h.c4 == (h.u4[:, 0::2] | (h.u4[:, 1::2] << 4))).all()


def _cache(rng, B, Hkv, S, d):
    K = [[None] * Hkv for _ in range(B)]
    V = [[None] * Hkv for _ in range(B)]
    for b in range(B):
        for h in range(Hkv):
            K[b][h] = rng.standard_normal((S, d))
            V[b][h] = rng.standard_normal((S, d))
    return K, V


def test_attention_special_cases():
    rng = np.random.default_rng(7)
    d, Hq, Hkv = 16, 4, 2
    K, V = _cache(rng, 2, Hkv, 5, d)
    q = rng.standard_normal((2, Hq, d)).astype(np.float16)
    # one position: the output is that value vector, whatever the score
    o = kv.attention_decode(q, K, V, [1, 1], Hq, Hkv)
    for b in range(2):
        for h in range(Hq):
            assert np.allclose(o[b, h], V[b][h // 2][0], rtol=0, atol=1e-15)
    # equal keys: uniform weights, the mean of the values
    for b in range(2):
        for h in range(Hkv):
            K[b][h][:] = K[b][h][0]
    o = kv.attention_decode(q, K, V, [5, 3], Hq, Hkv)
    assert np.allclose(o[0, 3], V[0][1].mean(0), atol=1e-14) and np.allclose(o[1, 0], V[1][0][:3].mean(0), atol=1e-14)
    # an empty sequence gives 0 and positions past seq_len are never read
    V[0][0][2:] = np.nan
    K[0][0][2:] = np.nan
    o = kv.attention_decode(q, K, V, [2, 0], Hq, Hkv)
    assert np.isfinite(o[0]).all() and (o[1] == 0).all()


def test_attention_brute_force_tiny():
    """Definition written out with Python loops and math.exp: softmax(q K^T / sqrt(d)) V, grouped heads."""
    rng = np.random.default_rng(8)
    d, Hq, Hkv, S = 8, 6, 2, 7
    K, V = _cache(rng, 1, Hkv, S, d)
    q = rng.standard_normal((1, Hq, d)).astype(np.float16)
    o = kv.attention_decode(q, K, V, [S], Hq, Hkv)
    for h in range(Hq):
        kvh = h // 3
        sc = [sum(float(q[0, h, i]) * K[0][kvh][j][i] for i in range(d)) / math.sqrt(d) for j in range(S)]
        w = [math.exp(s) for s in sc]
        for i in range(d):
            ref = sum(w[j] * V[0][kvh][j][i] for j in range(S)) / sum(w)
            assert abs(o[0, h, i] - ref) < 1e-13


def test_mixed_cache_beats_uniform_4bit_on_high_variance_heads():
    """Sanity (not parity): with the variance concentrated in the first d/8 coefficients, as the PCA basis
    arranges (Section 4.1), attention on the 8/4 cache is closer to the unquantized result than on a cache
    whose every coefficient has 4 bits."""
    rng = np.random.default_rng(9)
    d, S = 128, 256
    scale = np.r_[np.full(16, 6.0), np.ones(112)]
    Kf = (rng.standard_normal((S, d)) * scale).astype(np.float32)
    Vf = (rng.standard_normal((S, d)) * scale).astype(np.float32)
    q = (rng.standard_normal((1, 1, d)) * 0.3).astype(np.float16)
    exact = kv.attention_decode(q, [[Kf.astype(np.float64)]], [[Vf.astype(np.float64)]], [S], 1, 1)
    mixed = kv.attention_decode(q, [[kv.kv_dequantize(kv.kv_quantize(Kf))]], [[kv.kv_dequantize(kv.kv_quantize(Vf))]], [S], 1, 1)

    def uniform4(Y):
        u8, u4, s8, s4, z8, z4 = oracle.split_quantize_asym(Y, 0)
        return u4.astype(np.float64) * s4[:, None].astype(np.float64) + z4[:, None].astype(np.float64)

    uni = kv.attention_decode(q, [[uniform4(Kf)]], [[uniform4(Vf)]], [S], 1, 1)
    e_mixed, e_uni = np.linalg.norm(mixed - exact), np.linalg.norm(uni - exact)
    assert e_mixed < 0.5 * e_uni


def test_attention_queries_against_masked_matrix_form_and_special_cases():
    """Many-query attention pinned by an independent formulation -- causal self-attention written as one masked
    score matrix per head (mask, row softmax, matrix product) -- and by what the definition fixes: a query of
    prefix length 1 returns the first value vector, equal keys give the running mean of the values, an empty
    prefix gives 0, rows may come in any order and may address different sequences."""
    rng = np.random.default_rng(21)
    d, Hq, Hkv, S = 16, 4, 2, 9
    K, V = _cache(rng, 2, Hkv, S, d)
    q = rng.standard_normal((S, Hq, d)).astype(np.float16)
    # causal prefill of sequence 1: token at position p attends positions <= p
    out = kv.attention_queries(q, K, V, np.ones(S, int), np.arange(1, S + 1), Hq, Hkv)
    for h in range(Hq):
        sc = q[:, h].astype(np.float64) @ K[1][h // 2].T / math.sqrt(d)           # [S queries][S keys]
        sc = np.where(np.tril(np.ones((S, S), bool)), sc, -np.inf)
        w = np.exp(sc - sc.max(1, keepdims=True))
        ref = (w / w.sum(1, keepdims=True)) @ V[1][h // 2]
        assert np.abs(out[:, h] - ref).max() < 1e-13
        assert np.allclose(out[0, h], V[1][h // 2][0], rtol=0, atol=1e-15)         # prefix of one position
    # a permutation of the rows permutes the outputs; rows of different sequences do not interact
    perm = rng.permutation(S)
    seqs = np.r_[np.ones(S, int), np.zeros(3, int)]
    lens = np.r_[np.arange(1, S + 1)[perm], [0, 4, S]]
    qq = np.concatenate([q[perm], q[:3]])
    out2 = kv.attention_queries(qq, K, V, seqs, lens, Hq, Hkv)
    assert np.array_equal(out2[:S], out[perm])
    assert (out2[S] == 0).all()                                                    # empty prefix
    single = kv.attention_decode(q[1:3], K, V, [4, S], Hq, Hkv)                    # the single-query definition
    assert np.allclose(out2[S + 1], kv.attention_decode(q[1:2], [K[0]], [V[0]], [4], Hq, Hkv)[0], atol=1e-15)
    assert single.shape == (2, Hq, d)
    # equal keys: uniform weights over the prefix -> running means of the values
    for h in range(Hkv):
        K[1][h][:] = K[1][h][0]
    out3 = kv.attention_queries(q, K, V, np.ones(S, int), np.arange(1, S + 1), Hq, Hkv)
    for p in range(S):
        assert np.allclose(out3[p, 3], V[1][1][:p + 1].mean(0), atol=1e-14)
