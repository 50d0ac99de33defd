"""Pins for the oracle's integer products, epilogue, projection and the whole layer (Eq. 2-4)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import synth
from oracle import basis
from tests.cases import config1


def test_int_gemm_brute_force_python_ints():
    rng = np.random.default_rng(0)
    x = rng.integers(-128, 128, (3, 10)).astype(np.int8)
    w = rng.integers(-128, 128, (4, 10)).astype(np.int8)
    acc = oracle.int_gemm(x, w)
    for t in range(3):
        for n in range(4):
            assert int(acc[t, n]) == sum(int(x[t, j]) * int(w[n, j]) for j in range(10))
    # operand roles are not symmetric: w is indexed [n][j]
    assert acc.shape == (3, 4)
    # extreme magnitudes at the largest segment sizes of the 70B-shaped config still fit int32
    assert oracle.int_gemm(np.full((1, 3584), -128, np.int8), np.full((1, 3584), -128, np.int8))[0, 0] == 128 * 128 * 3584


def test_epilogue_against_exact_rationals():
    rng = np.random.default_rng(1)
    acc8 = rng.integers(-5_000_000, 5_000_000, (3, 5)).astype(np.int32)
    acc4 = rng.integers(-300_000, 300_000, (3, 5)).astype(np.int32)
    sx8, sx4 = rng.random(3).astype(np.float32) * 0.1, rng.random(3).astype(np.float32)
    sw8, sw4 = rng.random(5).astype(np.float32) * 1e-3, rng.random(5).astype(np.float32) * 1e-2
    y32, ybf = oracle.epilogue(acc8, acc4, sx8, sx4, sw8, sw4)
    for t in range(3):
        for n in range(5):
            exact = (int(acc8[t, n]) * Fraction(float(sx8[t])) * Fraction(float(sw8[n]))
                     + int(acc4[t, n]) * Fraction(float(sx4[t])) * Fraction(float(sw4[n])))
            mag = abs(int(acc8[t, n]) * Fraction(float(sx8[t])) * Fraction(float(sw8[n]))) + \
                abs(int(acc4[t, n]) * Fraction(float(sx4[t])) * Fraction(float(sw4[n])))
            assert abs(Fraction(float(y32[t, n])) - exact) <= mag * Fraction(1, 2 ** 23)
    assert (ybf == synth.f32_to_bf16_bits(y32)).all()
    # scales index rows by token and columns by channel
    y2, _ = oracle.epilogue(np.ones((2, 3), np.int32), np.zeros((2, 3), np.int32),
                            np.array([1, 2], np.float32), np.zeros(2, np.float32),
                            np.array([1, 10, 100], np.float32), np.zeros(3, np.float32))
    assert y2.tolist() == [[1, 10, 100], [2, 20, 200]]


def test_tiny_layer_equals_dequantized_fp64_product():
    """d=16, r=2, T=3, N=4: the integer path times the scales equals the product of dequantized operands,
    with the block structure of the mixed-precision matrix product (no high x low cross term)."""
    K, r, T, N = 16, 2, 3, 4
    C = (synth.normal(31, 0, T * K).reshape(T, K) * 2).astype(np.float32)
    Wp = (synth.normal(32, 0, N * K).reshape(N, K) * 0.3).astype(np.float32)
    pw = oracle.pack_weights(Wp, r)
    res = oracle.linear_from_coeff(C, pw)
    Xq = np.concatenate([res.x8 * res.s_x8[:, None].astype(np.float64), res.x4 * res.s_x4[:, None].astype(np.float64)], 1)
    Wq = np.concatenate([pw.q8 * pw.s8[:, None].astype(np.float64), pw.q4 * pw.s4[:, None].astype(np.float64)], 1)
    ref = Xq @ Wq.T
    assert np.abs(res.y32 - ref).max() <= 1e-6 * np.abs(ref).max()
    # and it approximates the unquantized product to within the 4-bit grid
    exact = C.astype(np.float64) @ Wp.astype(np.float64).T
    assert np.abs(res.y32 - exact).max() < 0.5 * np.abs(exact).max()
    assert (res.x4_packed == oracle.pack_nibbles(res.x4)).all()


def test_projection_matches_blas_fp64():
    X = synth.activations(5, 256, "t4", seed=41)
    P = synth.kron_orthogonal_bf16(256, inner=16)
    C = oracle.project(synth.f32_to_bf16_bits(X), synth.f32_to_bf16_bits(P))
    ref = X.astype(np.float64) @ P.astype(np.float64)
    assert np.abs(C - ref).max() <= 2e-7 * np.abs(ref).max() + 1e-30
    # orientation: rows of P are input features
    e = np.zeros((1, 256), np.float32)
    e[0, 3] = 1.0
    assert (oracle.project(synth.f32_to_bf16_bits(e), synth.f32_to_bf16_bits(P))[0] == P[3]).all()


def test_kron_orthogonal_is_orthogonal():
    P = synth.kron_orthogonal_bf16(512).astype(np.float64)
    assert np.abs(P.T @ P - np.eye(512)).max() < 2e-2   # bf16 rounding only


def _rel_err(y, ref):
    return np.linalg.norm(y - ref) / np.linalg.norm(ref)


def test_config1_layer_error_and_snr_ordering():
    """The mixed layer is close to X·W, and closer than uniform INT4 with a random rotation only
    (the paper's SNR comparison of ResQ against rotation-only quantization)."""
    c = config1()
    pw = oracle.pack_weights(c.W_proj, c.r)
    res = oracle.linear(c.C_bits, None, pw)
    ref = c.X.astype(np.float64) @ c.W.astype(np.float64)
    e_resq = _rel_err(res.y32, ref)
    assert e_resq < 0.12
    # rotation-only INT4: whole row is one 4-bit segment in a Haar-rotated basis
    Q = basis.random_rotation(synth.gaussian_matrix(c.K, 91))
    Cq = (c.X.astype(np.float64) @ Q).astype(np.float32)
    Wq = basis.project_weights(Q, c.W)
    def q4rows(M):
        out = np.empty(M.shape, np.float64)
        for i, row in enumerate(M):
            s, codes = oracle.quantize_vector(row, 4)
            out[i] = codes.astype(np.float64) * float(s)
        return out
    e_rot = _rel_err(q4rows(Cq) @ q4rows(Wq).T, ref)
    assert e_resq < e_rot
    # codes stay inside the symmetric ranges
    assert np.abs(res.x8).max() <= 127 and np.abs(res.x4).max() <= 7
    assert np.abs(pw.q8).max() <= 127 and np.abs(pw.q4).max() <= 7


def test_quantization_error_bound_of_the_lemma():
    """Lemma A.1: E||R - Q(R)||_F <= sqrt(pi log size(R)) / (2^(n-1) - 1) · E||R||_F for Gaussian R."""
    for bits, n in ((4, 448), (8, 64)):
        ratios = []
        for seed in range(20):
            x = synth.normal(200 + seed, 0, n).astype(np.float32)
            s, codes = oracle.quantize_vector(x, bits)
            ratios.append(np.linalg.norm(x - codes * float(s)) / np.linalg.norm(x))
        assert np.mean(ratios) <= np.sqrt(np.pi * np.log(n)) / ((1 << (bits - 1)) - 1)
