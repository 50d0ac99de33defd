"""Pins of the oracle's asymmetric-activation path (Eq. 1, second form; Section 5.1) against what the
paper and arithmetic fix: closed forms of the quantizer, an exact-rational restatement of its
rounding, the constant-segment case, brute-force dequantized products on a tiny layer (which is what
catches a dropped or mis-signed zero-point term), and the reduction to the symmetric layer when the
zero-points vanish."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import synth


def _rint_half_even(q: Fraction) -> int:
    f = q.numerator // q.denominator
    rem = q - f
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and f % 2):
        return f + 1
    return f


@pytest.mark.parametrize("bits,col", [(8, 0), (4, 1)])
def test_closed_forms(bits, col):
    rng = np.random.default_rng(bits)
    r = 64
    C = (rng.standard_normal((50, 128)) * np.exp(rng.uniform(-3, 3, (50, 1))) + rng.uniform(-5, 5, (50, 1))).astype(np.float32)
    out = oracle.split_quantize_asym(C, r)
    codes, s, z = out[col].astype(np.int64), out[2 + col], out[4 + col]
    seg = C[:, :r] if col == 0 else C[:, r:]
    qmax = 2 ** bits - 1
    assert codes.min() >= 0 and codes.max() <= qmax
    assert (z == seg.min(axis=1)).all()                                   # zero-point = min (Eq. 1)
    assert (s == ((seg.max(axis=1) - seg.min(axis=1)) / np.float32(qmax)).astype(np.float32)).all()
    rows = np.arange(seg.shape[0])
    assert (codes[rows, seg.argmin(axis=1)] == 0).all()                   # the minimum maps to code 0 ...
    assert (codes[rows, seg.argmax(axis=1)] == qmax).all()                # ... the maximum to 2^N - 1
    deq = codes * s[:, None].astype(np.float64) + z[:, None].astype(np.float64)
    assert (np.abs(deq - seg) <= 0.5 * s[:, None] * (1 + 1e-5) + 1e-30).all()  # round to nearest


def test_rounding_matches_exact_rationals():
    """code = round-half-even(fl(fl(x - z) / s)): the two fp32 roundings restated with numpy's correctly
    rounded fp32 operations, the final rounding with exact rationals; the data include exact .5 ties
    (s = 0.25, z = 0 by construction), which must land on even codes."""
    rng = np.random.default_rng(7)
    for bits, col in ((8, 0), (4, 1)):
        qmax = 2 ** bits - 1
        x = np.clip(rng.standard_normal(400), 0.0, 0.25 * qmax).astype(np.float32)
        ties = (np.arange(qmax // 2, dtype=np.float32)[:40] + np.float32(0.5)) * np.float32(0.25)
        x[2:2 + ties.size] = ties
        x[0], x[1] = np.float32(0.0), np.float32(0.25 * qmax)
        row = np.concatenate([x, x])[None, :]            # both segments hold the same data
        out = oracle.split_quantize_asym(row, x.size)
        codes, s, z = out[col][0], out[2 + col][0], out[4 + col][0]
        assert s == np.float32(0.25) and z == np.float32(0.0)
        q = ((x - z).astype(np.float32) / s).astype(np.float32)
        want = [min(max(_rint_half_even(Fraction(float(v))), 0), qmax) for v in q]
        assert codes.tolist() == want
        assert all(c % 2 == 0 for c in codes[2:2 + ties.size].tolist())


def test_constant_segment():
    C = np.full((2, 64), 3.25, np.float32)
    C[1, 32:] = np.linspace(-1, 1, 32, dtype=np.float32)
    u8, u4, s8, s4, z8, z4 = oracle.split_quantize_asym(C, 32)
    assert (u8 == 0).all() and (s8 == 0).all() and (z8 == np.float32(3.25)).all()
    assert (u4[0] == 0).all() and s4[0] == 0 and z4[0] == np.float32(3.25)
    assert s4[1] > 0


def test_dequantized_product_brute_force():
    """Tiny layer: dequantize activations (code*s + z) and weights (code*s) to fp64, multiply them out,
    and compare with the integer-product + row-sum form the oracle (and the kernels) use."""
    rng = np.random.default_rng(3)
    T, K, N, r = 3, 16, 4, 2
    C = (rng.standard_normal((T, K)) + 1.5).astype(np.float32)      # offset so that the zero-points matter
    Wp = rng.standard_normal((N, K)).astype(np.float32)
    pw = oracle.pack_weights(Wp, r)
    res = oracle.linear_asym_from_coeff(C, pw)
    x8 = res.u8.astype(np.float64) * res.s_x8[:, None] + res.z_x8[:, None]
    x4 = res.u4.astype(np.float64) * res.s_x4[:, None] + res.z_x4[:, None]
    w8 = pw.q8.astype(np.float64) * pw.s8[:, None]
    w4 = pw.q4.astype(np.float64) * pw.s4[:, None]
    y = x8 @ w8.T + x4 @ w4.T
    assert np.abs(res.y32 - y).max() <= 1e-6 * np.abs(y).max()
    assert np.abs(res.z_x8).min() > 0 and np.abs(res.z_x4).min() > 0   # the rank-one terms were exercised
    # and the quantized layer approximates the unquantized one (a sign error in a z term would not)
    exact = C.astype(np.float64) @ Wp.astype(np.float64).T
    assert np.abs(y - exact).max() < 0.5 * np.abs(exact).max()


def test_python_int_product_and_row_sums():
    rng = np.random.default_rng(5)
    u = rng.integers(0, 256, (4, 33)).astype(np.uint8)
    w = rng.integers(-128, 128, (5, 33)).astype(np.int8)
    acc = oracle.int_gemm_u8(u, w)
    for t in range(4):
        for n in range(5):
            assert int(acc[t, n]) == sum(int(a) * int(b) for a, b in zip(u[t], w[n]))
    assert oracle.weight_row_sums(w).tolist() == [sum(int(b) for b in row) for row in w]


def test_nibble_layout_unsigned():
    u = np.array([[0, 15, 7, 8, 1, 2]], np.uint8)
    assert oracle.pack_nibbles_u(u).tolist() == [[0xF0, 0x87, 0x21]]


def test_asymmetric_beats_symmetric_on_shifted_activations():
    """Why the paper's experiments use the asymmetric form: on coefficients with a per-token offset it
    spends no codes on the empty half of the range."""
    rng = np.random.default_rng(11)
    T, K, N, r = 32, 256, 64, 32
    C = (rng.standard_normal((T, K)) + 3.0).astype(np.float32)
    Wp = (rng.standard_normal((N, K)) / 16).astype(np.float32)
    pw = oracle.pack_weights(Wp, r)
    exact = C.astype(np.float64) @ Wp.astype(np.float64).T
    e_asym = np.linalg.norm(oracle.linear_asym_from_coeff(C, pw).y32 - exact)
    e_sym = np.linalg.norm(oracle.linear_from_coeff(C, pw).y32 - exact)
    assert e_asym < e_sym


def test_empty_high_precision_segment():
    """r = 0 (uniform 4-bit): the INT8 segment is empty, its scale and zero-point are 0 and it adds nothing."""
    rng = np.random.default_rng(9)
    C = (rng.standard_normal((3, 64)) + 2.0).astype(np.float32)
    u8, u4, s8, s4, z8, z4 = oracle.split_quantize_asym(C, 0)
    assert u8.shape == (3, 0) and (s8 == 0).all() and (z8 == 0).all() and (s4 > 0).all()
    pw = oracle.pack_weights(rng.standard_normal((8, 64)).astype(np.float32), 0)
    res = oracle.linear_asym_from_coeff(C, pw)
    assert np.isfinite(res.y32).all() and (res.acc8 == 0).all()
