"""Pins for the oracle's quantizer (Eq. 1), nibble packing and format helpers.

Nothing here calls the CUDA path.  Expected values come from exact rational arithmetic written
independently of the C code, from closed forms, or from a library routine (torch's bf16 cast).
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import synth


def fl32(q: Fraction) -> Fraction:
    """Round an exact rational to the nearest IEEE binary32 value (ties to even), as a Fraction.
    Independent of any float hardware path: scales to an integer significand and rounds there."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    q = abs(q)
    # exponent e with 2^e <= q < 2^(e+1)
    e = q.numerator.bit_length() - q.denominator.bit_length()
    if Fraction(2) ** e > q:
        e -= 1
    e = max(e, -126)                       # subnormal range keeps the 2^-149 grid
    ulp = Fraction(2) ** (e - 23)
    m = q / ulp
    n = m.numerator // m.denominator
    rem = m - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * ulp


def rne_int(q: Fraction) -> int:
    return round(q)  # Python rounds Fractions half to even


def expected_codes(vals, bits):
    """Eq. 1 symmetric with the stated precision: s = fl32(a / qmax), code = clip(rne(fl32(x / s)))."""
    qmax = (1 << (bits - 1)) - 1
    fr = [Fraction(float(v)) for v in vals]
    a = max(abs(f) for f in fr)
    s = fl32(a / qmax)
    if s == 0:
        return Fraction(0), [0] * len(fr)
    codes = [min(max(rne_int(fl32(f / s)), -qmax - 1), qmax) for f in fr]
    return s, codes


def _bf16_values_near(a, binades=12):
    bits_a = int(synth.f32_to_bf16_bits(np.array([a], np.float32))[0])
    lo = max(bits_a - binades * 128, 1)
    pos = synth.bf16_bits_to_f32(np.arange(lo, bits_a + 1, dtype=np.uint16))
    return np.concatenate([pos, -pos, np.zeros(1, np.float32)])


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("absmax", [1.0, 3.140625, 20.5, 0.00732421875, 127.0, 7.0, 1.9921875])
def test_quantizer_matches_exact_rational_evaluation(bits, absmax):
    vals = _bf16_values_near(absmax)
    s, codes = oracle.quantize_vector(vals, bits)
    s_exp, codes_exp = expected_codes(vals, bits)
    assert Fraction(float(s)) == s_exp
    assert codes.tolist() == codes_exp


@pytest.mark.parametrize("bits", [8, 4])
def test_quantizer_on_fp32_inputs_matches_exact_rational_evaluation(bits):
    # fp32 (not bf16-representable) inputs, as produced by the online projection
    x = (synth.normal(11, 0, 600) * 3.7).astype(np.float32)
    s, codes = oracle.quantize_vector(x, bits)
    s_exp, codes_exp = expected_codes(x, bits)
    assert Fraction(float(s)) == s_exp
    assert codes.tolist() == codes_exp


@pytest.mark.parametrize("bits,qmax", [(8, 127), (4, 7)])
def test_quantizer_closed_form_properties(bits, qmax):
    x = synth.activations(64, 512, "t4", seed=5).reshape(-1, 256)
    for row in x[:40]:
        s, codes = oracle.quantize_vector(row, bits)
        a = np.abs(row).max()
        assert s == np.float32(a) / np.float32(qmax)
        assert codes.min() >= -qmax and codes.max() <= qmax          # clip range never reached
        assert abs(int(codes[np.argmax(np.abs(row))])) == qmax       # the absmax element maps to +-qmax
        err = np.abs(row.astype(np.float64) - codes.astype(np.float64) * float(s))
        assert err.max() <= 0.5 * float(s) * (1 + 1e-6)              # nearest grid point
        # valid nearest integer of the exact ratio x*qmax/a
        exact = row.astype(np.float64) * qmax / float(a)
        assert np.abs(exact - codes).max() <= 0.5 + 1e-5


def test_quantizer_ties_go_to_even():
    # s = 7/7 = 1 exactly, so x/s = x and halves are exact ties
    x = np.array([7.0, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 6.5, -6.5], np.float32)
    s, codes = oracle.quantize_vector(x, 4)
    assert s == 1.0
    assert codes.tolist() == [7, 0, 2, 2, 4, 0, -2, -2, 6, -6]
    x8 = np.array([127.0, 0.5, 1.5, 2.5, 126.5, -126.5, -125.5], np.float32)
    s, codes = oracle.quantize_vector(x8, 8)
    assert s == 1.0
    assert codes.tolist() == [127, 0, 2, 2, 126, -126, -126]


def test_quantizer_zero_vector_and_negative_extreme():
    s, codes = oracle.quantize_vector(np.zeros(32, np.float32), 4)
    assert s == 0.0 and not codes.any()
    s, codes = oracle.quantize_vector(np.array([-3.0, 1.0, 0.0, 3.0], np.float32), 4)
    assert codes.tolist() == [-7, 2, 0, 7]     # 1/(3/7) = 2.333 -> 2; never -8


def test_quantizer_fp16_scale_is_the_stored_value():
    x = (synth.normal(3, 0, 512) * 0.02).astype(np.float32)
    for bits, qmax in ((8, 127), (4, 7)):
        s, codes = oracle.quantize_vector(x, bits, scale_fp16=True)
        s_full = np.float32(np.abs(x).max()) / np.float32(qmax)
        s_half = np.float32(torch.tensor(float(s_full)).to(torch.float16).item())
        assert s == s_half
        fr = [Fraction(float(v)) for v in x]
        exp = [min(max(rne_int(fl32(f / Fraction(float(s_half)))), -qmax - 1), qmax) for f in fr]
        assert codes.tolist() == exp


def test_split_quantize_is_two_independent_segments():
    C = synth.activations(8, 512, "t4", seed=9)
    q8, q4, s8, s4 = oracle.split_quantize(C, 64)
    for t in range(8):
        s, c = oracle.quantize_vector(C[t, :64], 8)
        assert s == s8[t] and (c == q8[t]).all()
        s, c = oracle.quantize_vector(C[t, 64:], 4)
        assert s == s4[t] and (c == q4[t]).all()
    # high-precision coefficients are the FIRST r of a row
    assert q8.shape == (8, 64) and q4.shape == (8, 448)


def test_nibble_layout_closed_form():
    codes = np.array([1, -1, -8, 7, 0, 3, -2, -3], np.int8)
    packed = oracle.pack_nibbles(codes)
    # element 2i in the low nibble, 2i+1 in the high nibble, two's complement
    assert packed.tolist() == [0xF1, 0x78, 0x30, 0xDE]
    assert oracle.unpack_nibbles(packed).tolist() == codes.tolist()
    allc = np.array([[a, b] for a in range(-8, 8) for b in range(-8, 8)], np.int8).ravel()
    assert (oracle.unpack_nibbles(oracle.pack_nibbles(allc)) == allc).all()


def test_bf16_conversion_matches_torch_cast():
    x = np.concatenate([
        (synth.normal(21, 0, 20000) * 10).astype(np.float32),
        np.array([1.00390625, 1.01171875, 1.0078125, -1.00390625, 3.0e38, 1e-40, 0.0], np.float32),  # ties
    ])
    ours = oracle.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (ours == ref).all()
    back = oracle.bf16_bits_to_f32(ours)
    ref_back = torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert (back == ref_back).all()
    # the input generator's converter agrees too (it feeds both sides)
    assert (synth.f32_to_bf16_bits(x) == ref).all()
