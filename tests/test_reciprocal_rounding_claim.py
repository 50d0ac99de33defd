"""Host-side checks of the claims the fast quantizer kernels rest on.

Symmetric quantizer: the kernel replaces code = rint(fl(x / s)) (the definition, Eq. 1 with round-half-even and
an IEEE fp32 division) by the rounding of two exact products, x * v_lo and x * v_hi with
v_lo = RN(inv (1 - 2^-20)), v_hi = RN(inv (1 + 2^-20)), inv = RN(1 / s), and falls back to the division whenever
the two roundings differ.  Claim: whenever they agree, they are the defined code, for every |x / s| <= 128.
Asymmetric quantizer: rint(d * inv) evaluated exactly, with a fallback whenever the product comes within 2^-14
of a half-integer.  Both are checked here with exact rationals on random and on adversarial near-tie inputs; the
defined values come from the oracle's quantizers.
"""
from fractions import Fraction

import numpy as np

import oracle

GUARD = Fraction(1, 2) - Fraction(1, 2 ** 15)


def _rint_half_even(q: Fraction) -> int:
    f = q.numerator // q.denominator
    rem = q - f
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and f % 2):
        return f + 1
    return f


def _f32(q: Fraction) -> np.float32:
    """Rounds an exact rational that a double holds exactly (at most 53 significant bits) to fp32 once."""
    d = float(q)
    assert Fraction(d) == q
    return np.float32(d)


def test_bracketing_products_agree_only_on_the_defined_code():
    rng = np.random.default_rng(3)
    checked = fallbacks = 0
    for qmax in (127, 7):
        for _ in range(40):
            a = np.float32(np.exp(rng.uniform(-20, 20)))
            s = np.float32(a / np.float32(qmax))
            inv = np.float32(np.float32(1.0) / s)  # numpy's fp32 division is correctly rounded
            v_lo = _f32(Fraction(float(inv)) * (1 - Fraction(1, 2 ** 20)))   # fma(inv, -2^-20, inv): one rounding
            v_hi = _f32(Fraction(float(inv)) * (1 + Fraction(1, 2 ** 20)))
            k = rng.integers(-qmax, qmax, 200).astype(np.float32) + np.float32(0.5)
            near = ((k * s).astype(np.float32).view(np.int32) + rng.integers(-4, 5, 200).astype(np.int32)).view(np.float32)
            rand = (rng.uniform(-1, 1, 200) * a).astype(np.float32)
            x = np.concatenate([near, rand, [a, -a]]).astype(np.float32)
            x = x[np.abs(x) <= a]
            # the definition, through the oracle: one row whose absmax is a
            row = np.concatenate([[a], x]).astype(np.float32)
            s_o, codes = oracle.quantize_vector(row, 8 if qmax == 127 else 4)
            assert s_o == s
            codes = codes[1:]
            for xv, code in zip(x, codes):
                n_lo = _rint_half_even(Fraction(float(xv)) * Fraction(float(v_lo)))
                n_hi = _rint_half_even(Fraction(float(xv)) * Fraction(float(v_hi)))
                if n_lo == n_hi:
                    assert n_lo == int(code), (float(xv), float(s), n_lo, int(code))
                    checked += 1
                else:
                    fallbacks += 1
    assert checked > 10000 and fallbacks > 1000  # both branches were exercised


def test_asymmetric_product_rounding_agrees_outside_guard_band():
    """Same claim for the asymmetric quantizer: d = fl(x - z), code = rint(fl(d / s)) against
    rint(d * RN(1 / s)); quotients reach 255, so the guard band is 2^-14."""
    guard = Fraction(1, 2) - Fraction(1, 2 ** 14)
    rng = np.random.default_rng(4)
    checked = fallbacks = 0
    for bits, qmax in ((8, 255), (4, 15)):
        for _ in range(40):
            lo = np.float32(rng.uniform(-10, 10))
            rng_w = np.float32(np.exp(rng.uniform(-12, 12)))
            hi = np.float32(lo + rng_w)
            s = np.float32(np.float32(hi - lo) / np.float32(qmax))
            inv = np.float32(np.float32(1.0) / s)
            k = rng.integers(0, qmax, 200).astype(np.float32) + np.float32(0.5)
            near = (np.float32(lo) + (k * s).astype(np.float32)).astype(np.float32)
            near = (near.view(np.int32) + rng.integers(-4, 5, 200).astype(np.int32)).view(np.float32)
            x = np.concatenate([near, rng.uniform(lo, hi, 200).astype(np.float32)])
            x = x[(x >= lo) & (x <= hi)]
            row = np.concatenate([[lo, hi], x]).astype(np.float32)
            pad = np.tile(row, 2)[None, :]                      # both segments hold the same data
            out = oracle.split_quantize_asym(pad, row.size)
            codes = out[0 if bits == 8 else 1][0, 2:]
            assert out[2 if bits == 8 else 3][0] == s and out[4 if bits == 8 else 5][0] == lo
            for xv, code in zip(x, codes):
                d = np.float32(xv - lo)
                p = Fraction(float(d)) * Fraction(float(inv))
                n = _rint_half_even(p)
                if abs(p - n) < guard:
                    assert n == int(code), (float(xv), float(s), n, int(code))
                    checked += 1
                else:
                    fallbacks += 1
    assert checked > 10000 and fallbacks > 500
