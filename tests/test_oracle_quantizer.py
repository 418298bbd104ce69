"""Pins for the oracle's scalar quantiser.

Nothing here re-types the oracle's C expression: expected values are worked by
hand, or come from exact rational arithmetic (fractions.Fraction) with an
explicit round-to-nearest-even to binary32, or are closed-form invariants of a
symmetric uniform quantiser with a min-max range (paper Section 4.1 and
Appendix A "Prior QAT Techniques on DLRM").
"""
from fractions import Fraction

import numpy as np
import pytest


# ---------------------------------------------------------------------------
# exact helpers (independent of the oracle)
# ---------------------------------------------------------------------------
def round_to_f32(fr: Fraction) -> Fraction:
    """Exact value of the binary32 nearest to `fr` (ties to even); normal range only."""
    if fr == 0:
        return Fraction(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    assert -126 <= e <= 127
    ulp = Fraction(2) ** (e - 23)
    k = a / ulp                      # in [2^23, 2^24)
    fl = k.numerator // k.denominator
    rem = k - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * fl * ulp


def rint_half_even(fr: Fraction) -> int:
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return int(fl)


def exact_quantize(x: np.float32, s: np.float32, bits: int) -> int:
    quo = round_to_f32(Fraction(float(x)) / Fraction(float(s)))   # one FP32 divide
    q = rint_half_even(quo)
    return max(-(2 ** (bits - 1)), min(2 ** (bits - 1) - 1, q))


# ---------------------------------------------------------------------------
# hand-worked cases
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("x,s,bits,want", [
    (0.5, 1.0, 8, 0), (1.5, 1.0, 8, 2), (2.5, 1.0, 8, 2), (3.5, 1.0, 8, 4),
    (-0.5, 1.0, 8, 0), (-1.5, 1.0, 8, -2), (-2.5, 1.0, 8, -2), (0.75, 1.0, 8, 1),
    (0.49, 1.0, 8, 0), (0.51, 1.0, 8, 1), (3.0, 0.5, 8, 6), (-3.0, 0.5, 8, -6),
    (100.0, 1.0, 4, 7), (-100.0, 1.0, 4, -8), (7.0, 1.0, 4, 7), (-8.0, 1.0, 4, -8),
    (7.49, 1.0, 4, 7), (-8.6, 1.0, 4, -8),
    (5.0, 1.0, 2, 1), (-5.0, 1.0, 2, -2), (1.0, 1.0, 2, 1), (-1.0, 1.0, 2, -1), (-2.0, 1.0, 2, -2),
    (127.0, 1.0, 8, 127), (128.0, 1.0, 8, 127), (-128.0, 1.0, 8, -128), (-129.0, 1.0, 8, -128),
    (40000.0, 1.0, 16, 32767), (-40000.0, 1.0, 16, -32768), (1234.0, 1.0, 16, 1234),
    (1e30, 1e-8, 4, 7), (-1e30, 1e-8, 4, -8),
])
def test_hand_cases(oracle, x, s, bits, want):
    assert oracle.quantize(x, s, bits) == want


@pytest.mark.parametrize("a,bits,want", [
    (7.0, 4, 1.0), (14.0, 4, 2.0), (127.0, 8, 1.0), (63.5, 8, 0.5), (1.0, 2, 1.0),
    (32767.0, 16, 1.0), (3.0, 3, 1.0),
])
def test_scale_hand_cases(oracle, a, bits, want):
    assert oracle.scale_from_absmax(a, bits) == np.float32(want)


def test_scale_floor_for_all_zero_tensor(oracle):
    # abs-max is floored at 1e-8 before the divide
    for bits in (2, 4, 8, 16):
        n = 2 ** (bits - 1) - 1
        want = round_to_f32(Fraction(float(np.float32(1e-8))) / n)
        got = oracle.scale_from_absmax(0.0, bits)
        assert Fraction(float(got)) == want
        assert oracle.quantize(0.0, got, bits) == 0
    assert oracle.scale_from_absmax(1e-12, 4) == oracle.scale_from_absmax(0.0, 4)


def test_scale_is_one_fp32_divide(oracle):
    rng = np.random.default_rng(1)
    for a in np.abs(rng.standard_normal(200)).astype(np.float32):
        for bits in (2, 3, 4, 8, 16):
            want = round_to_f32(Fraction(float(a)) / (2 ** (bits - 1) - 1))
            assert Fraction(float(oracle.scale_from_absmax(a, bits))) == want


def test_dequantize_is_one_fp32_multiply(oracle):
    rng = np.random.default_rng(2)
    for s in np.abs(rng.standard_normal(100)).astype(np.float32) + np.float32(1e-3):
        for q in (-128, -77, -8, -1, 0, 1, 3, 7, 100, 127, 32767, -32768):
            want = round_to_f32(Fraction(float(s)) * q)
            assert Fraction(float(oracle.dequantize(q, s))) == want


# ---------------------------------------------------------------------------
# exact rational cross-check, including exact ties
# ---------------------------------------------------------------------------
def test_against_exact_rational(oracle):
    rng = np.random.default_rng(3)
    n = 4000
    xs = (rng.standard_normal(n) * 0.05).astype(np.float32)
    ss = (np.abs(rng.standard_normal(n)) * 0.01 + 1e-4).astype(np.float32)
    for x, s in zip(xs, ss):
        for bits in (2, 4, 8):
            assert oracle.quantize(x, s, bits) == exact_quantize(x, s, bits), (x, s, bits)


def test_ties_round_to_even(oracle):
    # s a power of two makes x = (k + 0.5) * s an exact tie
    for e in (-10, -3, 0, 2):
        s = np.float32(2.0 ** e)
        for k in range(-130, 130):
            x = np.float32((k + 0.5) * float(s))
            want_unclamped = k if k % 2 == 0 else k + 1
            want = max(-128, min(127, want_unclamped))
            assert oracle.quantize(x, s, 8) == want
            assert oracle.quantize(x, s, 8) == exact_quantize(x, s, 8)


def test_near_ties_against_exact_rational(oracle):
    rng = np.random.default_rng(4)
    for _ in range(2000):
        s = np.float32(abs(rng.standard_normal()) * 0.01 + 1e-4)
        k = int(rng.integers(-7, 7))
        x = np.float32((k + 0.5) * float(s))
        for dx in (0, 1, -1, 2, -2):
            xi = (x.view(np.int32) + np.int32(dx)).view(np.float32)
            assert oracle.quantize(xi, s, 4) == exact_quantize(xi, s, 4)


# ---------------------------------------------------------------------------
# closed-form invariants
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16])
def test_invariants(oracle, bits):
    rng = np.random.default_rng(10 + bits)
    n = 2 ** (bits - 1) - 1
    xs = (rng.standard_normal(3000) * 0.03).astype(np.float32)
    absmax = np.float32(np.abs(xs).max())
    s = oracle.scale_from_absmax(absmax, bits)
    # fresh scale: the extreme maps to +-n exactly, nothing reaches -2^(b-1)
    assert oracle.quantize(absmax, s, bits) == n
    assert oracle.quantize(-absmax, s, bits) == -n
    order = np.argsort(xs, kind="stable")
    prev_q = None
    for x in xs[order]:
        q = oracle.quantize(x, s, bits)
        assert -(2 ** (bits - 1)) <= q <= n
        assert -n <= q                       # fresh scale
        fq = oracle.fake_quant(x, s, bits)
        # |x - FQ(x)| <= s/2 (+ rounding of the divide and the multiply)
        tol = float(s) / 2 + 2 * float(np.spacing(np.float32(abs(x)))) + 1e-12
        assert abs(float(x) - float(fq)) <= tol
        # idempotent, bit for bit, at a fixed scale
        assert oracle.fake_quant(fq, s, bits).tobytes() == fq.tobytes()
        assert oracle.quantize(fq, s, bits) == q
        # odd
        assert oracle.quantize(-x, s, bits) == -q
        # monotone
        if prev_q is not None:
            assert q >= prev_q
        prev_q = q


def test_stale_scale_clamps(oracle):
    # with a scale that is too small for the data the clamp is live, and it is asymmetric
    s = np.float32(0.01)
    assert oracle.quantize(1.0, s, 4) == 7
    assert oracle.quantize(-1.0, s, 4) == -8
    assert oracle.fake_quant(1.0, s, 4) == np.float32(7) * s
    assert oracle.fake_quant(-1.0, s, 4) == np.float32(-8) * s
