"""Pins of the oracle's quantisers against what the paper and arithmetic fix
(Eq. 1-8, Algorithm 1 steps 1-4): closed forms, exact rational arithmetic,
special cases.  No GPU."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import native, soft

RANGES = [(0.0, 2.0), (0.0, 6.0), (-0.1, 0.1), (-1.75, 3.25), (0.0, 15.0)]
BITS = [2, 3, 4]


def exact_code(x, bits, lo, hi):
    """floor((clip(x) - l)/Delta + 1/2) in exact rational arithmetic on the
    binary32 values of x, l, u."""
    X, L, U = (Fraction(float(np.float32(v))) for v in (x, lo, hi))
    xc = min(max(X, L), U)
    t = (xc - L) * (2 ** bits - 1) / (U - L) + Fraction(1, 2)
    return min(math.floor(t), 2 ** bits - 1), t


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("lo,hi", RANGES)
def test_endpoints_and_idempotence(bits, lo, hi):
    qmax = 2 ** bits - 1
    assert native.quantize_code(lo, bits, lo, hi) == 0
    assert native.quantize_code(hi, bits, lo, hi) == qmax
    assert native.quantize_code(lo - 10.0, bits, lo, hi) == 0
    assert native.quantize_code(hi + 10.0, bits, lo, hi) == qmax
    # quantise(dequantise(q)) == q for every code (levels l + q*Delta)
    d = (np.float32(hi) - np.float32(lo)) / np.float32(qmax)
    for q in range(qmax + 1):
        level = np.float32(lo) + np.float32(q) * d
        assert native.quantize_code(float(level), bits, lo, hi) == q
    codes = np.arange(qmax + 1, dtype=np.int8)
    back = native.quantize(native.dequantize(codes, bits, lo, hi), bits, lo, hi)
    assert np.array_equal(back, codes)


def test_midpoint_takes_upper_code():
    # sgn(0) = +1 (Eq. 1) composed with phi: a midpoint goes up.  Delta = 1 so
    # the midpoints are exact in binary32.
    assert native.quantize_code(0.5, 4, 0.0, 15.0) == 1
    assert native.quantize_code(2.5, 4, 0.0, 15.0) == 3     # half-even -> 2
    assert native.quantize_code(1.5, 2, 0.0, 3.0) == 2
    # negative side: levels -7.5 + q, midpoint -1.0 lies between q=6 and q=7;
    # half-away-from-zero would pick q=6.
    assert native.quantize_code(-1.0, 4, -7.5, 7.5) == 7
    assert native.quantize_code(-2.0, 3, -3.5, 3.5) == 2
    # just below a midpoint goes down
    assert native.quantize_code(float(np.nextafter(np.float32(2.5), np.float32(0))),
                                4, 0.0, 15.0) == 2


def test_nonfinite_inputs():
    for bits in BITS:
        qmax = 2 ** bits - 1
        assert native.quantize_code(float("nan"), bits, 0.0, 2.0) == 0
        assert native.quantize_code(float("inf"), bits, 0.0, 2.0) == qmax
        assert native.quantize_code(float("-inf"), bits, 0.0, 2.0) == 0


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("lo,hi", RANGES)
def test_monotone_and_matches_exact_rational(bits, lo, hi):
    rng = np.random.default_rng(7)
    span = hi - lo
    x = np.sort(rng.uniform(lo - 0.2 * span, hi + 0.2 * span, 20000)
                .astype(np.float32))
    q = native.quantize(x, bits, lo, hi).astype(np.int64)
    assert np.all(np.diff(q) >= 0)
    assert q.min() == 0 and q.max() == 2 ** bits - 1
    bad = 0
    for xi, qi in zip(x[::7], q[::7]):
        qe, t = exact_code(xi, bits, lo, hi)
        if qe != qi:
            # binary32 rounding may only matter within a hair of a midpoint
            frac = t - math.floor(t)
            assert min(frac, 1 - frac) < Fraction(1, 2 ** 18), (xi, qi, qe)
            assert abs(qe - qi) == 1
            bad += 1
    assert bad <= 3


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("alpha", [0.01, 0.2, 0.49])
def test_hard_quantiser_is_sgn_of_phi(bits, alpha):
    # "DSQ + sign" is the uniform quantiser for every alpha (Sec. 3.2, Fig. 3b)
    lo, hi = -0.4, 1.1
    rng = np.random.default_rng(11)
    x = rng.uniform(lo - 0.3, hi + 0.3, 5000).astype(np.float32)
    d = soft.delta(bits, lo, hi)
    t = (np.clip(x.astype(np.float64), lo, hi) - lo) / d
    off_mid = np.abs(t - np.floor(t) - 0.5) > 1e-4
    q_def = soft.code_via_sgn_phi(x, bits, lo, hi, alpha)
    q_nat = native.quantize(x, bits, lo, hi).astype(np.int64)
    assert np.array_equal(q_def[off_mid], q_nat[off_mid])
    # and at an exact midpoint sgn(0) = +1 gives the upper code
    assert soft.code_via_sgn_phi(np.array([2.5]), 4, 0.0, 15.0, alpha)[0] == 3


def test_signed_weight_storage():
    # c = q - 2^(b-1): range [-2^(b-1), 2^(b-1)-1]; symmetric clip puts the
    # grid at Delta*(c + 1/2)
    for bits in BITS:
        half = 2 ** (bits - 1)
        w = np.array([[-1.0, -0.1, 0.0, 0.1, 1.0]], np.float32)
        c = native.quantize_weights(w, bits, -0.1, 0.1)
        assert c[0, 0] == -half and c[0, 1] == -half
        assert c[0, 3] == half - 1 and c[0, 4] == half - 1
        assert c[0, 2] == 0     # 0 is the midpoint of the middle interval: up
    w = np.array([[0.05, 0.05], [0.05, 0.05]], np.float32)
    c = native.quantize_weights(w, 4, np.array([-0.1, -1.0], np.float32),
                                np.array([0.1, 1.0], np.float32), per_row=True)
    # row 0: (0.05+0.1)/0.2*15 + 1/2 = 11.75 -> q=11, c=3
    # row 1: (0.05+1)/2*15 + 1/2 = 8.375 -> q=8, c=0
    assert c[0, 0] == 3 and c[1, 0] == 0
