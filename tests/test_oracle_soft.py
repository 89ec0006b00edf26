"""Pins of the soft quantiser (Eq. 3-8) against its closed-form properties."""
import math

import numpy as np
import pytest

from oracle import soft

CASES = [(2, 0.0, 3.0), (3, -1.0, 2.5), (4, -0.1, 0.1), (4, 0.0, 6.0)]


def test_alpha_relations_at_the_papers_initial_value():
    # alpha = 0.2 (Sec. 4.1) => s = 1/(1-alpha) = 1.25 (Eq. 7),
    # k*Delta = log(2/alpha - 1) = ln 9 (Eq. 8), tanh(k*Delta/2) = 0.8 (Eq. 6)
    assert soft.s_from_alpha(0.2) == pytest.approx(1.25, abs=1e-15)
    for bits, lo, hi in CASES:
        k = soft.k_from_alpha(0.2, bits, lo, hi)
        assert k * soft.delta(bits, lo, hi) == pytest.approx(math.log(9.0),
                                                             rel=1e-14)
        assert soft.alpha_from_k(k, bits, lo, hi) == pytest.approx(0.2,
                                                                   rel=1e-13)


@pytest.mark.parametrize("alpha", [1e-3, 0.05, 0.2, 0.49])
def test_eq6_eq7_eq8_mutually_consistent(alpha):
    # s * tanh(0.5 k Delta) = 1 (Eq. 4) with s from Eq. 7 and k from Eq. 8
    for bits, lo, hi in CASES:
        k = soft.k_from_alpha(alpha, bits, lo, hi)
        d = soft.delta(bits, lo, hi)
        assert soft.s_from_alpha(alpha) * math.tanh(0.5 * k * d) == \
            pytest.approx(1.0, rel=1e-13)


@pytest.mark.parametrize("bits,lo,hi", CASES)
@pytest.mark.parametrize("alpha", [0.01, 0.2, 0.49])
def test_hits_interval_endpoints_and_midpoints(bits, lo, hi, alpha):
    d = soft.delta(bits, lo, hi)
    n = 2 ** bits - 1
    ends = lo + d * np.arange(n + 1)
    # phi = -1 / +1 at the two ends of an interval => Q_S(l + i*Delta) is the
    # level itself, from either side
    assert np.allclose(soft.q_soft(ends, bits, lo, hi, alpha), ends,
                       rtol=0, atol=1e-12 * max(1, abs(hi)))
    eps = d * 1e-9
    left = soft.q_soft(ends[1:-1] - eps, bits, lo, hi, alpha)
    right = soft.q_soft(ends[1:-1] + eps, bits, lo, hi, alpha)
    assert np.allclose(left, right, atol=d * 1e-6)      # continuity at joins
    mids = lo + d * (np.arange(n) + 0.5)
    assert np.allclose(soft.q_soft(mids, bits, lo, hi, alpha), mids,
                       atol=1e-12 * max(1, abs(hi)))     # phi(m_i) = 0
    # clipping branches of Eq. 5
    assert soft.q_soft(lo - 1.0, bits, lo, hi, alpha) == lo
    assert soft.q_soft(hi + 1.0, bits, lo, hi, alpha) == hi


@pytest.mark.parametrize("bits,lo,hi", CASES)
def test_slope_matches_across_interval_joins(bits, lo, hi):
    # continuously differentiable (Sec. 3.2): one-sided slopes agree at a join
    alpha = 0.2
    d = soft.delta(bits, lo, hi)
    h = d * 1e-6
    for i in range(1, 2 ** bits - 1):
        x0 = lo + i * d
        f = lambda x: float(soft.q_soft(x, bits, lo, hi, alpha))
        sl = (f(x0) - f(x0 - h)) / h
        sr = (f(x0 + h) - f(x0)) / h
        assert sl == pytest.approx(sr, rel=1e-3)


@pytest.mark.parametrize("bits,lo,hi", CASES)
def test_converges_to_hard_rounding_as_alpha_goes_to_zero(bits, lo, hi):
    rng = np.random.default_rng(5)
    x = rng.uniform(lo - 0.1 * (hi - lo), hi + 0.1 * (hi - lo), 4000)
    d = soft.delta(bits, lo, hi)
    t = (np.clip(x, lo, hi) - lo) / d
    # k*Delta grows only like log(1/alpha): look a quarter interval away from
    # the midpoints, where the error is Delta/2 * (1 - tanh(k*Delta/4))
    off_mid = np.abs(t - np.floor(t) - 0.5) > 0.25
    hard = soft.q_uniform(x, bits, lo, hi)
    prev = None
    for alpha in [0.4, 0.1, 1e-2, 1e-4, 1e-8, 1e-12]:
        err = np.max(np.abs(soft.q_soft(x, bits, lo, hi, alpha) - hard)[off_mid])
        if prev is not None:
            assert err < prev
        prev = err
    assert prev < d * 1e-3
    # and it is monotone non-decreasing in x for any alpha
    xs = np.sort(x)
    assert np.all(np.diff(soft.q_soft(xs, bits, lo, hi, 0.2)) >= -1e-15)
