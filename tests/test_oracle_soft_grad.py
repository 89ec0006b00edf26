"""Pins of the soft quantiser's analytic gradients (Eq. 10-13) by central
finite differences of the forward function Q_S (oracle/soft.py, itself pinned
by its closed-form properties), in float64, away from interval boundaries."""
import numpy as np
import pytest

from oracle import soft, soft_grad

CASES = [(1, -1.0, 1.0), (2, 0.0, 3.0), (3, -1.0, 2.5), (4, -0.1, 0.1), (4, 0.0, 6.0)]


def sample_points(bits, lo, hi, rng, n=400):
    """Points inside the clip range and not within 2 % of an interval boundary
    (where the interval index, hence one-sided derivatives, changes), plus
    points outside the range."""
    d = soft.delta(bits, lo, hi)
    x = rng.uniform(lo, hi, n)
    frac = (x - lo) / d
    frac = frac - np.floor(frac)
    x = x[(frac > 0.02) & (frac < 0.98)]
    outside = np.concatenate([lo - rng.uniform(0.01, 2, 20) * (hi - lo),
                              hi + rng.uniform(0.01, 2, 20) * (hi - lo)])
    return np.concatenate([x, outside])


@pytest.mark.parametrize("bits,lo,hi", CASES)
@pytest.mark.parametrize("alpha", [0.05, 0.2, 0.45])
def test_partials_against_central_differences(bits, lo, hi, alpha):
    rng = np.random.default_rng(bits * 100 + int(alpha * 100))
    x = sample_points(bits, lo, hi, rng)
    dx, da, dl, du = soft_grad.partials(x, bits, lo, hi, alpha)
    scale = hi - lo
    h = 1e-6 * scale
    fx = (soft.q_soft(x + h, bits, lo, hi, alpha) - soft.q_soft(x - h, bits, lo, hi, alpha)) / (2 * h)
    inside = (x > lo + 2 * h) & (x < hi - 2 * h)
    assert np.allclose(dx[inside], fx[inside], rtol=1e-6, atol=1e-7)
    assert np.all(dx[~inside & ((x < lo) | (x > hi))] == 0.0)
    ha = 1e-7
    fa = (soft.q_soft(x, bits, lo, hi, alpha + ha) - soft.q_soft(x, bits, lo, hi, alpha - ha)) / (2 * ha)
    assert np.allclose(da, fa, rtol=1e-5, atol=1e-8 * scale)
    fl = (soft.q_soft(x, bits, lo + h, hi, alpha) - soft.q_soft(x, bits, lo - h, hi, alpha)) / (2 * h)
    fu = (soft.q_soft(x, bits, lo, hi + h, alpha) - soft.q_soft(x, bits, lo, hi - h, alpha)) / (2 * h)
    assert np.allclose(dl, fl, rtol=1e-5, atol=1e-6)
    assert np.allclose(du, fu, rtol=1e-5, atol=1e-6)


def test_clipped_points_feed_only_their_bound():
    # Eq. 11-12: x < l contributes 1 to dl and 0 to du; x > u the other way
    dx, da, dl, du = soft_grad.partials(np.array([-5.0, 9.0]), 3, -1.0, 2.5, 0.2)
    assert list(dx) == [0.0, 0.0] and list(da) == [0.0, 0.0]
    assert list(dl) == [1.0, 0.0] and list(du) == [0.0, 1.0]


def test_value_at_an_interval_midpoint():
    # at x = m_i: tanh = 0, so dQ/dx = (Delta/2) s k, dQ/dalpha = 0 and
    # dQ/dl + dQ/du = 1 (shifting both bounds by c shifts Q_S(x + c) by c; at
    # the midpoint the x-term is (Delta/2) s k which the l, u terms cancel)
    bits, lo, hi, alpha = 2, 0.0, 3.0, 0.2
    d = soft.delta(bits, lo, hi)
    x = np.array([lo + 1.5 * d])
    dx, da, dl, du = soft_grad.partials(x, bits, lo, hi, alpha)
    s, k = 1.25, np.log(9.0) / d
    assert dx[0] == pytest.approx(0.5 * d * s * k, rel=1e-12)
    assert da[0] == pytest.approx(0.0, abs=1e-15)
    assert dx[0] + dl[0] + du[0] == pytest.approx(1.0, rel=1e-12)


@pytest.mark.parametrize("bits,lo,hi", CASES)
def test_translation_and_scale_identities(bits, lo, hi):
    """Q_S(x + c; l + c, u + c) = Q_S(x; l, u) + c  =>  dx + dl + du = 1, and
    Q_S(t x; t l, t u) = t Q_S(x; l, u)  =>  x dx + l dl + u du = Q_S, for
    every x inside the range and every alpha."""
    rng = np.random.default_rng(7)
    x = rng.uniform(lo, hi, 300)
    for alpha in (0.02, 0.2, 0.49):
        dx, da, dl, du = soft_grad.partials(x, bits, lo, hi, alpha)
        assert np.allclose(dx + dl + du, 1.0, rtol=1e-10, atol=1e-12)
        assert np.allclose(x * dx + lo * dl + hi * du, soft.q_soft(x, bits, lo, hi, alpha),
                           rtol=1e-10, atol=1e-12)


def test_backward_sums():
    rng = np.random.default_rng(3)
    x = rng.normal(0.5, 1.5, 1000)
    g = rng.normal(0, 1, 1000)
    gx, gp = soft_grad.backward(x, g, 3, -1.0, 2.5, 0.2)
    dx, da, dl, du = soft_grad.partials(x, 3, -1.0, 2.5, 0.2)
    assert np.array_equal(gx, g * dx)
    assert gp[0] == pytest.approx(float(np.dot(g, da)), rel=1e-12)
    assert gp[1] == pytest.approx(float(np.dot(g, dl)), rel=1e-12)
    assert gp[2] == pytest.approx(float(np.dot(g, du)), rel=1e-12)
