"""GPU parity of the training-side kernels: DSQ's soft quantiser Q_S (Eq. 5)
and its back-propagation (Eq. 10-13) against the float64 oracle.

The kernels compute in binary32.  Tolerance (derived from the arithmetic): the
argument z = k (x - m_i) of tanh carries an absolute error of about
k * eps * max(|l|, |u|) (eps = 2^-23: rounding of m_i and of the difference), which
the slope (Delta/2) s of Q_S in z turns into an error of the output; on top come a
few roundings of the result itself.  So
    |y - y_ref| <= 4 eps max(|l|,|u|) (1 + (Delta/2) s k)
and the gradients, which are smooth functions of the same z, agree to a relative
1e-4 plus the same absolute floor scaled by their magnitude."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import soft, soft_grad
from gpu_util import T, N

EPS = 2.0 ** -23
CASES = [(1, -1.0, 1.0, 0.2), (2, 0.0, 3.0, 0.2), (3, -1.0, 2.5, 0.05), (4, -0.1, 0.1, 0.45),
         (4, 0.0, 6.0, 0.2), (8, -2.0, 2.0, 0.3), (2, 0.0, 1.0, 0.004)]


@pytest.fixture(scope="module")
def dsq():
    import paper_1908_05033_b200 as d
    return d


def f32(v):
    """The binary32 value the library receives, as a Python float: the oracle
    gets exactly the same bounds and alpha."""
    return float(np.float32(v))


def inputs(lo, hi, n, seed):
    rng = np.random.default_rng(seed)
    x = rng.normal((lo + hi) / 2, (hi - lo) * 0.6, n).astype(np.float32)
    # exact bounds, interval ends and midpoints, far outliers
    special = np.array([lo, hi, lo - 1, hi + 1, (lo + hi) / 2, lo + (hi - lo) / 3, 1e30, -1e30],
                       np.float32)
    x[:min(8, n)] = special[:min(8, n)]
    g = rng.normal(0, 1, n).astype(np.float32)
    return x, g


def bound(bits, lo, hi, alpha):
    d = soft.delta(bits, lo, hi)
    s, k = soft.s_from_alpha(alpha), soft.k_from_alpha(alpha, bits, lo, hi)
    return 4 * EPS * max(abs(lo), abs(hi)) * (1 + 0.5 * d * s * k), 0.5 * d * s * k


@pytest.mark.parametrize("bits,lo,hi,alpha", CASES)
@pytest.mark.parametrize("n", [1, 1000, 4099, 1 << 20])
def test_soft_quantize_forward(dsq, bits, lo, hi, alpha, n):
    lo, hi, alpha = f32(lo), f32(hi), f32(alpha)
    x, _ = inputs(lo, hi, n, bits + n)
    y = N(dsq.dsq_soft_quantize_fwd(T(x), bits, lo, hi, alpha))
    ref = soft.q_soft(x.astype(np.float64), bits, lo, hi, alpha)
    tol, _ = bound(bits, lo, hi, alpha)
    assert np.max(np.abs(y - ref)) <= tol
    # outside the range the result is exactly the bound
    assert np.all(y[x < lo] == np.float32(lo)) and np.all(y[x > hi] == np.float32(hi))


@pytest.mark.parametrize("bits,lo,hi,alpha", CASES)
@pytest.mark.parametrize("n", [1000, 4099, 1 << 20])
def test_soft_quantize_backward(dsq, bits, lo, hi, alpha, n):
    lo, hi, alpha = f32(lo), f32(hi), f32(alpha)
    x, g = inputs(lo, hi, n, bits * 7 + n)
    # keep the sample off the interval boundaries: there the interval index of
    # a binary32 and a binary64 evaluation may differ, and the one-sided
    # derivatives with respect to l and u are not equal
    d = soft.delta(bits, lo, hi)
    frac = (x.astype(np.float64) - lo) / d
    frac -= np.floor(frac)
    near = (frac < 1e-3) | (frac > 1 - 1e-3)
    x[near & (x > lo) & (x < hi)] += np.float32(0.01 * d)
    gx, gp = dsq.dsq_soft_quantize_bwd(T(x), T(g), bits, lo, hi, alpha)
    gx, gp = N(gx), N(gp)
    rx, rp = soft_grad.backward(x.astype(np.float64), g.astype(np.float64), bits, lo, hi, alpha)
    tol, slope = bound(bits, lo, hi, alpha)
    scale_k = soft.k_from_alpha(alpha, bits, lo, hi)
    assert np.all(np.abs(gx - rx) <= 1e-4 * np.abs(rx) + np.abs(g) * slope * 2 * scale_k * tol + 1e-30)
    # the three sums: every element term within the same relative bound
    dx, da, dl, du = soft_grad.partials(x.astype(np.float64), bits, lo, hi, alpha)
    for j, part in enumerate((da, dl, du)):
        mag = float(np.sum(np.abs(g * part)))
        assert abs(gp[j] - rp[j]) <= 2e-4 * mag + 1e-12, (j, gp[j], rp[j], mag)


def test_soft_quantize_converges_to_the_deployed_codes(dsq):
    """As alpha -> 0 the soft quantiser's output approaches l + Delta * code with
    the code dsq_quantize_act produces (the deployed hard quantiser): points
    within 0.2 Delta of a level, where s tanh(k * 0.3 Delta) is within 1 % of 1
    at alpha = 1e-4 (k Delta = log(2/alpha - 1) = 9.9)."""
    bits, lo, hi = 4, 0.0, 2.0
    rng = np.random.default_rng(0)
    d = (hi - lo) / 15
    level = rng.integers(0, 16, (1, 1, 4096, 64))
    x = (lo + d * (level + rng.uniform(-0.2, 0.2, level.shape))).astype(np.float32)
    codes = dsq.dsq_unpack(dsq.dsq_quantize_act(T(x), bits, lo, hi).view(4096, -1), 4096, 64, bits, False)
    assert np.array_equal(N(codes).reshape(level.shape), level)
    hard = lo + d * level
    y = N(dsq.dsq_soft_quantize_fwd(T(x), bits, lo, hi, 1e-4))
    assert np.max(np.abs(y - hard)) < 0.01 * d


def test_soft_quantize_argument_checks(dsq):
    x = torch.zeros(16, device="cuda")
    for bad_alpha in (0.0, 1.0, -0.1, float("nan")):
        with pytest.raises(dsq.DsqError) as e:
            dsq.dsq_soft_quantize_fwd(x, 4, 0.0, 1.0, bad_alpha)
        assert e.value.status == -6
    with pytest.raises(dsq.DsqError) as e:
        dsq.dsq_soft_quantize_fwd(x, 9, 0.0, 1.0, 0.2)
    assert e.value.status == -3
    with pytest.raises(dsq.DsqError) as e:
        dsq.dsq_soft_quantize_bwd(x, x, 4, 1.0, 1.0, 0.2)
    assert e.value.status == -6
