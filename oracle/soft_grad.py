"""Gradients of DSQ's soft quantiser in numpy float64 (TEST INFRASTRUCTURE ONLY).

Eq. 10-13 of the paper and the back-propagation lines of Algorithm 1, written
out for one tensor.  With the notation of oracle/soft.py, for x in P_i

    Q_S = l + Delta * q,   q = i + (phi + 1)/2                       (Eq. 5, 13)
    phi = s * tanh(z),     z = k (x - m_i),  m_i = l + (i + 1/2) Delta
    s = 1/(1 - alpha),     k = log(2/alpha - 1) / Delta              (Eq. 7, 8)
    Delta = (u - l)/(2^b - 1)

the interval index i is piecewise constant, so

    dQ_S/dx     = (Delta/2) * s * k * (1 - tanh(z)^2)
    dQ_S/dalpha = (Delta/2) * dphi/dalpha                            (Eq. 10)
        dphi/dalpha = ds/dalpha * tanh(z) + s (1 - tanh^2) (x - m_i) dk/dalpha
        ds/dalpha = 1/(1 - alpha)^2,  dk/dalpha = -2 / (Delta alpha (2 - alpha))
    dQ_S/dl     = 1 + q dDelta/dl + (Delta/2) dphi/dl                (Eq. 11)
    dQ_S/du     =     q dDelta/du + (Delta/2) dphi/du                (Eq. 12)
        dDelta/dl = -1/(2^b - 1),  dDelta/du = +1/(2^b - 1)
        dphi/dp = s (1 - tanh^2) [ dk/dp (x - m_i) - k dm_i/dp ],  p in {l, u}
        dk/dp = -(k/Delta) dDelta/dp
        dm_i/dl = 1 + (i + 1/2) dDelta/dl,  dm_i/du = (i + 1/2) dDelta/du

and outside the clip range Q_S is the constant l (x < l) or u (x > u):
dQ_S/dx = dQ_S/dalpha = 0 there, dQ_S/dl = 1 and dQ_S/du = 0 for x < l,
dQ_S/dl = 0 and dQ_S/du = 1 for x > u.

Pinned by central finite differences of soft.q_soft (tests/test_oracle_soft_grad.py).
"""
import numpy as np

from . import soft


def partials(x, bits, lo, hi, alpha):
    """(dQ/dx, dQ/dalpha, dQ/dl, dQ/du) elementwise, float64."""
    x = np.asarray(x, np.float64)
    lo, hi, alpha = float(lo), float(hi), float(alpha)
    n = 2 ** bits - 1
    d = soft.delta(bits, lo, hi)
    k = soft.k_from_alpha(alpha, bits, lo, hi)
    s = soft.s_from_alpha(alpha)
    xc = np.clip(x, lo, hi)
    i = soft.interval_index(xc, bits, lo, hi)
    m = lo + (i + 0.5) * d
    t = np.tanh(k * (xc - m))
    sech2 = 1.0 - t * t
    phi = s * t
    q = i + (phi + 1.0) / 2.0

    dx = 0.5 * d * s * k * sech2

    ds_da = 1.0 / (1.0 - alpha) ** 2
    dk_da = -2.0 / (d * alpha * (2.0 - alpha))
    da = 0.5 * d * (ds_da * t + s * sech2 * (xc - m) * dk_da)

    dd_dl, dd_du = -1.0 / n, 1.0 / n
    dk_dl, dk_du = -(k / d) * dd_dl, -(k / d) * dd_du
    dm_dl = 1.0 + (i + 0.5) * dd_dl
    dm_du = (i + 0.5) * dd_du
    dphi_dl = s * sech2 * (dk_dl * (xc - m) - k * dm_dl)
    dphi_du = s * sech2 * (dk_du * (xc - m) - k * dm_du)
    dl = 1.0 + q * dd_dl + 0.5 * d * dphi_dl
    du = q * dd_du + 0.5 * d * dphi_du

    below, above = x < lo, x > hi
    out = below | above
    dx = np.where(out, 0.0, dx)
    da = np.where(out, 0.0, da)
    dl = np.where(below, 1.0, np.where(above, 0.0, dl))
    du = np.where(below, 0.0, np.where(above, 1.0, du))
    return dx, da, dl, du


def backward(x, grad_y, bits, lo, hi, alpha):
    """Back-propagation through y = Q_S(x): returns (grad_x elementwise,
    [dL/dalpha, dL/dl, dL/du]) for the upstream gradient grad_y = dL/dy."""
    g = np.asarray(grad_y, np.float64)
    dx, da, dl, du = partials(x, bits, lo, hi, alpha)
    return g * dx, np.array([np.sum(g * da), np.sum(g * dl), np.sum(g * du)])
