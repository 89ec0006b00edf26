"""Soft quantiser of DSQ in numpy float64 (TEST INFRASTRUCTURE ONLY).

Follows the paper's notation, Sec. 3.2-3.3:
  Delta = (u - l) / (2^b - 1)                          (below Eq. 2)
  intervals P_i = [l + i*Delta, l + (i+1)*Delta), i = 0 .. 2^b - 2, the last
  one closed at u (the text's "i in 0..2^b-1" is read as an off-by-one)
  m_i = l + (i + 0.5) * Delta,  s = 1 / tanh(0.5 k Delta)            (Eq. 4)
  phi(x) = s * tanh(k (x - m_i)),  x in P_i                          (Eq. 3)
  Q_S(x) = l (x < l);  u (x > u);  l + Delta (i + (phi(x)+1)/2)      (Eq. 5)
  alpha = 1 - tanh(0.5 k Delta) = 1 - 1/s                            (Eq. 6)
  s = 1 / (1 - alpha)                                                (Eq. 7)
  k = (1/Delta) log(2/alpha - 1)                                     (Eq. 8)
and the deployed code of Algorithm 1 steps 3-4: q = i + (sgn(phi)+1)/2 with
sgn(0) = +1 (Eq. 1).
"""
import numpy as np


def delta(bits, lo, hi):
    return (float(hi) - float(lo)) / (2 ** bits - 1)


def k_from_alpha(alpha, bits, lo, hi):
    """Eq. 8."""
    return np.log(2.0 / alpha - 1.0) / delta(bits, lo, hi)


def s_from_alpha(alpha):
    """Eq. 7."""
    return 1.0 / (1.0 - alpha)


def alpha_from_k(k, bits, lo, hi):
    """Eq. 6."""
    return 1.0 - np.tanh(0.5 * k * delta(bits, lo, hi))


def interval_index(x, bits, lo, hi):
    """Index i of the interval P_i holding x (x already inside [l, u])."""
    d = delta(bits, lo, hi)
    i = np.floor((np.asarray(x, np.float64) - lo) / d)
    return np.clip(i, 0, 2 ** bits - 2)


def phi(x, bits, lo, hi, alpha):
    """Eq. 3 with (s, k) expressed through alpha (Eq. 7-8).  Returns
    (phi(x), i)."""
    x = np.asarray(x, np.float64)
    d = delta(bits, lo, hi)
    i = interval_index(x, bits, lo, hi)
    m = lo + (i + 0.5) * d
    k = k_from_alpha(alpha, bits, lo, hi)
    s = s_from_alpha(alpha)
    return s * np.tanh(k * (x - m)), i


def q_soft(x, bits, lo, hi, alpha):
    """Eq. 5."""
    x = np.asarray(x, np.float64)
    d = delta(bits, lo, hi)
    xc = np.clip(x, lo, hi)
    p, i = phi(xc, bits, lo, hi, alpha)
    y = lo + d * (i + (p + 1.0) / 2.0)
    y = np.where(x < lo, float(lo), y)
    y = np.where(x > hi, float(hi), y)
    return y


def code_via_sgn_phi(x, bits, lo, hi, alpha):
    """Algorithm 1 steps 1, 3: clip, then q = i + (sgn(phi(x)) + 1)/2 with
    sgn(0) = +1.  Returns integer codes 0 .. 2^b - 1."""
    x = np.asarray(x, np.float64)
    xc = np.clip(x, lo, hi)
    p, i = phi(xc, bits, lo, hi, alpha)
    sgn = np.where(p >= 0.0, 1.0, -1.0)
    return (i + (sgn + 1.0) / 2.0).astype(np.int64)


def q_uniform(x, bits, lo, hi):
    """Hard quantise-dequantise in float64: l + Delta * floor((x_c-l)/Delta
    + 1/2) (Eq. 2 with the offset and clip of Algorithm 1)."""
    x = np.asarray(x, np.float64)
    d = delta(bits, lo, hi)
    xc = np.clip(x, lo, hi)
    q = np.minimum(np.floor((xc - lo) / d + 0.5), 2 ** bits - 1)
    return lo + d * q
