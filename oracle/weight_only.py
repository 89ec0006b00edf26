"""Weight-only low-bit linear layer in numpy float64 (TEST INFRASTRUCTURE ONLY).

The W-bit / full-precision-activation rows of the paper's Table 7: only the
weights go through the quantiser (Algorithm 1 steps 1, 3, 4: clip to
[l_w, u_w], q = round((w - l_w)/Delta_w), w^ = l_w + Delta_w q), activations
stay real.  The layer is then the plain product

    Y[m][n] = sum_k X[m][k] * w^[n][k] + bias[n]

evaluated here exactly as written, in float64, from the unsigned weight codes
q and the per-row (per-output-channel) range.
"""
import numpy as np


def dequantize_weights(q, bits, lo, hi):
    """w^ = l_w + Delta_w q per output channel; q [N,K] unsigned codes, lo/hi [N] or scalars."""
    q = np.asarray(q, np.float64)
    lo = np.broadcast_to(np.asarray(lo, np.float64), (q.shape[0],))[:, None]
    hi = np.broadcast_to(np.asarray(hi, np.float64), (q.shape[0],))[:, None]
    delta = (hi - lo) / (2 ** bits - 1)
    return lo + delta * q


def linear(x, q, bits, lo, hi, bias=None):
    """Y = X w^T + bias in float64.  x [M,K] real, q [N,K] unsigned codes."""
    y = np.asarray(x, np.float64) @ dequantize_weights(q, bits, lo, hi).T
    if bias is not None:
        y = y + np.asarray(bias, np.float64)[None, :]
    return y


def abs_linear(x, q, bits, lo, hi):
    """sum_k |X w^|: the scale of the rounding error of an fp32 accumulation."""
    return np.abs(np.asarray(x, np.float64)) @ np.abs(dequantize_weights(q, bits, lo, hi)).T
