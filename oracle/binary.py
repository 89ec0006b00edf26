"""Binary (1-bit) quantiser and GEMM in numpy (TEST INFRASTRUCTURE ONLY).

Eq. 1 of the paper: the binary quantiser is Q_B(x) = sgn(x) with sgn(0) = +1,
values in {-1, +1}.  It is the 1-bit case of the uniform quantiser (Eq. 2) on
the symmetric range [-1, 1]: Delta = 2, one interval, code q = 0 below the
midpoint 0 and q = 1 from the midpoint up, value l + Delta q = 2 q - 1.

A binary layer's contraction is then, for bit rows a, b of K values each,

    C[m][n] = sum_k (2 a[m][k] - 1) (2 b[n][k] - 1)
            = K - 2 * popcount(a[m] xor b[n])          (the xnor-popcount form)

since equal bits contribute +1 and differing bits -1.  binary_gemm computes the
popcount form on packed bytes; tests pin it to the +-1 matrix product written
out with plain integer arithmetic and to the general-b integer oracle.
"""
import numpy as np


def q_binary(x):
    """Eq. 1: sgn with sgn(0) = +1, as bits (1 = +1, 0 = -1)."""
    return (np.asarray(x) >= 0).astype(np.int8)


def pack_bits(bits):
    """[rows, K] array of 0/1 -> bytes, element j in bit j & 7 of byte j >> 3."""
    bits = np.asarray(bits).astype(np.uint8)
    return np.packbits(bits, axis=1, bitorder="little")


_POPCOUNT = np.array([bin(i).count("1") for i in range(256)], np.int32)


def binary_gemm(a_bits, b_bits):
    """C[m][n] = K - 2 popcount(a[m] xor b[n]); a_bits [M,K], b_bits [N,K] of 0/1."""
    a_bits = np.asarray(a_bits)
    b_bits = np.asarray(b_bits)
    K = a_bits.shape[1]
    pa, pb = pack_bits(a_bits), pack_bits(b_bits)
    out = np.empty((pa.shape[0], pb.shape[0]), np.int32)
    for m in range(pa.shape[0]):
        out[m] = K - 2 * _POPCOUNT[np.bitwise_xor(pa[m][None, :], pb)].sum(axis=1)
    return out
