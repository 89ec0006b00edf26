"""Pins of oracle/binary.py and oracle/weight_only.py."""
import numpy as np
import pytest

from oracle import binary, native, soft, weight_only


def test_q_binary_is_the_one_bit_uniform_quantiser():
    # Eq. 1: sgn with sgn(0) = +1; equals the hard quantiser at b = 1 on [-1, 1]
    x = np.array([-3.0, -1.0, -1e-6, -0.0, 0.0, 1e-6, 0.3, 1.0, 7.0], np.float32)
    bits = binary.q_binary(x)
    assert bits.tolist() == [0, 0, 0, 1, 1, 1, 1, 1, 1]
    assert np.array_equal(native.quantize(x, 1, -1.0, 1.0), bits)
    # dequantised: l + Delta q = 2 q - 1 in {-1, +1}
    assert np.array_equal(native.dequantize(bits, 1, -1.0, 1.0), 2.0 * bits - 1.0)
    # the sgn . phi form of the soft quantiser gives the same code
    xs = np.linspace(-0.999, 0.999, 41)
    assert np.array_equal(soft.code_via_sgn_phi(xs, 1, -1.0, 1.0, 0.2), binary.q_binary(xs))


def test_pack_bits_layout():
    # element j in bit j & 7 of byte j >> 3
    row = np.zeros((1, 19), np.int8)
    row[0, [0, 3, 8, 18]] = 1
    assert binary.pack_bits(row).tolist() == [[0b00001001, 0b00000001, 0b00000100]]


@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 7), (17, 9, 130), (8, 8, 64)])
def test_binary_gemm_is_the_plus_minus_one_product(shape):
    M, N, K = shape
    rng = np.random.default_rng(K)
    a = rng.integers(0, 2, (M, K)).astype(np.int8)
    b = rng.integers(0, 2, (N, K)).astype(np.int8)
    want = np.zeros((M, N), np.int64)
    for m in range(M):
        for n in range(N):
            for k in range(K):
                want[m, n] += (1 if a[m, k] else -1) * (1 if b[n, k] else -1)
    got = binary.binary_gemm(a, b)
    assert np.array_equal(got, want)
    # through the general-b integer oracle: sum (2a-1)(2b-1) = 4 sum ab - 2 sum a - 2 sum b + K
    ab = native.gemm(a, b).astype(np.int64)
    assert np.array_equal(4 * ab - 2 * a.sum(1)[:, None] - 2 * b.sum(1)[None, :] + K, want)


def test_binary_gemm_closed_forms():
    K = 77
    a = np.ones((2, K), np.int8)
    assert np.all(binary.binary_gemm(a, a) == K)          # equal rows: +K
    assert np.all(binary.binary_gemm(a, 1 - a) == -K)     # opposite rows: -K
    b = a.copy()
    b[:, :10] = 0
    assert np.all(binary.binary_gemm(a, b) == K - 20)     # ten differing bits


def test_weight_only_linear_hand_computed():
    # two output channels, 2-bit weights on [-0.3, 0.3]: levels -0.3, -0.1, 0.1, 0.3
    q = np.array([[0, 1, 2, 3], [3, 3, 0, 1]])
    x = np.array([[1.0, 2.0, -1.0, 0.5]])
    y = weight_only.linear(x, q, 2, -0.3, 0.3, bias=[0.25, -1.0])
    assert np.allclose(y, [[-0.3 - 0.2 - 0.1 + 0.15 + 0.25, 0.3 + 0.6 + 0.3 - 0.05 - 1.0]], atol=1e-15)
    # a one-hot activation row reads out one dequantised weight column
    w_hat = weight_only.dequantize_weights(q, 2, -0.3, 0.3)
    assert np.allclose(weight_only.linear(np.eye(4), q, 2, -0.3, 0.3), w_hat.T, atol=1e-15)
    # per-channel ranges; equals the oracle's dequantiser
    lo, hi = np.array([-0.3, -0.6]), np.array([0.3, 0.6])
    w2 = weight_only.dequantize_weights(q, 2, lo, hi)
    for n in range(2):
        assert np.allclose(w2[n], native.dequantize(q[n].astype(np.int8), 2, lo[n], hi[n]))


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_weight_only_equals_integer_form(bits):
    """Y = (Delta/2) sum x (2c + 1) + bias on a symmetric clip: the form the GPU
    kernel evaluates (c = q - 2^(b-1)) is the same number."""
    rng = np.random.default_rng(bits)
    N, K, M = 5, 33, 4
    q = rng.integers(0, 2 ** bits, (N, K))
    x = rng.standard_normal((M, K))
    u = rng.uniform(0.1, 0.5, N)
    y = weight_only.linear(x, q, bits, -u, u)
    c = q - 2 ** (bits - 1)
    delta = 2 * u / (2 ** bits - 1)
    assert np.allclose(y, (x @ (2 * c + 1).T) * (delta / 2)[None, :], rtol=1e-13, atol=1e-13)
