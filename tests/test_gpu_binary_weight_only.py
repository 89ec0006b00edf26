"""GPU parity of the binary GEMM (bit-exact against the xnor-popcount oracle)
and of the weight-only bf16 x low-bit GEMM (fp32 accumulation on the tensor
core against the float64 oracle, within K 2^-23 sum|x w^| per element)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import binary, native, weight_only
import dsq_inputs
from gpu_util import T, N


@pytest.fixture(scope="module")
def dsq():
    import paper_1908_05033_b200 as d
    return d


BIN_SIZES = [(1, 1, 1), (3, 5, 7), (128, 256, 128), (130, 70, 200), (300, 257, 1000),
             (257, 516, 1031), (1024, 1024, 1024)]


@pytest.mark.parametrize("size", BIN_SIZES)
def test_binary_gemm(dsq, size):
    M, Nn, K = size
    A, B, rs = dsq_inputs.binary_gemm_case(M, Nn, K)
    C = binary.binary_gemm(A, B)
    Ap, Bp = dsq.dsq_pack_codes(T(A), 1), dsq.dsq_pack_codes(T(B), 1)
    # the library's 1-bit rows are the oracle's byte layout
    assert np.array_equal(N(Ap)[:, :(K + 7) // 8], binary.pack_bits(A))
    Cg, Dg = dsq.dsq_binary_gemm(Ap, Bp, M, Nn, K, row_scale=T(rs))
    assert np.array_equal(C, N(Cg))
    assert np.array_equal(native.gemm_dequant(C, rs), N(Dg))


def test_binary_gemm_ignores_bits_past_k(dsq):
    """Spare bits of a packed row must not count (they would read as -1)."""
    M, Nn, K = 64, 64, 100
    A, B, rs = dsq_inputs.binary_gemm_case(M, Nn, K)
    Ap, Bp = dsq.dsq_pack_codes(T(A), 1), dsq.dsq_pack_codes(T(B), 1)
    Ap[:, K // 8 + 1:] = 0xFF
    Ap[:, K // 8] |= 0xF0                                  # bits 100..103
    Bp[:, K // 8 + 1:] = 0x5A
    Cg, _ = dsq.dsq_binary_gemm(Ap, Bp, M, Nn, K)
    assert np.array_equal(binary.binary_gemm(A, B), N(Cg))


def test_binary_gemm_extremes_and_full_size(dsq):
    K = 4096
    ones = np.ones((256, K), np.int8)
    Ap, Bp = dsq.dsq_pack_codes(T(ones), 1), dsq.dsq_pack_codes(T(1 - ones), 1)
    Cg, _ = dsq.dsq_binary_gemm(Ap, Ap, 256, 256, K)
    assert torch.all(Cg == K)
    Cg, _ = dsq.dsq_binary_gemm(Ap, Bp, 256, 256, K)
    assert torch.all(Cg == -K)
    # 4096^3 as the benchmark times it: sampled dot products and the last rows
    size = 4096
    A, B, rs = dsq_inputs.binary_gemm_case(size, size, size)
    Cg, _ = dsq.dsq_binary_gemm(dsq.dsq_pack_codes(T(A), 1), dsq.dsq_pack_codes(T(B), 1),
                                size, size, size)
    Cg = N(Cg)
    rng = np.random.default_rng(7)
    rows = np.sort(rng.choice(size, 64, replace=False))
    cols = np.sort(rng.choice(size, 64, replace=False))
    assert np.array_equal(binary.binary_gemm(A[rows], B[cols]), Cg[np.ix_(rows, cols)])
    assert np.array_equal(binary.binary_gemm(A[size - 2:], B), Cg[size - 2:])


def run_wgemm(dsq, x, q, u, bias, bits, w_offset=0.5):
    M, K = x.shape
    Nn = q.shape[0]
    half = 1 << (bits - 1)
    c = (q.astype(np.int16) - half).astype(np.int8)                # signed codes
    Wp = dsq.dsq_pack_codes(T(c), bits)
    X = T(x).to(torch.bfloat16)
    assert torch.equal(X.to(torch.float32), T(x))                  # inputs hold bf16 values
    delta = (2.0 * u.astype(np.float64)) / (2 ** bits - 1)
    scale = (delta / 2 if w_offset == 0.5 else delta).astype(np.float32)
    Y = dsq.dsq_wgemm_bf16(X, Wp, M, Nn, K, bits, T(scale), T(bias), w_offset=w_offset)
    return N(Y), scale


WG_SIZES = [(1, 1, 8), (5, 3, 64), (128, 256, 128), (130, 70, 200), (300, 257, 1000),
            (257, 516, 1032), (1024, 1024, 1024)]


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("size", WG_SIZES)
def test_weight_only_gemm(dsq, bits, size):
    M, Nn, K = size
    x, q, u, bias = dsq_inputs.weight_only_case(M, Nn, K, bits)
    Yg, scale = run_wgemm(dsq, x, q, u, bias, bits)
    # the oracle gets the scale the kernel got (binary32), as the range of its grid
    u_eff = scale.astype(np.float64) * (2 ** bits - 1)
    Y = weight_only.linear(x, q, bits, -u_eff, u_eff, bias)
    tol = K * 2.0 ** -23 * weight_only.abs_linear(x, q, bits, -u_eff, u_eff) + 1e-6 * np.abs(Y)
    assert np.all(np.abs(Yg - Y) <= tol)
    # and it is far inside that bound on average
    assert np.mean(np.abs(Yg - Y)) <= 0.05 * np.mean(tol)


def test_weight_only_plain_grid_and_no_bias(dsq):
    """w_offset = 0: w^ = Delta c (zero is a level); no bias operand."""
    M, Nn, K, bits = 70, 130, 264, 4
    x, q, u, _ = dsq_inputs.weight_only_case(M, Nn, K, bits)
    c = q.astype(np.float64) - 8
    delta = 2.0 * u.astype(np.float64) / 15
    scale = delta.astype(np.float32)
    Wp = dsq.dsq_pack_codes(T((q.astype(np.int16) - 8).astype(np.int8)), bits)
    Y = dsq.dsq_wgemm_bf16(T(x).to(torch.bfloat16), Wp, M, Nn, K, bits, T(scale), None, w_offset=0.0)
    want = (x.astype(np.float64) @ c.T) * scale.astype(np.float64)[None, :]
    tol = K * 2.0 ** -23 * (np.abs(x.astype(np.float64)) @ np.abs(c).T) * scale[None, :] + 1e-30
    assert np.all(np.abs(N(Y) - want) <= tol)


def test_weight_only_exact_on_integers(dsq):
    """Small-integer activations: every partial sum is an integer below 2^24, so
    fp32 accumulation is exact whatever its order and Y must equal the oracle
    bit for bit (scale 1, no bias)."""
    M, Nn, K, bits = 200, 300, 512, 3
    rng = np.random.default_rng(3)
    x = rng.integers(-8, 9, (M, K)).astype(np.float32)
    q = rng.integers(0, 8, (Nn, K)).astype(np.int8)
    Wp = dsq.dsq_pack_codes(T((q.astype(np.int16) - 4).astype(np.int8)), bits)
    ones = np.ones(Nn, np.float32)
    Y = dsq.dsq_wgemm_bf16(T(x).to(torch.bfloat16), Wp, M, Nn, K, bits, T(ones), None)
    want = x.astype(np.int64) @ (2 * (q.astype(np.int64) - 4) + 1).T
    assert np.array_equal(N(Y).astype(np.int64), want)


def test_argument_checks(dsq):
    x, q, u, bias = dsq_inputs.weight_only_case(8, 8, 12, 4)       # K not a multiple of 8
    Wp = dsq.dsq_pack_codes(T((q.astype(np.int16) - 8).astype(np.int8)), 4)
    with pytest.raises(dsq.DsqError):
        dsq.dsq_wgemm_bf16(T(x).to(torch.bfloat16), Wp, 8, 8, 12, 4, T(u), None)
    x, q, u, bias = dsq_inputs.weight_only_case(8, 8, 16, 4)
    Wp = dsq.dsq_pack_codes(T((q.astype(np.int16) - 8).astype(np.int8)), 4)
    with pytest.raises(dsq.DsqError):                              # unsupported grid offset
        dsq.dsq_wgemm_bf16(T(x).to(torch.bfloat16), Wp, 8, 8, 16, 4, T(u), None, w_offset=0.25)
    small = dsq.new_workspace()
    with pytest.raises(dsq.DsqError):                              # workspace too small
        dsq.dsq_wgemm_bf16(T(x).to(torch.bfloat16), Wp, 8, 8, 16, 4, T(u), None, ws=small)
    A, B, _ = dsq_inputs.binary_gemm_case(8, 8, 64)
    with pytest.raises(dsq.DsqError):
        dsq.dsq_binary_gemm(dsq.dsq_pack_codes(T(A), 1), dsq.dsq_pack_codes(T(B), 1), 8, 8, 64,
                            ws=small)
