"""GPU parity, low-bit GEMM on the tensor cores: int32 results bit-exact
against the oracle, fp32 dequantised results bit-exact too (one multiply)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import native
import dsq_inputs
from gpu_util import T, N


@pytest.fixture(scope="module")
def dsq():
    import paper_1908_05033_b200 as d
    return d


def run(dsq, A, B, rs, bits):
    M, K = A.shape
    Nn = B.shape[0]
    ws = dsq.new_workspace()
    Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
    Cg, Dg = dsq.dsq_gemm(Ap, Bp, M, Nn, K, bits, ws, row_scale=T(rs))
    assert dsq.dsq_workspace_status(ws) == 0
    return N(Cg), N(Dg)


SIZES = [(1, 1, 1), (128, 32, 128), (128, 256, 128), (130, 70, 200),
         (300, 257, 1000), (129, 513, 129), (64, 48, 4096), (515, 130, 771),
         (130, 72, 200), (300, 260, 1000), (257, 516, 300)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("size", SIZES)
def test_gemm_small_and_ragged(dsq, bits, size):
    M, Nn, K = size
    A, B, rs = dsq_inputs.gemm_case(M, Nn, K, bits)
    C = native.gemm(A, B)
    Cg, Dg = run(dsq, A, B, rs, bits)
    assert np.array_equal(C, Cg)
    assert np.array_equal(native.gemm_dequant(C, rs), Dg)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_gemm_extreme_codes(dsq, bits):
    # every product at its most negative: K * (-2^(b-1)) * (2^b - 1)
    half = 1 << (bits - 1)
    M, Nn, K = 128, 64, 8192
    A = np.full((M, K), -half, np.int8)
    B = np.full((Nn, K), 2 * half - 1, np.int8)
    rs = np.ones(M, np.float32)
    Cg, Dg = run(dsq, A, B, rs, bits)
    assert np.all(Cg == K * -half * (2 * half - 1))
    A[:] = half - 1
    Cg, _ = run(dsq, A, B, rs, bits)
    assert np.all(Cg == K * (half - 1) * (2 * half - 1))
    Cg, _ = run(dsq, np.zeros_like(A), B, rs, bits)
    assert not Cg.any()


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_gemm_1024_full(dsq, bits):
    A, B, rs = dsq_inputs.gemm_case(1024, 1024, 1024, bits)
    C = native.gemm(A, B)
    Cg, Dg = run(dsq, A, B, rs, bits)
    assert np.array_equal(C, Cg)
    assert np.array_equal(native.gemm_dequant(C, rs), Dg)


@pytest.mark.parametrize("bits,size", [(4, 4096), (2, 4096), (3, 4096), (4, 8192)])
def test_gemm_full_size_sampled(dsq, bits, size):
    """Full-size launch as the benchmark times it; 64 sampled rows x 64
    sampled columns (4096 complete dot products) against the oracle, plus the
    whole first tile row."""
    A, B, rs = dsq_inputs.gemm_case(size, size, size, bits)
    Cg, Dg = run(dsq, A, B, rs, bits)
    rng = np.random.default_rng(size + bits)
    rows = np.sort(rng.choice(size, 64, replace=False))
    cols = np.sort(rng.choice(size, 64, replace=False))
    C = native.gemm(A[rows], B[cols])
    assert np.array_equal(C, Cg[np.ix_(rows, cols)])
    assert np.array_equal(native.gemm_dequant(C, rs[rows]), Dg[np.ix_(rows, cols)])
    C = native.gemm(A[size - 3:], B)                      # last rows, all columns
    assert np.array_equal(C, Cg[size - 3:])
    # determinism: a second run gives identical bits
    Cg2, _ = run(dsq, A, B, rs, bits)
    assert np.array_equal(Cg, Cg2)


def run_two_pass(dsq, A, B, rs, bits, want_i32=True):
    """dsq_gemm with a workspace that has room for the expanded operands."""
    M, K = A.shape
    Nn = B.shape[0]
    dsq.dsq_set_gemm_two_pass(2)          # two passes whatever the size
    try:
        assert dsq.dsq_gemm_workspace_bytes(M, Nn, K, bits) > dsq.dsq_workspace_bytes()
        ws = dsq.new_gemm_workspace(M, Nn, K, bits)
        Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
        Cg, Dg = dsq.dsq_gemm(Ap, Bp, M, Nn, K, bits, ws, row_scale=T(rs), want_i32=want_i32)
        assert dsq.dsq_workspace_status(ws) == 0
    finally:
        dsq.dsq_set_gemm_two_pass(1)
    return (N(Cg) if want_i32 else None), N(Dg)


# the two-pass path (rows expanded to 8-bit once, then an 8-bit GEMM): whole
# tiles, ragged M / N / K, an N that is not a multiple of 8 (scalar stores), a K
# that is not a multiple of 16
TWO_PASS_SIZES = [(1, 1, 1), (130, 70, 200), (300, 257, 1000), (1024, 1024, 1024),
                  (1100, 1030, 1050), (1024, 1027, 1031), (1281, 1536, 2048)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("size", TWO_PASS_SIZES)
def test_gemm_two_pass_full(dsq, bits, size):
    M, Nn, K = size
    A, B, rs = dsq_inputs.gemm_case(M, Nn, K, bits)
    C = native.gemm(A, B)
    Cg, Dg = run_two_pass(dsq, A, B, rs, bits)
    assert np.array_equal(C, Cg)
    assert np.array_equal(native.gemm_dequant(C, rs), Dg)
    _, Dg = run_two_pass(dsq, A, B, rs, bits, want_i32=False)
    assert np.array_equal(native.gemm_dequant(C, rs), Dg)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_gemm_two_pass_extreme_codes(dsq, bits):
    half = 1 << (bits - 1)
    M, Nn, K = 1024, 1024, 8192
    A = np.full((M, K), -half, np.int8)
    B = np.full((Nn, K), 2 * half - 1, np.int8)
    rs = np.ones(M, np.float32)
    Cg, _ = run_two_pass(dsq, A, B, rs, bits)
    assert np.all(Cg == K * -half * (2 * half - 1))
    A[:] = half - 1
    Cg, _ = run_two_pass(dsq, A, B, rs, bits)
    assert np.all(Cg == K * (half - 1) * (2 * half - 1))


@pytest.mark.parametrize("bits,size", [(4, 4096), (2, 4096), (3, 4096), (4, 8192)])
def test_gemm_two_pass_full_size_sampled(dsq, bits, size):
    """Full-size launch as the benchmark times it: sampled dot products and the
    last rows against the oracle, and every element against the fused kernel."""
    A, B, rs = dsq_inputs.gemm_case(size, size, size, bits)
    Cg, Dg = run_two_pass(dsq, A, B, rs, bits)
    rng = np.random.default_rng(size + bits)
    rows = np.sort(rng.choice(size, 64, replace=False))
    cols = np.sort(rng.choice(size, 64, replace=False))
    C = native.gemm(A[rows], B[cols])
    assert np.array_equal(C, Cg[np.ix_(rows, cols)])
    assert np.array_equal(native.gemm_dequant(C, rs[rows]), Dg[np.ix_(rows, cols)])
    C = native.gemm(A[size - 3:], B)
    assert np.array_equal(C, Cg[size - 3:])
    Cf, Df = run(dsq, A, B, rs, bits)                 # fused kernel, small workspace
    assert np.array_equal(Cf, Cg) and np.array_equal(Df, Dg)


def test_gemm_two_pass_repeated_launches_identical(dsq):
    """300 launches of 4096^3 through the two-pass path (a shared scratch
    rewritten every call, two accumulators, a CTA pair's barriers crossing SMs):
    every launch equals the first, whose rows are checked against the oracle."""
    size, bits = 4096, 4
    A, B, rs = dsq_inputs.gemm_case(size, size, size, bits)
    ws = dsq.new_gemm_workspace(size, size, size, bits)
    Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
    rst = T(rs)
    C0, D0 = dsq.dsq_gemm(Ap, Bp, size, size, size, bits, ws, row_scale=rst)
    C0, D0 = C0.clone(), D0.clone()
    C = torch.empty_like(C0)
    D = torch.empty_like(D0)
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for _ in range(300):
        dsq.dsq_gemm(Ap, Bp, size, size, size, bits, ws, row_scale=rst, out_i32=C, out_f32=D)
        bad += (C != C0).any().to(torch.int64) + (D != D0).any().to(torch.int64)
    assert int(bad.item()) == 0
    assert dsq.dsq_workspace_status(ws) == 0
    rows = np.arange(0, size, 257)
    Cref = native.gemm(A[rows], B)
    assert np.array_equal(Cref, N(C0)[rows])


def test_gemm_repeated_launches_identical(dsq):
    """Regression test of a race between the two CTAs of a pair that showed
    about once in 150 launches (a stale half of the expanded B operand read by
    the peer SM's tensor core): 600 launches of 8192^3 with both outputs, many
    tiles per CTA pair, every launch compared bit for bit on the device with
    the first, whose rows are checked against the oracle."""
    size, bits = 8192, 4
    A, B, rs = dsq_inputs.gemm_case(size, size, size, bits)
    ws = dsq.new_workspace()
    Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
    rst = T(rs)
    C0, D0 = dsq.dsq_gemm(Ap, Bp, size, size, size, bits, ws, row_scale=rst)
    C0, D0 = C0.clone(), D0.clone()
    C = torch.empty_like(C0)
    D = torch.empty_like(D0)
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for _ in range(600):
        dsq.dsq_gemm(Ap, Bp, size, size, size, bits, ws, row_scale=rst, out_i32=C, out_f32=D)
        bad += (C != C0).any().to(torch.int64) + (D != D0).any().to(torch.int64)
    assert int(bad.item()) == 0
    assert dsq.dsq_workspace_status(ws) == 0
    rows = np.arange(0, size, 517)
    Cref = native.gemm(A[rows], B)
    assert np.array_equal(Cref, N(C0)[rows])
    assert np.array_equal(native.gemm_dequant(Cref, rs[rows]), N(D0)[rows])


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_bounded_wait_runs_out_and_the_next_call_is_clean(dsq, bits):
    """A wait that nothing satisfies: the test hook makes the TMA producer of
    the B operand leave out one round, so the warps waiting for it run into
    the wait limit (set to 3 ms here).  The kernel must return by itself with
    DSQ_ERR_TIMEOUT in the workspace (nothing faults, nothing hangs), and the
    same problem launched right after, with the hook off and the default
    limit, must give the oracle's result."""
    M, Nn, K = 128, 64, 1024               # one tile, one CTA (no pair)
    A, B, rs = dsq_inputs.gemm_case(M, Nn, K, bits)
    Cref = native.gemm(A, B)
    ws = dsq.new_workspace()
    Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
    for skip in (0, 2):
        dsq.dsq_set_wait_limit_ns(3_000_000)
        dsq.dsq_set_test_skip_b_round(skip)
        try:
            dsq.dsq_gemm(Ap, Bp, M, Nn, K, bits, ws)
            torch.cuda.synchronize()       # the kernel came back
        finally:
            dsq.dsq_set_test_skip_b_round(-1)
            dsq.dsq_set_wait_limit_ns(0)
        assert dsq.dsq_workspace_status(ws) == -10          # DSQ_ERR_TIMEOUT
        assert dsq.dsq_workspace_status(ws) == 0            # reading clears it
        Cg, Dg = dsq.dsq_gemm(Ap, Bp, M, Nn, K, bits, ws, row_scale=T(rs))
        assert dsq.dsq_workspace_status(ws) == 0
        assert np.array_equal(N(Cg), Cref)
        assert np.array_equal(N(Dg), native.gemm_dequant(Cref, rs))


def test_bounded_wait_runs_out_in_a_convolution(dsq):
    """Same for dsq_conv2d (TMA im2col A boxes, codes epilogue)."""
    c = dsq_inputs.conv3x3_case(N=1, H=12, W=12, Cin=128, Cout=64)
    bits = c["bits"]
    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(c["x"]), bits, 0.0, 2.0)
    blob, conv = dsq.dsq_pack_weights(T(c["w"]), bits, -0.1, 0.1, ws, stride=1, pad=1)
    args = (act, c["x"].shape, (bits, 0.0, 2.0), blob, conv, T(c["scale"]), T(c["bias"]), ws)
    good, _, _ = dsq.dsq_conv2d(*args, requant=(bits, 0.0, 1.0))
    assert dsq.dsq_workspace_status(ws) == 0
    dsq.dsq_set_wait_limit_ns(3_000_000)
    dsq.dsq_set_test_skip_b_round(1)
    try:
        dsq.dsq_conv2d(*args, requant=(bits, 0.0, 1.0))
        torch.cuda.synchronize()
    finally:
        dsq.dsq_set_test_skip_b_round(-1)
        dsq.dsq_set_wait_limit_ns(0)
    assert dsq.dsq_workspace_status(ws) == -10
    again, _, _ = dsq.dsq_conv2d(*args, requant=(bits, 0.0, 1.0))
    assert dsq.dsq_workspace_status(ws) == 0
    assert torch.equal(good, again)
