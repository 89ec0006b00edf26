"""Pins of the oracle's integer contraction and epilogue: brute force written
a second, different way (im2col + int64 matmul in numpy), closed-form cases,
and the real-valued convolution of the dequantised tensors in float64
(Algorithm 1 steps 4-5)."""
import numpy as np
import pytest

from oracle import native, stack
import dsq_inputs


def im2col_conv(act, wgt, stride, pad):
    """Independent restatement: zero-pad, gather patches, int64 matmul."""
    N, H, W, C = act.shape
    Co, KH, KW, _ = wgt.shape
    a = np.zeros((N, H + 2 * pad, W + 2 * pad, C), np.int64)
    a[:, pad:pad + H, pad:pad + W] = act
    Ho = (H + 2 * pad - KH) // stride + 1
    Wo = (W + 2 * pad - KW) // stride + 1
    cols = np.empty((N, Ho, Wo, KH, KW, C), np.int64)
    for kh in range(KH):
        for kw in range(KW):
            cols[:, :, :, kh, kw] = a[:, kh:kh + stride * Ho:stride,
                                      kw:kw + stride * Wo:stride]
    out = cols.reshape(N * Ho * Wo, -1) @ wgt.reshape(Co, -1).astype(np.int64).T
    return out.reshape(N, Ho, Wo, Co), cols.reshape(N, Ho, Wo, -1).sum(-1)


SHAPES = [  # N, H, W, Cin, Cout, k, stride, pad
    (1, 3, 3, 3, 5, 3, 1, 1), (2, 5, 4, 7, 3, 3, 1, 1), (1, 9, 7, 5, 4, 3, 2, 1),
    (2, 6, 6, 17, 9, 1, 1, 0), (1, 7, 7, 8, 6, 1, 2, 0), (1, 4, 5, 3, 2, 3, 1, 0),
    (1, 8, 8, 4, 4, 3, 2, 0)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("shape", SHAPES)
def test_conv_matches_im2col_brute_force(bits, shape):
    N, H, W, Ci, Co, k, s, p = shape
    rng = np.random.default_rng(hash(shape) % 2 ** 31 + bits)
    half = 1 << (bits - 1)
    act = rng.integers(0, 2 * half, (N, H, W, Ci), dtype=np.int8)
    wgt = rng.integers(-half, half, (Co, k, k, Ci), dtype=np.int8)
    acc, sa = native.conv2d(act, wgt, s, p, want_sa=True)
    ref, ref_sa = im2col_conv(act, wgt, s, p)
    assert np.array_equal(acc, ref) and np.array_equal(sa, ref_sa)


def test_conv_closed_forms():
    bits, half = 4, 8
    N, H, W, Ci, Co = 1, 5, 6, 4, 3
    ones_a = np.ones((N, H, W, Ci), np.int8)
    ones_w = np.ones((Co, 3, 3, Ci), np.int8)
    acc = native.conv2d(ones_a, ones_w, 1, 1)
    # accumulator = number of in-image taps * Cin
    taps = np.array([[(min(h + 1, H - 1) - max(h - 1, 0) + 1) *
                      (min(w + 1, W - 1) - max(w - 1, 0) + 1)
                      for w in range(W)] for h in range(H)])
    assert np.array_equal(acc[0, :, :, 0], taps * Ci)
    # all-extreme codes: K * (-2^(b-1)) * (2^b - 1) at an interior pixel
    acc = native.conv2d(ones_a * (2 * half - 1), ones_w * (-half), 1, 1)
    assert acc[0, 2, 2, 1] == 9 * Ci * (-half) * (2 * half - 1)
    # one-hot weight = shifted input
    rng = np.random.default_rng(3)
    act = rng.integers(0, 16, (1, 6, 7, 2), dtype=np.int8)
    wgt = np.zeros((2, 3, 3, 2), np.int8)
    wgt[0, 0, 2, 1] = 1      # output ch 0 reads channel 1 at (h-1, w+1)
    wgt[1, 1, 1, 0] = -3     # output ch 1 = -3 * channel 0, centre tap
    acc = native.conv2d(act, wgt, 1, 1)
    want = np.zeros((6, 7), np.int64)
    want[1:, :-1] = act[0, :-1, 1:, 1]
    assert np.array_equal(acc[0, :, :, 0], want)
    assert np.array_equal(acc[0, :, :, 1], -3 * act[0, :, :, 0].astype(np.int64))
    # linear in the weights
    w1 = rng.integers(-4, 4, (3, 3, 3, 2), dtype=np.int8)
    w2 = rng.integers(-4, 4, (3, 3, 3, 2), dtype=np.int8)
    assert np.array_equal(native.conv2d(act, w1 + w2, 2, 1),
                          native.conv2d(act, w1, 2, 1) +
                          native.conv2d(act, w2, 2, 1))


def test_gemm_and_1x1_conv_agree_with_numpy():
    rng = np.random.default_rng(9)
    for bits in (2, 3, 4):
        A, B, _ = dsq_inputs.gemm_case(37, 29, 131, bits)
        C = native.gemm(A, B)
        assert np.array_equal(C, A.astype(np.int64) @ B.astype(np.int64).T)
        half = 1 << (bits - 1)
        assert A.min() == -half and A.max() == half - 1
        assert B.min() == 0 and B.max() == 2 * half - 1
    act = rng.integers(0, 16, (2, 4, 5, 11), dtype=np.int8)
    wgt = rng.integers(-8, 8, (6, 1, 1, 11), dtype=np.int8)
    acc = native.conv2d(act, wgt, 1, 0)
    # a 1x1 convolution is the GEMM pixels x channels (weights are the signed
    # operand A, activations the unsigned operand B)
    C = native.gemm(wgt.reshape(6, 11), act.reshape(-1, 11))
    assert np.array_equal(acc.reshape(-1, 6), C.T)
    K = 8192
    A = np.full((1, K), -8, np.int8)
    B = np.full((1, K), 15, np.int8)
    assert native.gemm(A, B)[0, 0] == K * -8 * 15


@pytest.mark.parametrize("bits", [2, 4])
def test_depthwise_is_the_diagonal_of_a_dense_conv(bits):
    rng = np.random.default_rng(21 + bits)
    half = 1 << (bits - 1)
    for (N, H, W, C, s) in [(1, 5, 5, 3, 1), (2, 8, 6, 5, 2), (1, 7, 9, 4, 2)]:
        act = rng.integers(0, 2 * half, (N, H, W, C), dtype=np.int8)
        wd = rng.integers(-half, half, (C, 3, 3), dtype=np.int8)
        acc, sa = native.dwconv2d(act, wd, s, 1, want_sa=True)
        dense = np.zeros((C, 3, 3, C), np.int8)
        for c in range(C):
            dense[c, :, :, c] = wd[c]
        ref, _ = im2col_conv(act, dense, s, 1)
        assert np.array_equal(acc, ref)
        ones = np.zeros((C, 3, 3, C), np.int8)
        for c in range(C):
            ones[c, :, :, c] = 1
        ref_sa, _ = im2col_conv(act, ones, s, 1)
        assert np.array_equal(sa, ref_sa)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_integer_form_equals_real_convolution_of_dequantised_tensors(bits):
    """o = Convolution(w^, a^) (Algorithm 1 step 5) in float64 equals
    Delta_a * Delta_w * (acc + o_w * S_a) with o_w = l_w/Delta_w + 2^(b-1)."""
    rng = np.random.default_rng(bits)
    N, H, W, Ci, Co = 1, 6, 5, 7, 4
    a_lo, a_hi = 0.0, 2.0
    for (w_lo, w_hi) in [(-0.1, 0.1), (-0.07, 0.15)]:
        x = np.maximum(rng.standard_normal((N, H, W, Ci)), 0).astype(np.float32)
        w = (rng.standard_normal((Co, 3, 3, Ci)) * 0.05).astype(np.float32)
        qa = native.quantize(x, bits, a_lo, a_hi)
        cw = native.quantize_weights(w, bits, w_lo, w_hi)
        a_hat = native.dequantize(qa, bits, a_lo, a_hi)
        half = 1 << (bits - 1)
        w_hat = native.dequantize(cw + half, bits, w_lo, w_hi)
        # real-valued conv through the independent im2col, in float64
        ap = np.zeros((N, H + 2, W + 2, Ci))
        ap[:, 1:-1, 1:-1] = a_hat
        o = np.zeros((N, H, W, Co))
        for kh in range(3):
            for kw in range(3):
                o += ap[:, kh:kh + H, kw:kw + W] @ w_hat[:, kh, kw].T
        acc, sa = native.conv2d(qa, cw, 1, 1, want_sa=True)
        da = (a_hi - a_lo) / (2 ** bits - 1)
        dw = (w_hi - w_lo) / (2 ** bits - 1)
        o_w = w_lo / dw + half
        if w_lo == -w_hi:
            assert o_w == pytest.approx(0.5, abs=1e-12)
        integer_form = da * dw * (acc + o_w * sa[..., None])
        assert np.allclose(o, integer_form, rtol=1e-12, atol=1e-13)
        # and the binary32 epilogue reproduces it to single precision
        scale = np.full(Co, da * dw, np.float32)
        y = native.epilogue(acc, scale, np.zeros(Co, np.float32),
                            np.float32(o_w), sa)
        assert np.allclose(y, o, rtol=2e-6, atol=1e-7)


def test_epilogue_special_cases_and_pool():
    rng = np.random.default_rng(2)
    acc = rng.integers(-5000, 5000, (3, 4, 4, 6), dtype=np.int32)
    one, zero = np.ones(6, np.float32), np.zeros(6, np.float32)
    # scale 1, bias 0 => y = (float)acc exactly
    assert np.array_equal(native.epilogue(acc, one, zero), acc.astype(np.float32))
    scale = rng.standard_normal(6).astype(np.float32)
    bias = rng.standard_normal(6).astype(np.float32)
    y = native.epilogue(acc, scale, bias)
    exact = acc.astype(np.float64) * scale.astype(np.float64) + bias.astype(np.float64)
    assert np.array_equal(y, exact.astype(np.float32))   # one rounding: fma
    # residual term adds l_r + q_r * Delta_r
    res = rng.integers(0, 16, acc.shape, dtype=np.int8)
    yr = native.epilogue(acc, scale, bias, 0.0, None, res, -1.0, 0.25)
    want = y + (res.astype(np.float32) * np.float32(0.25) + np.float32(-1.0))
    assert np.array_equal(yr, want)
    # w_offset = 1/2 form against float64
    sa = rng.integers(0, 900, (3, 4, 4), dtype=np.int32)
    yh = native.epilogue(acc, scale, bias, 0.5, sa)
    exact = (acc + 0.5 * sa[..., None]) * scale.astype(np.float64) + bias
    assert np.allclose(yh, exact, rtol=1e-6, atol=1e-6)
    # max-pool commutes with the (monotone) quantiser
    yq = rng.standard_normal((2, 6, 8, 5)).astype(np.float32) * 2
    a = native.maxpool2x2(native.quantize(yq, 2, 0.0, 3.0))
    pooled = yq.reshape(2, 3, 2, 4, 2, 5).max(axis=(2, 4))
    assert np.array_equal(a, native.quantize(pooled, 2, 0.0, 3.0))
    # GEMM dequantisation is one multiply
    Cm = rng.integers(-10 ** 6, 10 ** 6, (5, 7), dtype=np.int32)
    rs = rng.uniform(0.5, 1.5, 5).astype(np.float32)
    assert np.array_equal(native.gemm_dequant(Cm, rs),
                          Cm.astype(np.float32) * rs[:, None])


def test_printed_table_values():
    here = __import__("os").path.dirname(__file__)
    for line in open(here + "/golden/table1_mla_per_saddw.txt"):
        if line.startswith("#") or not line.strip():
            continue
        b, ratio = map(int, line.split())
        assert native.mla_per_saddw(b) == ratio
    macs = set()
    for line in open(here + "/golden/table8_shapes.txt"):
        if line.startswith("#") or not line.strip():
            continue
        ci, h, w, co = map(int, line.split())
        act = np.ones((1, h, w, ci), np.int8)
        # MACs counted with padding taps included, as a dense rate would
        macs.add(h * w * co * ci * 9)
    assert macs == {115605504}


def test_tiny_stack_runs_and_is_not_degenerate():
    st = dsq_inputs.tiny_stack()
    x = dsq_inputs.stack_input(st, workload_id=9)
    params = dsq_inputs.stack_params(st, workload_id=9)
    out = stack.run_stack(st, x, params)
    for name, (H, W, C) in st.tensor_shapes().items():
        assert out[name].shape == (st.batch, H, W, C)
        assert out[name].min() >= 0 and out[name].max() <= 15
        assert len(np.unique(out[name])) > 4, name
