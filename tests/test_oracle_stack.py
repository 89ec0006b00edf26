"""Pins of oracle/stack.py (run_stack, layer_scale) and of the GEMM
dequantisation against something other than themselves.

run_stack chains the integer layer (codes x codes -> int32 -> binary32
epilogue -> requantise).  Here every layer of a small network with every
kind of layer - convolution, strided convolution with a 1x1 shortcut whose
output range is symmetric, convolution with a residual operand, depthwise
convolution with per-channel weight clips, 1x1 projection, pool - is
recomputed as Algorithm 1 states it, in float64 and in real values:

    a^ = l_a + Delta_a q_a,  w^ = l_w + Delta_w q_w        (step 4)
    o  = Conv(w^, a^) + bias (+ residual^)                 (step 5)
    next codes = hard quantiser of o with the output range (steps 1, 3)

using the dequantiser and the float64 quantiser of oracle/soft.py, a
convolution written here with numpy slices, and the ranges as the layer list
declares them - none of run_stack's or layer_scale's arithmetic.  A wrong
source range, residual range, scale or offset in run_stack changes its codes
and fails the comparison.
"""
import numpy as np
import pytest

from oracle import native, soft, stack
import dsq_inputs


def conv_real(a, w, stride, pad):
    """float64 direct convolution, a [N,H,W,Ci], w [Co,k,k,Ci], zero padding."""
    N, H, W, Ci = a.shape
    Co, k, _, _ = w.shape
    Ho = (H + 2 * pad - k) // stride + 1
    Wo = (W + 2 * pad - k) // stride + 1
    ap = np.zeros((N, H + 2 * pad, W + 2 * pad, Ci))
    ap[:, pad:pad + H, pad:pad + W] = a
    out = np.zeros((N, Ho, Wo, Co))
    for kh in range(k):
        for kw in range(k):
            win = ap[:, kh:kh + stride * (Ho - 1) + 1:stride,
                     kw:kw + stride * (Wo - 1) + 1:stride]
            out += np.einsum("nhwc,oc->nhwo", win, w[:, kh, kw])
    return out


def dwconv_real(a, w, stride, pad):
    N, H, W, C = a.shape
    k = w.shape[1]
    Ho = (H + 2 * pad - k) // stride + 1
    Wo = (W + 2 * pad - k) // stride + 1
    ap = np.zeros((N, H + 2 * pad, W + 2 * pad, C))
    ap[:, pad:pad + H, pad:pad + W] = a
    out = np.zeros((N, Ho, Wo, C))
    for kh in range(k):
        for kw in range(k):
            win = ap[:, kh:kh + stride * (Ho - 1) + 1:stride,
                     kw:kw + stride * (Wo - 1) + 1:stride]
            out += win * w[:, kh, kw]
    return out


def declared_ranges(st):
    """(lo, hi) of every code tensor, read off the layer list alone."""
    r = {"in": (st.in_lo, st.in_hi)}
    for L in st.layers:
        r[L.dst] = r[L.src] if L.kind == "pool" else (L.out_lo, L.out_hi)
    return r


@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("w_offset", [0.0, 0.5])
def test_run_stack_equals_the_real_valued_chain_layer_by_layer(bits, w_offset):
    st = dsq_inputs.tiny_stack(bits=bits)
    x = dsq_inputs.stack_input(st, workload_id=9)
    params = dsq_inputs.stack_params(st, workload_id=9)
    got = stack.run_stack(st, x, params, w_offset=w_offset)
    ranges = declared_ranges(st)
    half = 2 ** (bits - 1)
    # the input codes are the hard quantiser of the fp32 input
    d_in = soft.delta(bits, st.in_lo, st.in_hi)
    q_in = np.rint((soft.q_uniform(x.astype(np.float64), bits, st.in_lo, st.in_hi)
                    - st.in_lo) / d_in)
    t_in = (np.clip(x.astype(np.float64), st.in_lo, st.in_hi) - st.in_lo) / d_in + 0.5
    away = np.abs(t_in - np.rint(t_in)) > 1e-4
    assert np.array_equal(q_in[away], got["in"][away])
    checked = total = 0
    for L in st.layers:
        src = got[L.src]                       # this layer's input codes
        a_lo, a_hi = ranges[L.src]
        if L.kind == "pool":
            N_, H, W, C = src.shape
            want = src.reshape(N_, H // 2, 2, W // 2, 2, C).max(axis=(2, 4))
            assert np.array_equal(got[L.dst], want)
            continue
        p = params[L.name]
        a_hat = native.dequantize(src, bits, a_lo, a_hi)
        # weight codes: Algorithm 1 steps 1, 3 on w, per output channel
        w = p["w"].astype(np.float64)
        lo = np.broadcast_to(p["w_lo"].astype(np.float64), (L.cout,))
        hi = np.broadcast_to(p["w_hi"].astype(np.float64), (L.cout,))
        w_hat = np.empty_like(w)
        for co in range(L.cout):
            wq = soft.q_uniform(w[co], bits, lo[co], hi[co])     # l_w + Delta_w q_w
            if w_offset == 0.5:
                w_hat[co] = wq                                   # the paper's grid
            else:
                # plain form: w^ = Delta_w * c with c = q_w - 2^(b-1)
                dw = (hi[co] - lo[co]) / (2 ** bits - 1)
                w_hat[co] = np.rint((wq - lo[co]) / dw - half) * dw
        if L.kind == "dw":
            o = dwconv_real(a_hat, w_hat, L.stride, L.pad)
        else:
            o = conv_real(a_hat, w_hat, L.stride, L.pad)
        o = o + p["bias"].astype(np.float64)
        if L.residual is not None:
            r_lo, r_hi = ranges[L.residual]
            o = o + native.dequantize(got[L.residual], bits, r_lo, r_hi)
        d_out = soft.delta(bits, L.out_lo, L.out_hi)
        want = np.rint((soft.q_uniform(o, bits, L.out_lo, L.out_hi) - L.out_lo) / d_out)
        # binary32 and binary64 may part ways within a hair of a midpoint
        t = (np.clip(o, L.out_lo, L.out_hi) - L.out_lo) / d_out + 0.5
        away = np.abs(t - np.rint(t)) > 2e-5
        assert away.mean() > 0.97, L.name
        assert np.array_equal(want[away], got[L.dst][away].astype(np.float64)), L.name
        # ... and there only by one code
        assert np.abs(want - got[L.dst]).max() <= 1, L.name
        checked += int(away.sum())
        total += away.size
    assert checked > 0.98 * total


def test_run_stack_pin_detects_a_wrong_range():
    """The pin is sharp: the same comparison fails when the chain is fed a
    wrong source range (what a slip in run_stack would amount to)."""
    st = dsq_inputs.tiny_stack(bits=4)
    x = dsq_inputs.stack_input(st, workload_id=9)
    params = dsq_inputs.stack_params(st, workload_id=9)
    got = stack.run_stack(st, x, params)
    L = st.layers[2]                           # strided conv reading c1 (range [0, 2.5])
    p = params[L.name]
    w_hat = soft.q_uniform(p["w"].astype(np.float64), 4, float(p["w_lo"][0]), float(p["w_hi"][0]))
    for a_hi, must_match in ((2.5, True), (2.0, False)):
        a_hat = native.dequantize(got[L.src], 4, 0.0, a_hi)
        o = conv_real(a_hat, w_hat, L.stride, L.pad) + p["bias"].astype(np.float64)
        d_out = soft.delta(4, L.out_lo, L.out_hi)
        want = np.rint((soft.q_uniform(o, 4, L.out_lo, L.out_hi) - L.out_lo) / d_out)
        same = np.mean(want == got[L.dst])
        assert (same > 0.99) == must_match


def test_layer_scale_values():
    # Delta_a * Delta_w in binary32, hand-computed: (3-0)/15 * (0.3+0.3)/15
    s = stack.layer_scale(4, 0.0, 3.0, np.float32(-0.3), np.float32(0.3), 2)
    da = np.float32(3.0) / np.float32(15)
    dw = (np.float32(0.3) - np.float32(-0.3)) / np.float32(15)
    assert s.dtype == np.float32 and s.shape == (2,)
    assert s[0] == np.float32(da * dw) and abs(float(s[0]) - 0.2 * 0.04) < 1e-9
    # per channel, 2-bit: (6-0)/3 * [(1+1)/3, (2+2)/3]
    s = stack.layer_scale(2, 0.0, 6.0, np.array([-1, -2], np.float32),
                          np.array([1, 2], np.float32), 2)
    assert np.allclose(s, [2.0 * 2 / 3, 2.0 * 4 / 3], rtol=1e-6)


def test_gemm_dequant_hand_computed():
    """D = (float)C * row_scale[m]: products worked out by hand, including one
    where the int32 -> binary32 conversion rounds first (2^24 + 1 -> 2^24)."""
    Cm = np.array([[3, -7], [16777217, 1000]], np.int32)
    rs = np.array([0.5, 1.5 * 2.0 ** -10], np.float32)
    D = native.gemm_dequant(Cm, rs)
    assert D.dtype == np.float32
    assert D[0, 0] == np.float32(1.5) and D[0, 1] == np.float32(-3.5)
    assert D[1, 0] == np.float32(16777216.0 * 1.5 * 2.0 ** -10)      # 24576.0
    assert D[1, 1] == np.float32(1.46484375)
