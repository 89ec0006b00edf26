"""Run a whole layer stack through the CPU oracle (TEST INFRASTRUCTURE ONLY).

Each layer is Algorithm 1's feed-forward pass in its deployed form: the input
codes and the weight codes are contracted in integers, the accumulator is
dequantised with scale = Delta_a * Delta_w (per output channel when the weight
clip is per channel) and the weight-grid offset w_offset, the bias and the
optional residual are added, and the result is requantised with the output
tensor's range (the next layer's steps 1 and 3).
"""
import numpy as np

from . import native


def delta_f32(bits, lo, hi):
    """Interval length as the binary32 value (hi - lo) / (2^b - 1)."""
    return (np.float32(hi) - np.float32(lo)) / np.float32(2 ** bits - 1)


def layer_scale(bits, act_lo, act_hi, w_lo, w_hi, cout):
    """scale[co] = Delta_a * Delta_w[co], binary32."""
    da = delta_f32(bits, act_lo, act_hi)
    w_lo = np.broadcast_to(np.asarray(w_lo, np.float32), (cout,))
    w_hi = np.broadcast_to(np.asarray(w_hi, np.float32), (cout,))
    dw = ((w_hi - w_lo) / np.float32(2 ** bits - 1)).astype(np.float32)
    return (da * dw).astype(np.float32)


def run_stack(st, x, params, w_offset=0.5, keep=None):
    """st: dsq_inputs.Stack; x: fp32 NHWC input; params: dsq_inputs.stack_params.
    Returns {tensor name: int8 codes NHWC} for every tensor (or those in
    `keep`), plus "acc:<layer>" int32 accumulators and "y:<layer>" fp32
    pre-requantisation outputs when keep is None."""
    bits = st.bits
    t = {"in": native.quantize(x, bits, st.in_lo, st.in_hi)}
    rng = {"in": (st.in_lo, st.in_hi)}
    extra = {}
    for L in st.layers:
        src = t[L.src]
        if L.kind == "pool":
            t[L.dst] = native.maxpool2x2(src)
            rng[L.dst] = rng[L.src]
            continue
        p = params[L.name]
        a_lo, a_hi = rng[L.src]
        per_ch = p["w_hi"].size > 1
        wc = native.quantize_weights(p["w"], bits, p["w_lo"], p["w_hi"],
                                     per_row=per_ch)
        if L.kind == "dw":
            acc, sa = native.dwconv2d(src, wc, L.stride, L.pad, want_sa=True)
        else:
            acc, sa = native.conv2d(src, wc, L.stride, L.pad, want_sa=True)
        scale = layer_scale(bits, a_lo, a_hi, p["w_lo"], p["w_hi"], L.cout)
        res = res_lo = res_d = None
        if L.residual is not None:
            res = t[L.residual]
            r_lo, r_hi = rng[L.residual]
            res_lo, res_d = np.float32(r_lo), delta_f32(bits, r_lo, r_hi)
        y = native.epilogue(acc, scale, p["bias"], w_offset,
                            sa if w_offset != 0.0 else None, res,
                            res_lo or 0.0, res_d or 0.0)
        t[L.dst] = native.quantize(y, bits, L.out_lo, L.out_hi)
        rng[L.dst] = (L.out_lo, L.out_hi)
        if keep is None:
            extra["acc:" + L.name] = acc
            extra["y:" + L.name] = y
    if keep is not None:
        return {k: t[k] for k in keep}
    t.update(extra)
    return t
