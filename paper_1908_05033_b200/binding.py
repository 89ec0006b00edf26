"""ctypes binding of libdsq_b200.so.

Two layers, both marshalling only:
  * `lib.<name>`: the raw C entry points with ctypes signatures, named exactly
    as in include/dsq.h;
  * functions of the same names taking torch CUDA tensors: they check dtypes,
    allocate the output tensors with torch, pass data pointers and the current
    CUDA stream, and raise DsqError on a non-zero status.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdsq_b200.so")

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with "
        "`python -m paper_1908_05033_b200.build` (needs nvcc; there is no "
        "fallback path)")
lib = C.CDLL(_LIB_PATH)


class dsq_quant_t(C.Structure):
    _fields_ = [("bits", C.c_int32), ("lo", C.c_float), ("hi", C.c_float)]


class dsq_nhwc_t(C.Structure):
    _fields_ = [("N", C.c_int32), ("H", C.c_int32), ("W", C.c_int32),
                ("C", C.c_int32)]


class dsq_conv_t(C.Structure):
    _fields_ = [("Cout", C.c_int32), ("KH", C.c_int32), ("KW", C.c_int32),
                ("Cin", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32),
                ("groups", C.c_int32)]


class dsq_epilogue_t(C.Structure):
    _fields_ = [("scale", C.c_void_p), ("bias", C.c_void_p),
                ("w_offset", C.c_float), ("residual_codes", C.c_void_p),
                ("residual_q", dsq_quant_t), ("requant", dsq_quant_t)]


_vp, _i64, _int, _sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
_SIGNATURES = {
    "dsq_row_pitch": (_sz, [_i64, _int]),
    "dsq_packed_bytes": (_sz, [_i64, _i64, _int]),
    "dsq_weight_bytes": (_sz, [C.POINTER(dsq_conv_t), _int]),
    "dsq_workspace_bytes": (_sz, []),
    "dsq_workspace_init": (_int, [_vp, _sz, _vp]),
    "dsq_workspace_status": (_int, [_vp, _vp]),
    "dsq_pack_weights": (_int, [_vp, C.POINTER(dsq_conv_t), _int, _vp, _vp,
                                _int, _vp, _sz, _vp, _sz, _vp]),
    "dsq_quantize_act": (_int, [_vp, C.POINTER(dsq_nhwc_t),
                                C.POINTER(dsq_quant_t), _vp, _sz, _vp]),
    "dsq_conv2d": (_int, [_vp, C.POINTER(dsq_nhwc_t), C.POINTER(dsq_quant_t),
                          _vp, C.POINTER(dsq_conv_t),
                          C.POINTER(dsq_epilogue_t), _vp, _vp, _vp, _vp, _sz,
                          _vp]),
    "dsq_dwconv2d": (_int, [_vp, C.POINTER(dsq_nhwc_t),
                            C.POINTER(dsq_quant_t), _vp,
                            C.POINTER(dsq_conv_t), C.POINTER(dsq_epilogue_t),
                            _vp, _vp, _vp, _vp]),
    "dsq_gemm": (_int, [_vp, _vp, _i64, _i64, _i64, _int, _vp, _vp, _vp, _vp,
                        _sz, _vp]),
    "dsq_gemm_workspace_bytes": (_sz, [_i64, _i64, _i64, _int]),
    "dsq_binary_gemm_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "dsq_binary_gemm": (_int, [_vp, _vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _sz, _vp]),
    "dsq_wgemm_workspace_bytes": (_sz, [_i64, _i64]),
    "dsq_wgemm_bf16": (_int, [_vp, _vp, _i64, _i64, _i64, _int, C.c_float, _vp, _vp, _vp, _vp,
                              _sz, _vp]),
    "dsq_gemm_static_ws": (_int, [_vp, _vp, _i64, _i64, _i64, _int, _vp, _vp, _vp,
                                  _int, _vp]),
    "dsq_maxpool2x2": (_int, [_vp, C.POINTER(dsq_nhwc_t), _int, _vp, _sz,
                              _vp]),
    "dsq_soft_quantize_fwd": (_int, [_vp, _i64, C.POINTER(dsq_quant_t), C.c_float, _vp, _vp]),
    "dsq_soft_quantize_bwd": (_int, [_vp, _vp, _i64, C.POINTER(dsq_quant_t), C.c_float, _vp,
                                     _vp, _vp]),
    "dsq_pack_codes": (_int, [_vp, _i64, _i64, _int, _vp, _sz, _vp]),
    "dsq_unpack": (_int, [_vp, _i64, _i64, _int, _int, _vp, _vp]),
    "dsq_probe_i8_mma_rate": (_int, [_int, C.POINTER(C.c_float),
                                     C.POINTER(C.c_double), _vp, _sz, _vp]),
    "dsq_status_string": (C.c_char_p, [_int]),
    "dsq_version": (_int, []),
}
# tuning / test hooks (csrc/dsq_hooks.h; not part of include/dsq.h)
_HOOKS = {
    "dsq_set_tile_n": (_int, [_int]),
    "dsq_set_round_k_steps": (_int, [_int]),
    "dsq_set_cta_pairs": (_int, [_int]),
    "dsq_set_dependent_launch": (_int, [_int]),
    "dsq_set_wait_limit_ns": (_int, [C.c_longlong]),
    "dsq_set_test_skip_b_round": (_int, [_int]),
    "dsq_set_conv3_window": (_int, [_int]),
    "dsq_set_gemm_two_pass": (_int, [_int]),
    "dsq_set_conv3_expanded_weights": (_int, [_int]),
}
for _name, (_res, _args) in list(_SIGNATURES.items()) + list(_HOOKS.items()):
    _f = getattr(lib, _name)       # AttributeError if a symbol is missing
    _f.restype, _f.argtypes = _res, _args

EXPORTED_SYMBOLS = tuple(_SIGNATURES)
HOOK_SYMBOLS = tuple(_HOOKS)


class DsqError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib.dsq_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


def _check(status, where):
    if status != 0:
        raise DsqError(status, where)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _need(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype
            and t.is_contiguous()):
        raise TypeError(f"{name}: want a contiguous CUDA tensor of {dtype}")
    return t


# ---- sizes ------------------------------------------------------------------
def dsq_row_pitch(k, bits):
    return int(lib.dsq_row_pitch(k, bits))


def dsq_packed_bytes(rows, k, bits):
    return int(lib.dsq_packed_bytes(rows, k, bits))


def dsq_weight_bytes(conv, bits):
    return int(lib.dsq_weight_bytes(C.byref(conv), bits))


def dsq_workspace_bytes():
    return int(lib.dsq_workspace_bytes())


def dsq_version():
    return int(lib.dsq_version())


def dsq_status_string(status):
    return lib.dsq_status_string(status).decode()


# ---- workspace ----------------------------------------------------------------
def new_workspace(device="cuda"):
    ws = torch.empty(dsq_workspace_bytes(), dtype=torch.uint8, device=device)
    _check(lib.dsq_workspace_init(_p(ws), ws.numel(), _stream()),
           "dsq_workspace_init")
    return ws


def dsq_gemm_workspace_bytes(M, N, K, bits):
    return int(lib.dsq_gemm_workspace_bytes(M, N, K, bits))


def new_gemm_workspace(M, N, K, bits, device="cuda"):
    """Workspace with room for the expanded operands of an M x N x K GEMM (the
    two-pass path of dsq_gemm); the status words in front are cleared."""
    ws = torch.empty(dsq_gemm_workspace_bytes(M, N, K, bits), dtype=torch.uint8, device=device)
    _check(lib.dsq_workspace_init(_p(ws), ws.numel(), _stream()),
           "dsq_workspace_init")
    return ws


def dsq_workspace_status(ws):
    return int(lib.dsq_workspace_status(_p(ws), _stream()))


def check_workspace(ws, where="kernel"):
    _check(dsq_workspace_status(ws), where)


# ---- format helpers -----------------------------------------------------------
def dsq_pack_codes(codes, bits):
    """int8 [rows, k] -> uint8 [rows, pitch] packed rows."""
    _need(codes, torch.int8, "codes")
    rows, k = codes.shape
    pitch = dsq_row_pitch(k, bits)
    out = torch.empty((rows, pitch), dtype=torch.uint8, device=codes.device)
    _check(lib.dsq_pack_codes(_p(codes), rows, k, bits, _p(out), out.numel(),
                              _stream()), "dsq_pack_codes")
    return out


def dsq_unpack(packed, rows, k, bits, signed):
    """packed rows -> int8 [rows, k]."""
    _need(packed, torch.uint8, "packed")
    out = torch.empty((rows, k), dtype=torch.int8, device=packed.device)
    _check(lib.dsq_unpack(_p(packed), rows, k, bits, int(signed), _p(out),
                          _stream()), "dsq_unpack")
    return out


# ---- quantise -----------------------------------------------------------------
def dsq_quantize_act(x, bits, lo, hi, out=None):
    """fp32 NHWC [N,H,W,C] -> packed codes uint8 [N,H,W,pitch]."""
    _need(x, torch.float32, "x")
    N, H, W, Cc = x.shape
    pitch = dsq_row_pitch(Cc, bits)
    if out is None:
        out = torch.empty((N, H, W, pitch), dtype=torch.uint8, device=x.device)
    shape = dsq_nhwc_t(N, H, W, Cc)
    q = dsq_quant_t(bits, lo, hi)
    _check(lib.dsq_quantize_act(_p(x), C.byref(shape), C.byref(q), _p(out),
                                out.numel(), _stream()), "dsq_quantize_act")
    return out


def dsq_pack_weights(w, bits, lo, hi, ws, depthwise=False, stride=1, pad=0):
    """fp32 weights [Cout,KH,KW,Cin] (or [C,KH,KW] depthwise) + clip bounds
    (python floats, or fp32 CUDA tensors of Cout elements) -> (blob, conv)."""
    _need(w, torch.float32, "w")
    if depthwise:
        Cout, KH, KW = w.shape
        Cin, groups = Cout, Cout
    else:
        Cout, KH, KW, Cin = w.shape
        groups = 1
    conv = dsq_conv_t(Cout, KH, KW, Cin, stride, pad, groups)

    def bound(v):
        if isinstance(v, torch.Tensor):
            return _need(v, torch.float32, "clip bound")
        return torch.tensor([float(v)], dtype=torch.float32, device=w.device)

    lo_t, hi_t = bound(lo), bound(hi)
    per_channel = int(lo_t.numel() > 1)
    if per_channel and (lo_t.numel() != Cout or hi_t.numel() != Cout):
        raise ValueError("per-channel clip bounds need Cout elements")
    nbytes = dsq_weight_bytes(conv, bits)
    blob = torch.empty(nbytes, dtype=torch.uint8, device=w.device)
    _check(lib.dsq_pack_weights(_p(w), C.byref(conv), bits, _p(lo_t), _p(hi_t),
                                per_channel, _p(blob), nbytes, _p(ws),
                                ws.numel(), _stream()), "dsq_pack_weights")
    return blob, conv


# ---- convolution ----------------------------------------------------------------
def _epilogue(scale, bias, w_offset, residual, residual_q, requant):
    ep = dsq_epilogue_t()
    ep.scale = scale.data_ptr()
    ep.bias = bias.data_ptr()
    ep.w_offset = w_offset
    ep.residual_codes = residual.data_ptr() if residual is not None else None
    if residual_q is not None:
        ep.residual_q = dsq_quant_t(*residual_q)
    if requant is not None:
        ep.requant = dsq_quant_t(*requant)
    return ep


def _conv_common(fn_name, act, shape, act_q, blob, conv, scale, bias, w_offset,
                 residual, residual_q, requant, want_f32, want_acc, ws,
                 out_codes):
    _need(act, torch.uint8, "act")
    _need(blob, torch.uint8, "weights")
    _need(scale, torch.float32, "scale")
    _need(bias, torch.float32, "bias")
    N, H, W, Cc = shape
    bits = act_q[0]
    Ho = (H + 2 * conv.pad - conv.KH) // conv.stride + 1
    Wo = (W + 2 * conv.pad - conv.KW) // conv.stride + 1
    dev = act.device
    y = torch.empty((N, Ho, Wo, conv.Cout), dtype=torch.float32,
                    device=dev) if want_f32 else None
    acc = torch.empty((N, Ho, Wo, conv.Cout), dtype=torch.int32,
                      device=dev) if want_acc else None
    codes = None
    if requant is not None:
        codes = out_codes if out_codes is not None else torch.empty(
            (N, Ho, Wo, dsq_row_pitch(conv.Cout, bits)), dtype=torch.uint8,
            device=dev)
    ep = _epilogue(scale, bias, w_offset, residual, residual_q, requant)
    nhwc = dsq_nhwc_t(N, H, W, Cc)
    aq = dsq_quant_t(*act_q)
    if fn_name == "dsq_conv2d":
        st = lib.dsq_conv2d(_p(act), C.byref(nhwc), C.byref(aq), _p(blob),
                            C.byref(conv), C.byref(ep), _p(y), _p(codes),
                            _p(acc), _p(ws), ws.numel(), _stream())
    else:
        st = lib.dsq_dwconv2d(_p(act), C.byref(nhwc), C.byref(aq), _p(blob),
                              C.byref(conv), C.byref(ep), _p(y), _p(codes),
                              _p(acc), _stream())
    _check(st, fn_name)
    return codes, y, acc


def dsq_conv2d(act, shape, act_q, blob, conv, scale, bias, ws, w_offset=0.0,
               residual=None, residual_q=None, requant=None, want_f32=False,
               want_acc=False, out_codes=None):
    """act: packed codes of NHWC `shape`; act_q / residual_q / requant are
    (bits, lo, hi) tuples.  Returns (codes | None, y_f32 | None, acc | None)."""
    return _conv_common("dsq_conv2d", act, shape, act_q, blob, conv, scale,
                        bias, w_offset, residual, residual_q, requant,
                        want_f32, want_acc, ws, out_codes)


def dsq_dwconv2d(act, shape, act_q, blob, conv, scale, bias, w_offset=0.0,
                 residual=None, residual_q=None, requant=None, want_f32=False,
                 want_acc=False, out_codes=None):
    return _conv_common("dsq_dwconv2d", act, shape, act_q, blob, conv, scale,
                        bias, w_offset, residual, residual_q, requant,
                        want_f32, want_acc, None, out_codes)


def dsq_maxpool2x2(codes, shape, bits, out=None):
    _need(codes, torch.uint8, "codes")
    N, H, W, Cc = shape
    pitch = dsq_row_pitch(Cc, bits)
    if out is None:
        out = torch.empty((N, H // 2, W // 2, pitch), dtype=torch.uint8,
                          device=codes.device)
    nhwc = dsq_nhwc_t(N, H, W, Cc)
    _check(lib.dsq_maxpool2x2(_p(codes), C.byref(nhwc), bits, _p(out),
                              out.numel(), _stream()), "dsq_maxpool2x2")
    return out


# ---- training side: soft quantiser -----------------------------------------------
def dsq_soft_quantize_fwd(x, bits, lo, hi, alpha, out=None):
    """y = Q_S(x) (Eq. 5), fp32 CUDA tensor of any shape."""
    _need(x, torch.float32, "x")
    y = out if out is not None else torch.empty_like(x)
    q = dsq_quant_t(bits, lo, hi)
    _check(lib.dsq_soft_quantize_fwd(_p(x), x.numel(), C.byref(q), alpha, _p(y), _stream()),
           "dsq_soft_quantize_fwd")
    return y


def dsq_soft_quantize_bwd(x, grad_y, bits, lo, hi, alpha, out=None, grad_params=None):
    """Returns (grad_x fp32 like x, grad_params fp64 [3] = dL/d(alpha, l, u))."""
    _need(x, torch.float32, "x")
    _need(grad_y, torch.float32, "grad_y")
    gx = out if out is not None else torch.empty_like(x)
    gp = grad_params if grad_params is not None else torch.empty(
        3, dtype=torch.float64, device=x.device)
    q = dsq_quant_t(bits, lo, hi)
    _check(lib.dsq_soft_quantize_bwd(_p(x), _p(grad_y), x.numel(), C.byref(q), alpha, _p(gx),
                                     _p(gp), _stream()), "dsq_soft_quantize_bwd")
    return gx, gp


# ---- GEMM -------------------------------------------------------------------------
def dsq_gemm(A, B, M, N, K, bits, ws, row_scale=None, want_i32=True,
             out_i32=None, out_f32=None):
    """A: packed signed codes [M, pitch], B: packed unsigned codes [N, pitch].
    Returns (C int32 [M,N] | None, D fp32 [M,N] | None)."""
    _need(A, torch.uint8, "A")
    _need(B, torch.uint8, "B")
    Cm = out_i32
    if Cm is None and want_i32:
        Cm = torch.empty((M, N), dtype=torch.int32, device=A.device)
    D = out_f32
    if D is None and row_scale is not None:
        D = torch.empty((M, N), dtype=torch.float32, device=A.device)
    _check(lib.dsq_gemm(_p(A), _p(B), M, N, K, bits, _p(Cm), _p(row_scale),
                        _p(D), _p(ws), ws.numel(), _stream()), "dsq_gemm")
    return Cm, D


def _sized_workspace(nbytes, device):
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    _check(lib.dsq_workspace_init(_p(ws), ws.numel(), _stream()), "dsq_workspace_init")
    return ws


def dsq_binary_gemm(A, B, M, N, K, ws=None, row_scale=None, want_i32=True):
    """A, B: packed 1-bit rows [M, pitch], [N, pitch] (bit 1 = +1, 0 = -1).
    Returns (C int32 [M,N] | None, D fp32 [M,N] | None)."""
    _need(A, torch.uint8, "A")
    _need(B, torch.uint8, "B")
    if ws is None:
        ws = _sized_workspace(int(lib.dsq_binary_gemm_workspace_bytes(M, N, K)), A.device)
    Cm = torch.empty((M, N), dtype=torch.int32, device=A.device) if want_i32 else None
    D = torch.empty((M, N), dtype=torch.float32, device=A.device) if row_scale is not None else None
    _check(lib.dsq_binary_gemm(_p(A), _p(B), M, N, K, _p(Cm), _p(row_scale), _p(D), _p(ws),
                               ws.numel(), _stream()), "dsq_binary_gemm")
    check_workspace(ws, "dsq_binary_gemm")
    return Cm, D


def dsq_wgemm_bf16(X, W, M, N, K, bits, col_scale, col_bias=None, w_offset=0.5, ws=None,
                   out=None):
    """X: bf16 [M, K]; W: packed signed codes [N, pitch].  Returns Y fp32 [M, N]."""
    _need(X, torch.bfloat16, "X")
    _need(W, torch.uint8, "W")
    _need(col_scale, torch.float32, "col_scale")
    if ws is None:
        ws = _sized_workspace(int(lib.dsq_wgemm_workspace_bytes(N, K)), X.device)
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float32, device=X.device)
    _check(lib.dsq_wgemm_bf16(_p(X), _p(W), M, N, K, bits, w_offset, _p(col_scale),
                              _p(col_bias), _p(Y), _p(ws), ws.numel(), _stream()),
           "dsq_wgemm_bf16")
    return Y


def dsq_set_round_k_steps(ks):
    _check(lib.dsq_set_round_k_steps(ks), "dsq_set_round_k_steps")


def dsq_set_conv3_expanded_weights(on):
    _check(lib.dsq_set_conv3_expanded_weights(int(on)), "dsq_set_conv3_expanded_weights")


def dsq_set_gemm_two_pass(on):
    _check(lib.dsq_set_gemm_two_pass(int(on)), "dsq_set_gemm_two_pass")


def dsq_set_cta_pairs(mode):
    _check(lib.dsq_set_cta_pairs(mode), "dsq_set_cta_pairs")


def dsq_set_wait_limit_ns(ns):
    """Test hook: limit of the kernels' barrier waits (0 = default 2 s)."""
    _check(lib.dsq_set_wait_limit_ns(int(ns)), "dsq_set_wait_limit_ns")


def dsq_set_test_skip_b_round(r):
    """Test hook: the B producer leaves out round r (-1 = off)."""
    _check(lib.dsq_set_test_skip_b_round(int(r)), "dsq_set_test_skip_b_round")


def dsq_set_conv3_window(mode):
    _check(lib.dsq_set_conv3_window(int(mode)), "dsq_set_conv3_window")


def dsq_set_dependent_launch(on):
    _check(lib.dsq_set_dependent_launch(on), "dsq_set_dependent_launch")


def dsq_set_tile_n(bn):
    _check(lib.dsq_set_tile_n(bn), "dsq_set_tile_n")


def dsq_gemm_static_ws(A, B, M, N, K, bits, out_i32=None, row_scale=None,
                       out_f32=None, wait_and_check=True):
    """dsq_gemm without a caller workspace (the library's own 256-byte static
    array is the scratch).  The caller passes the outputs; nothing is
    allocated here.  Returns the status of the call."""
    _need(A, torch.uint8, "A")
    _need(B, torch.uint8, "B")
    st = lib.dsq_gemm_static_ws(_p(A), _p(B), M, N, K, bits, _p(out_i32),
                                _p(row_scale), _p(out_f32),
                                int(wait_and_check), _stream())
    _check(st, "dsq_gemm_static_ws")
    return st


# ---- measurement ------------------------------------------------------------------
def dsq_probe_i8_mma_rate(iters, ws):
    """Returns (TOPS, ms) of the MMA-only probe."""
    ms, macs = C.c_float(), C.c_double()
    _check(lib.dsq_probe_i8_mma_rate(iters, C.byref(ms), C.byref(macs), _p(ws),
                                     ws.numel(), _stream()),
           "dsq_probe_i8_mma_rate")
    return 2.0 * macs.value / (ms.value * 1e-3) / 1e12, ms.value


__all__ = [n for n in dir() if n.startswith("dsq_")] + [
    "lib", "DsqError", "EXPORTED_SYMBOLS", "HOOK_SYMBOLS", "new_workspace",
    "new_gemm_workspace",
    "check_workspace"]
