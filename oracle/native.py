"""ctypes binding of dsq_oracle.c (TEST INFRASTRUCTURE ONLY).

Every function takes and returns numpy arrays; shapes follow the C source:
activations NHWC, weights [Cout][KH][KW][Cin], codes int8, accumulators int32.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_i64, _i32, _f32, _f64 = C.c_int64, C.c_int32, C.c_float, C.c_double
_p = C.c_void_p


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_p)


def _sig(name, res, *args):
    f = getattr(_lib, name)
    f.restype = res
    f.argtypes = list(args)
    return f


_num_threads = _sig("dsqo_num_threads", C.c_int)
_quantize_code = _sig("dsqo_quantize_code", _i32, _f32, C.c_int, _f32, _f32)
_quantize = _sig("dsqo_quantize", None, _p, _i64, C.c_int, _f32, _f32, _p)
_quantize_weights = _sig("dsqo_quantize_weights", None, _p, _i64, _i64,
                         C.c_int, _p, _p, C.c_int, _p)
_dequantize = _sig("dsqo_dequantize", None, _p, _i64, C.c_int, _f64, _f64, _p)
_row_pitch = _sig("dsqo_row_pitch", _i64, _i64, C.c_int)
_pack_rows = _sig("dsqo_pack_rows", None, _p, _i64, _i64, C.c_int, _p, _i64)
_unpack_rows = _sig("dsqo_unpack_rows", None, _p, _i64, _i64, C.c_int,
                    C.c_int, _i64, _p)
_gemm = _sig("dsqo_gemm", None, _p, _p, _i64, _i64, _i64, _p)
_conv2d = _sig("dsqo_conv2d", None, _p, _i64, _i64, _i64, _i64, _p, _i64,
               _i64, _i64, _i64, _i64, _p, _p)
_dwconv2d = _sig("dsqo_dwconv2d", None, _p, _i64, _i64, _i64, _i64, _p, _i64,
                 _i64, _i64, _i64, _p, _p)
_epilogue = _sig("dsqo_epilogue", None, _p, _p, C.c_int, _i64, _i64, _p, _p,
                 _f32, _p, _f32, _f32, _p)
_gemm_dequant = _sig("dsqo_gemm_dequant", None, _p, _i64, _i64, _p, _p)
_maxpool = _sig("dsqo_maxpool2x2", None, _p, _i64, _i64, _i64, _i64, _p)
_mla = _sig("dsqo_mla_per_saddw", _i32, C.c_int)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_num_threads())


def quantize_code(x: float, bits: int, lo: float, hi: float) -> int:
    return int(_quantize_code(x, bits, lo, hi))


def quantize(x, bits, lo, hi):
    """fp32 array -> unsigned codes (int8), same shape."""
    x = _c(x, np.float32)
    q = np.empty(x.shape, np.int8)
    _quantize(_ptr(x), x.size, bits, lo, hi, _ptr(q))
    return q


def quantize_weights(w, bits, lo, hi, per_row=False):
    """fp32 [rows, ...] -> signed codes c = q - 2^(b-1) (int8), same shape.
    lo/hi: scalars, or [rows] arrays when per_row."""
    w = _c(w, np.float32)
    rows = w.shape[0]
    k = w.size // rows
    lo = _c(np.broadcast_to(np.asarray(lo, np.float32),
                            (rows,) if per_row else (1,)), np.float32)
    hi = _c(np.broadcast_to(np.asarray(hi, np.float32),
                            (rows,) if per_row else (1,)), np.float32)
    c = np.empty(w.shape, np.int8)
    _quantize_weights(_ptr(w), rows, k, bits, _ptr(lo), _ptr(hi),
                      int(per_row), _ptr(c))
    return c


def dequantize(q, bits, lo, hi):
    q = _c(q, np.int8)
    out = np.empty(q.shape, np.float64)
    _dequantize(_ptr(q), q.size, bits, lo, hi, _ptr(out))
    return out


def row_pitch(k: int, bits: int) -> int:
    return int(_row_pitch(k, bits))


def pack_rows(codes, bits, pitch=None):
    """int8 [rows, k] -> uint8 [rows, pitch] dense little-endian bit stream."""
    codes = _c(codes, np.int8)
    rows, k = codes.shape
    if pitch is None:
        pitch = row_pitch(k, bits)
    out = np.empty((rows, pitch), np.uint8)
    _pack_rows(_ptr(codes), rows, k, bits, _ptr(out), pitch)
    return out


def unpack_rows(packed, k, bits, signed):
    packed = _c(packed, np.uint8)
    rows, pitch = packed.shape
    out = np.empty((rows, k), np.int8)
    _unpack_rows(_ptr(packed), rows, k, bits, int(signed), pitch, _ptr(out))
    return out


def gemm(A, B):
    """int8 A[M,K] (signed codes), B[N,K] (unsigned codes) -> int32 [M,N]."""
    A, B = _c(A, np.int8), _c(B, np.int8)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    out = np.empty((M, N), np.int32)
    _gemm(_ptr(A), _ptr(B), M, N, K, _ptr(out))
    return out


def conv_out_hw(H, W, KH, KW, stride, pad):
    return (H + 2 * pad - KH) // stride + 1, (W + 2 * pad - KW) // stride + 1


def conv2d(act, wgt, stride, pad, want_sa=False):
    """act int8 [N,H,W,Cin] unsigned codes, wgt int8 [Cout,KH,KW,Cin] signed
    codes -> acc int32 [N,Ho,Wo,Cout] (, sa int32 [N,Ho,Wo])."""
    act, wgt = _c(act, np.int8), _c(wgt, np.int8)
    N, H, W, Cin = act.shape
    Cout, KH, KW, Cin2 = wgt.shape
    assert Cin == Cin2
    Ho, Wo = conv_out_hw(H, W, KH, KW, stride, pad)
    acc = np.empty((N, Ho, Wo, Cout), np.int32)
    sa = np.empty((N, Ho, Wo), np.int32) if want_sa else None
    _conv2d(_ptr(act), N, H, W, Cin, _ptr(wgt), Cout, KH, KW, stride, pad,
            _ptr(acc), _ptr(sa))
    return (acc, sa) if want_sa else acc


def dwconv2d(act, wgt, stride, pad, want_sa=False):
    """act int8 [N,H,W,C], wgt int8 [C,KH,KW] -> acc int32 [N,Ho,Wo,C]
    (, sa int32 [N,Ho,Wo,C])."""
    act, wgt = _c(act, np.int8), _c(wgt, np.int8)
    N, H, W, Cc = act.shape
    C2, KH, KW = wgt.shape
    assert Cc == C2
    Ho, Wo = conv_out_hw(H, W, KH, KW, stride, pad)
    acc = np.empty((N, Ho, Wo, Cc), np.int32)
    sa = np.empty((N, Ho, Wo, Cc), np.int32) if want_sa else None
    _dwconv2d(_ptr(act), N, H, W, Cc, _ptr(wgt), KH, KW, stride, pad,
              _ptr(acc), _ptr(sa))
    return (acc, sa) if want_sa else acc


def epilogue(acc, scale, bias, w_offset=0.0, sa=None, residual=None,
             res_lo=0.0, res_delta=0.0):
    """acc int32 [..., Cout] -> fp32 y, same shape (pinned binary32 ops)."""
    acc = _c(acc, np.int32)
    cout = acc.shape[-1]
    rows = acc.size // cout
    scale, bias = _c(scale, np.float32), _c(bias, np.float32)
    assert scale.shape == (cout,) and bias.shape == (cout,)
    per_ch = 0
    if sa is not None:
        sa = _c(sa, np.int32)
        per_ch = int(sa.size == acc.size)
        assert per_ch or sa.size == rows
    if residual is not None:
        residual = _c(residual, np.int8)
        assert residual.size == acc.size
    y = np.empty(acc.shape, np.float32)
    _epilogue(_ptr(acc), _ptr(sa), per_ch, rows, cout, _ptr(scale),
              _ptr(bias), w_offset, _ptr(residual), res_lo, res_delta,
              _ptr(y))
    return y


def gemm_dequant(Cacc, row_scale):
    Cacc = _c(Cacc, np.int32)
    M, N = Cacc.shape
    row_scale = _c(row_scale, np.float32)
    D = np.empty((M, N), np.float32)
    _gemm_dequant(_ptr(Cacc), M, N, _ptr(row_scale), _ptr(D))
    return D


def maxpool2x2(q):
    q = _c(q, np.int8)
    N, H, W, Cc = q.shape
    out = np.empty((N, H // 2, W // 2, Cc), np.int8)
    _maxpool(_ptr(q), N, H, W, Cc, _ptr(out))
    return out


def mla_per_saddw(bits: int) -> int:
    return int(_mla(bits))
