"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every symbol include/dsq.h declares, its size queries agree with the format
definition, and argument validation returns the documented status codes
before anything is launched."""
import ctypes as C
import os
import re

import pytest

import paper_1908_05033_b200 as dsq
from paper_1908_05033_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions(path=("include", "dsq.h")):
    text = open(os.path.join(ROOT, *path)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = declared_functions()
    assert "dsq_conv2d" in names and "dsq_gemm" in names and \
        "dsq_quantize_act" in names and "dsq_pack_weights" in names and \
        "dsq_dwconv2d" in names
    for n in names:
        assert hasattr(dsq.lib, n), n
    assert set(names) == set(B.EXPORTED_SYMBOLS)
    # the tuning / test hooks live in an internal header, not in include/dsq.h
    hooks = declared_functions(("paper_1908_05033_b200", "csrc", "dsq_hooks.h"))
    assert set(hooks) == set(B.HOOK_SYMBOLS) and not set(hooks) & set(names)
    for n in hooks:
        assert hasattr(dsq.lib, n), n


def test_size_queries():
    assert dsq.dsq_row_pitch(64, 4) == 32
    assert dsq.dsq_row_pitch(144, 4) == 80
    assert dsq.dsq_row_pitch(64, 2) == 16
    assert dsq.dsq_row_pitch(4096, 3) == 1536
    assert dsq.dsq_row_pitch(0, 4) == 0
    assert dsq.dsq_packed_bytes(10, 64, 4) == 320
    conv = B.dsq_conv_t(64, 3, 3, 64, 1, 1, 1)
    # config 1: 18432 bytes of packed rows + (3x3, stride 1, pad 1 only) the rows
    # expanded to int8, 5 K steps of 128 bytes each
    assert dsq.dsq_weight_bytes(conv, 4) == 64 * 9 * 32 + 64 * 5 * 128
    assert dsq.dsq_weight_bytes(B.dsq_conv_t(64, 3, 3, 64, 2, 1, 1), 4) == 64 * 9 * 32
    assert dsq.dsq_weight_bytes(B.dsq_conv_t(64, 3, 3, 64, 1, 1, 1), 3) == 64 * 9 * 32
    assert dsq.dsq_weight_bytes(B.dsq_conv_t(128, 3, 3, 256, 1, 1, 1), 2) == \
        128 * 9 * 64 + 128 * 18 * 128
    dw = B.dsq_conv_t(96, 3, 3, 96, 1, 1, 96)
    assert dsq.dsq_weight_bytes(dw, 4) == 9 * 48
    assert dsq.dsq_workspace_bytes() >= 16
    assert dsq.dsq_version() >= 100
    assert "aligned" in dsq.dsq_status_string(-2)


def test_validation_status_codes_without_a_gpu():
    lib = dsq.lib
    fake = C.c_void_p(0x1000)          # aligned, never dereferenced
    odd = C.c_void_p(0x1004)
    shape = B.dsq_nhwc_t(1, 8, 8, 64)
    q4 = B.dsq_quant_t(4, 0.0, 2.0)
    # NULL
    assert lib.dsq_quantize_act(None, C.byref(shape), C.byref(q4), fake, 1 << 20, None) == -1
    # bits
    q9 = B.dsq_quant_t(9, 0.0, 2.0)
    assert lib.dsq_quantize_act(fake, C.byref(shape), C.byref(q9), fake, 1 << 20, None) == -3
    # range: hi <= lo, NaN
    for lo, hi in [(1.0, 1.0), (2.0, 1.0), (float("nan"), 1.0), (0.0, float("inf"))]:
        qb = B.dsq_quant_t(4, lo, hi)
        assert lib.dsq_quantize_act(fake, C.byref(shape), C.byref(qb), fake, 1 << 20, None) == -6
    # shape
    bad = B.dsq_nhwc_t(1, 0, 8, 64)
    assert lib.dsq_quantize_act(fake, C.byref(bad), C.byref(q4), fake, 1 << 20, None) == -4
    # alignment
    assert lib.dsq_quantize_act(odd, C.byref(shape), C.byref(q4), fake, 1 << 20, None) == -2
    # size
    assert lib.dsq_quantize_act(fake, C.byref(shape), C.byref(q4), fake, 100, None) == -5

    # gemm
    assert lib.dsq_gemm(fake, fake, 128, 128, 128, 4, None, None, None, fake, 256, None) == -1
    assert lib.dsq_gemm(fake, fake, 128, 128, 128, 5, fake, None, None, fake, 256, None) == -3
    assert lib.dsq_gemm(fake, fake, 0, 128, 128, 4, fake, None, None, fake, 256, None) == -4
    assert lib.dsq_gemm(fake, fake, 128, 128, 128, 4, fake, None, None, fake, 8, None) == -5
    assert lib.dsq_gemm(fake, fake, 128, 128, 128, 4, fake, None, fake, fake, 256, None) == -1
    # K so large that 2^7 * (2^b - 1) * K overflows int32
    assert lib.dsq_gemm(fake, fake, 128, 128, 1 << 21, 4, fake, None, None, fake, 256, None) == -7
    # workspace query: small problems keep the status words only, large ones get
    # room for both operands as 8-bit rows (K rounded up to 16)
    assert lib.dsq_gemm_workspace_bytes(512, 4096, 4096, 4) == lib.dsq_workspace_bytes()
    assert lib.dsq_gemm_workspace_bytes(4096, 4096, 4096, 7) == lib.dsq_workspace_bytes()
    assert lib.dsq_gemm_workspace_bytes(4096, 4096, 4096, 4) == 256 + 1024 + 2 * 4096 * 4096
    assert lib.dsq_gemm_workspace_bytes(2048, 2048, 2048, 4) == lib.dsq_workspace_bytes()
    assert lib.dsq_gemm_workspace_bytes(4100, 4099, 2049, 2) >= 256 + 1024 + (4100 + 4099) * 2064
    assert lib.dsq_set_gemm_two_pass(2) == 0
    assert lib.dsq_gemm_workspace_bytes(1025, 1030, 1031, 2) >= 256 + 1024 + (1025 + 1030) * 1040
    assert lib.dsq_gemm_workspace_bytes(3, 5, 7, 4) > lib.dsq_workspace_bytes()
    assert lib.dsq_set_gemm_two_pass(1) == 0 and lib.dsq_set_gemm_two_pass(3) == -4
    # the no-workspace variant rejects bad arguments before it looks up its
    # scratch or enqueues anything (so this works without a GPU)
    assert lib.dsq_gemm_static_ws(None, fake, 128, 128, 128, 4, fake, None, None, 1, None) == -1
    assert lib.dsq_gemm_static_ws(fake, fake, 128, 128, 128, 5, fake, None, None, 1, None) == -3
    assert lib.dsq_gemm_static_ws(fake, fake, 128, 128, 128, 4, odd, None, None, 1, None) == -2
    assert lib.dsq_gemm_static_ws(fake, fake, 65537, 16, 16, 4, fake, None, None, 1, None) == -5

    # conv: unsupported geometry, lo != 0 with padding, 3-bit, bad w_offset
    scale = C.c_void_p(0x2000)
    ep = B.dsq_epilogue_t()
    ep.scale, ep.bias = 0x2000, 0x3000
    conv = B.dsq_conv_t(64, 3, 3, 64, 1, 1, 1)

    def call(conv=conv, q=q4, ep=ep, shape=shape):
        return lib.dsq_conv2d(fake, C.byref(shape), C.byref(q), fake, C.byref(conv),
                              C.byref(ep), fake, None, None, fake, 256, None)
    assert call(conv=B.dsq_conv_t(64, 5, 5, 64, 1, 2, 1)) == -8
    assert call(conv=B.dsq_conv_t(64, 3, 3, 64, 3, 1, 1)) == -8
    assert call(conv=B.dsq_conv_t(64, 3, 3, 32, 1, 1, 1)) == -4
    assert call(q=B.dsq_quant_t(4, -1.0, 2.0)) == -8
    assert call(q=B.dsq_quant_t(5, 0.0, 2.0)) == -3
    ep2 = B.dsq_epilogue_t()
    ep2.scale, ep2.bias, ep2.w_offset = 0x2000, 0x3000, float("nan")
    assert call(ep=ep2) == -6
    ep3 = B.dsq_epilogue_t()
    assert call(ep=ep3) == -1            # scale / bias missing
    # code output requested but no requantiser given
    assert lib.dsq_conv2d(fake, C.byref(shape), C.byref(q4), fake, C.byref(conv),
                          C.byref(ep), None, fake, None, fake, 256, None) == -3

    # soft quantiser: alpha outside (0, 1), bits outside 1..8, NULL
    qs = B.dsq_quant_t(4, 0.0, 1.0)
    assert lib.dsq_soft_quantize_fwd(fake, 16, C.byref(qs), C.c_float(0.0), fake, None) == -6
    assert lib.dsq_soft_quantize_fwd(fake, 16, C.byref(qs), C.c_float(1.5), fake, None) == -6
    assert lib.dsq_soft_quantize_fwd(fake, 16, C.byref(B.dsq_quant_t(0, 0.0, 1.0)), C.c_float(0.2),
                                     fake, None) == -3
    assert lib.dsq_soft_quantize_fwd(None, 16, C.byref(qs), C.c_float(0.2), fake, None) == -1
    assert lib.dsq_soft_quantize_bwd(fake, fake, 16, C.byref(qs), C.c_float(0.2), fake, None, None) == -1
    assert lib.dsq_soft_quantize_bwd(fake, fake, 0, C.byref(qs), C.c_float(0.2), fake, fake, None) == -4

    # depthwise wants groups = C
    assert lib.dsq_dwconv2d(fake, C.byref(shape), C.byref(q4), fake, C.byref(conv),
                            C.byref(ep), fake, None, None, None) == -4
    # pool: odd extent
    assert lib.dsq_maxpool2x2(fake, C.byref(B.dsq_nhwc_t(1, 7, 8, 64)), 4, fake, 1 << 20, None) == -4


def test_import_fails_loudly_without_the_library(tmp_path, monkeypatch):
    # the binding refuses to import when the shared object is absent
    import importlib.util
    src = open(B.__file__).read()
    mod = tmp_path / "binding_copy.py"
    mod.write_text(src)
    spec = importlib.util.spec_from_file_location("binding_copy", mod)
    m = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(m)
