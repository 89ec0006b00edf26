"""GPU parity, convolution paths: int32 accumulators and codes bit-exact
against the oracle; fp32 epilogue outputs within 1e-6 relative (they are in
fact bit-identical because both sides use the same binary32 sequence)."""
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


def assert_f32_close(got, ref):
    # tolerance stated by the benchmark spec: 1e-6 relative (with a floor for values
    # that cancel to ~0: relative to the largest magnitude in the tensor)
    tol = 1e-6 * np.maximum(np.abs(ref), np.abs(ref).max() * 1e-3 + 1e-30)
    assert np.all(np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= tol)
    assert np.array_equal(got, ref)        # and in fact bit-identical


def conv_case(dsq, N_, H, W, Ci, Co, k, s, p, bits, w_off, residual=False,
              per_channel=False, seed=5, a_hi=2.0, out_rng=(0.0, 1.0)):
    rng = np.random.default_rng(seed)
    x = np.maximum(rng.standard_normal((N_, H, W, Ci)), 0).astype(np.float32)
    w = (rng.standard_normal((Co, k, k, Ci)) * 0.05).astype(np.float32)
    scale = (rng.standard_normal(Co) * 0.1).astype(np.float32)
    bias = (rng.standard_normal(Co) * 0.1).astype(np.float32)
    if per_channel:
        w_hi = (3 * w.reshape(Co, -1).std(1)).astype(np.float32)
        w_lo = -w_hi
    else:
        w_lo, w_hi = -0.1, 0.1
    qa = native.quantize(x, bits, 0.0, a_hi)
    cw = native.quantize_weights(w, bits, w_lo, w_hi, per_row=per_channel)
    acc, sa = native.conv2d(qa, cw, s, p, want_sa=True)
    res = res_q = None
    r_lo, r_hi = -1.5, 2.5
    if residual:
        res = rng.integers(0, 2 ** bits, acc.shape, dtype=np.int8)
        res_q = (bits, r_lo, r_hi)
    d_r = (np.float32(r_hi) - np.float32(r_lo)) / np.float32(2 ** bits - 1)
    y = native.epilogue(acc, scale, bias, w_off, sa if w_off else None, res,
                        r_lo, d_r)
    qo = native.quantize(y, bits, *out_rng)
    ref_codes = native.pack_rows(qo.reshape(-1, Co), bits)

    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(x), bits, 0.0, a_hi)
    lo_t = T(w_lo) if per_channel else w_lo
    hi_t = T(w_hi) if per_channel else w_hi
    blob, conv = dsq.dsq_pack_weights(T(w), bits, lo_t, hi_t, ws, stride=s, pad=p)
    res_t = None
    if residual:
        res_t = T(native.pack_rows(res.reshape(-1, Co), bits))
    codes, yg, accg = dsq.dsq_conv2d(
        act, (N_, H, W, Ci), (bits, 0.0, a_hi), blob, conv, T(scale), T(bias),
        ws, w_offset=w_off, residual=res_t, residual_q=res_q,
        requant=(bits,) + out_rng, want_f32=True, want_acc=True)
    assert dsq.dsq_workspace_status(ws) == 0
    want_acc = 2 * acc + sa[..., None] if w_off == 0.5 else acc
    assert np.array_equal(N(accg), want_acc)
    assert_f32_close(N(yg), y)
    assert np.array_equal(N(codes).reshape(ref_codes.shape), ref_codes)
    # codes-only call (the form the stacks use) gives the same codes
    codes2, _, _ = dsq.dsq_conv2d(
        act, (N_, H, W, Ci), (bits, 0.0, a_hi), blob, conv, T(scale), T(bias),
        ws, w_offset=w_off, residual=res_t, residual_q=res_q,
        requant=(bits,) + out_rng)
    assert torch.equal(codes, codes2)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_table8_layer_shapes_at_every_bit_width(dsq, bits):
    """The four 3x3 layer shapes of the paper's Table 8 (batch 1, stride 1,
    pad 1) at 4, 3 and 2 bits, every accumulator and code against the oracle."""
    import os
    here = os.path.dirname(__file__)
    for line in open(os.path.join(here, "golden", "table8_shapes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ci, h, w, co = map(int, line.split())
        conv_case(dsq, 1, h, w, ci, co, 3, 1, 1, bits, 0.5, seed=ci)


def test_workload_1_single_3x3_conv(dsq):
    """64x56x56 -> 64, 3x3, stride 1, pad 1, 4-bit (Table 8, first row)."""
    c = dsq_inputs.conv3x3_case()
    bits = c["bits"]
    qa = native.quantize(c["x"], bits, c["act_lo"], c["act_hi"])
    cw = native.quantize_weights(c["w"], bits, c["w_lo"], c["w_hi"])
    assert qa.max() == 15 and cw.min() == -8 and cw.max() == 7
    acc = native.conv2d(qa, cw, c["stride"], c["pad"])
    y = native.epilogue(acc, c["scale"], c["bias"])
    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(c["x"]), bits, c["act_lo"], c["act_hi"])
    assert np.array_equal(N(act).reshape(-1, 32),
                          native.pack_rows(qa.reshape(-1, 64), bits))
    blob, conv = dsq.dsq_pack_weights(T(c["w"]), bits, c["w_lo"], c["w_hi"], ws,
                                      stride=1, pad=1)
    # packed rows first (18432 bytes), then the rows expanded to int8 K step by K step
    assert blob.numel() == 18432 + 64 * 5 * 128
    assert np.array_equal(N(blob)[:18432].reshape(64 * 9, 32),
                          native.pack_rows(cw.reshape(64 * 9, 64), bits))
    _, yg, accg = dsq.dsq_conv2d(act, c["x"].shape, (bits, c["act_lo"], c["act_hi"]),
                                 blob, conv, T(c["scale"]), T(c["bias"]), ws,
                                 want_f32=True, want_acc=True)
    assert dsq.dsq_workspace_status(ws) == 0
    assert np.array_equal(N(accg), acc)
    assert_f32_close(N(yg), y)


GEOMS = [  # N, H, W, Cin, Cout, k, stride, pad
    (1, 8, 8, 32, 32, 1, 1, 0), (1, 8, 8, 64, 64, 3, 1, 1),
    (2, 9, 7, 24, 40, 3, 2, 1), (1, 14, 14, 144, 24, 1, 1, 0),
    (3, 7, 7, 512, 512, 3, 1, 1), (2, 14, 14, 64, 128, 1, 2, 0),
    (1, 5, 5, 16, 96, 1, 1, 0), (1, 6, 6, 8, 8, 3, 1, 0),
    (2, 28, 28, 128, 128, 3, 1, 1), (1, 3, 3, 3, 5, 3, 1, 1),
    (1, 17, 13, 100, 300, 3, 2, 1), (1, 12, 12, 960, 160, 1, 1, 0)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("w_off", [0.0, 0.5])
@pytest.mark.parametrize("geom", GEOMS)
def test_conv_geometries(dsq, geom, bits, w_off):
    conv_case(dsq, *geom, bits, w_off, seed=hash(geom) % 1000)


@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("geom", [(6, 60, 60), (4, 70, 70), (1, 150, 150), (3, 97, 83)])
def test_conv_whole_k_rounds(dsq, geom, bits):
    """3x3 over 64 channels on more tiles than SMs: one round per tile, the A
    rows staged as whole image rows (rows of at most 2 KB) or as im2col boxes
    (wider images); image widths that do not divide the 128-pixel tile, a
    ragged last tile, every element against the oracle."""
    n, h, w = geom
    conv_case(dsq, n, h, w, 64, 64, 3, 1, 1, bits, 0.5, residual=(n == 6), seed=n + h)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_conv_residual_and_per_channel(dsq, bits):
    conv_case(dsq, 2, 14, 14, 64, 64, 3, 1, 1, bits, 0.5, residual=True)
    conv_case(dsq, 1, 10, 10, 48, 200, 1, 1, 0, bits, 0.5, residual=True,
              per_channel=True, out_rng=(0.0, 6.0))
    conv_case(dsq, 1, 9, 9, 32, 24, 3, 2, 1, bits, 0.0, residual=True,
              per_channel=True, out_rng=(-1.0, 1.0))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_conv_extreme_codes(dsq, bits):
    """All activations at the top code, all weights at the bottom code."""
    half = 1 << (bits - 1)
    N_, H, W, Ci, Co = 1, 9, 9, 512, 64
    x = np.full((N_, H, W, Ci), 5.0, np.float32)
    w = np.full((Co, 3, 3, Ci), -1.0, np.float32)
    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(x), bits, 0.0, 2.0)
    blob, conv = dsq.dsq_pack_weights(T(w), bits, -0.1, 0.1, ws, stride=1, pad=1)
    one = T(np.ones(Co, np.float32))
    zero = T(np.zeros(Co, np.float32))
    _, yg, accg = dsq.dsq_conv2d(act, x.shape, (bits, 0.0, 2.0), blob, conv, one,
                                 zero, ws, want_f32=True, want_acc=True)
    a = N(accg)
    assert a[0, 4, 4, 0] == 9 * Ci * -half * (2 * half - 1)
    assert a[0, 0, 0, 0] == 4 * Ci * -half * (2 * half - 1)
    assert np.array_equal(N(yg), a.astype(np.float32))     # scale 1, bias 0


def dw_case(dsq, N_, H, W, Cc, s, bits, w_off, residual=False, seed=6):
    rng = np.random.default_rng(seed)
    x = np.maximum(rng.standard_normal((N_, H, W, Cc)), 0).astype(np.float32)
    w = (rng.standard_normal((Cc, 3, 3)) * 0.3).astype(np.float32)
    scale = (rng.standard_normal(Cc) * 0.1).astype(np.float32)
    bias = (rng.standard_normal(Cc) * 0.1).astype(np.float32)
    hi = np.abs(w).reshape(Cc, -1).max(1).astype(np.float32)
    qa = native.quantize(x, bits, 0.0, 6.0)
    cw = native.quantize_weights(w, bits, -hi, hi, per_row=True)
    acc, sa = native.dwconv2d(qa, cw, s, 1, want_sa=True)
    res = res_q = res_t = None
    if residual:
        res = rng.integers(0, 2 ** bits, acc.shape, dtype=np.int8)
        res_q = (bits, 0.0, 6.0)
        res_t = T(native.pack_rows(res.reshape(-1, Cc), bits))
    d_r = np.float32(6.0) / np.float32(2 ** bits - 1)
    y = native.epilogue(acc, scale, bias, w_off, sa if w_off else None, res,
                        0.0, d_r)
    qo = native.quantize(y, bits, 0.0, 6.0)
    ref_codes = native.pack_rows(qo.reshape(-1, Cc), bits)
    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(x), bits, 0.0, 6.0)
    blob, conv = dsq.dsq_pack_weights(T(w), bits, T(-hi), T(hi), ws,
                                      depthwise=True, stride=s, pad=1)
    codes, yg, accg = dsq.dsq_dwconv2d(
        act, (N_, H, W, Cc), (bits, 0.0, 6.0), blob, conv, T(scale), T(bias),
        w_offset=w_off, residual=res_t, residual_q=res_q,
        requant=(bits, 0.0, 6.0), want_f32=True, want_acc=True)
    want_acc = 2 * acc + sa if w_off == 0.5 else acc
    assert np.array_equal(N(accg), want_acc)
    assert_f32_close(N(yg), y)
    assert np.array_equal(N(codes).reshape(ref_codes.shape), ref_codes)
    # codes-only call (the form the stacks use; 4-bit takes the dp4a kernel)
    codes2, _, _ = dsq.dsq_dwconv2d(
        act, (N_, H, W, Cc), (bits, 0.0, 6.0), blob, conv, T(scale), T(bias),
        w_offset=w_off, residual=res_t, residual_q=res_q, requant=(bits, 0.0, 6.0))
    assert torch.equal(codes, codes2)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("w_off", [0.0, 0.5])
@pytest.mark.parametrize("geom", [(1, 8, 8, 32, 1), (2, 9, 7, 144, 2),
                                  (1, 12, 12, 96, 1), (1, 3, 3, 20, 2),
                                  (2, 28, 28, 192, 2), (1, 1, 1, 8, 1),
                                  (3, 57, 61, 96, 1), (2, 30, 31, 40, 2), (1, 5, 2, 960, 1)])
def test_depthwise(dsq, geom, bits, w_off):
    dw_case(dsq, *geom, bits, w_off)
    if geom[4] == 1:
        dw_case(dsq, *geom, bits, w_off, residual=True)


WINDOW_GEOMS = [  # N, H, W, Cin, Cout: 3x3, stride 1, pad 1 on the shared-memory window
    (1, 3, 3, 64, 64), (2, 9, 7, 64, 40), (2, 9, 7, 128, 200), (1, 1, 1, 128, 64),
    (3, 7, 7, 512, 512), (2, 28, 28, 256, 300), (5, 14, 14, 256, 256),
    (1, 20, 150, 64, 64),      # wide image: three bands of 136 pixels
    (1, 6, 300, 128, 72), (2, 56, 56, 128, 128), (70, 5, 5, 64, 96)]


@pytest.mark.parametrize("w8", [1, 0])
@pytest.mark.parametrize("form", [3, 4])
@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("geom", WINDOW_GEOMS)
def test_conv3x3_window_kernel(dsq, geom, bits, form, w8):
    """3x3 stride-1 convolutions whose A operand is an expanded window of the
    input in shared memory (one constant row shift per filter tap): image sizes
    from 1x1 to wider than a window, tiles that span several images, channel
    counts with a ragged last N tile, one to four planes of 128 channels, with
    and without a residual operand, every element against the oracle.  Both
    forms of the kernel: form 3 = transposed tiles (256 positions x 128
    channels, weights as the A operand) where the geometry allows, form 4 =
    plain tiles only (128 positions x up to 256 channels).  w8 = 1: weight
    tiles of the wide layers come by TMA from the blob's pre-expanded int8 copy
    (grid Delta (c + 1/2) only); w8 = 0: the kernel expands the packed rows."""
    n, h, w, ci, co = geom
    if bits == 3 and (form == 4 or w8 == 0):
        pytest.skip("3-bit codes take the plain form and packed weights in every setting")
    dsq.dsq_set_conv3_window(form)     # this kernel wherever the geometry allows
    dsq.dsq_set_conv3_expanded_weights(w8)
    try:
        conv_case(dsq, n, h, w, ci, co, 3, 1, 1, bits, 0.5, residual=(n % 2 == 0),
                  seed=n + h + ci)
        conv_case(dsq, n, h, w, ci, co, 3, 1, 1, bits, 0.0, per_channel=True, seed=co)
    finally:
        dsq.dsq_set_conv3_window(1)
        dsq.dsq_set_conv3_expanded_weights(1)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_conv3x3_window_and_im2col_kernels_agree(dsq, bits):
    """The same convolution through both tensor-core kernels (hook) gives the
    same codes; both are compared with the oracle elsewhere."""
    c = dsq_inputs.conv3x3_case(N=3, H=19, W=23, Cin=128, Cout=128, bits=bits)
    ws = dsq.new_workspace()
    act = dsq.dsq_quantize_act(T(c["x"]), bits, 0.0, 2.0)
    blob, conv = dsq.dsq_pack_weights(T(c["w"]), bits, -0.1, 0.1, ws, stride=1, pad=1)
    args = (act, c["x"].shape, (bits, 0.0, 2.0), blob, conv, T(c["scale"]), T(c["bias"]), ws)
    dsq.dsq_set_conv3_window(3)
    try:
        a, _, _ = dsq.dsq_conv2d(*args, w_offset=0.5, requant=(bits, 0.0, 1.5))
        dsq.dsq_set_conv3_window(0)
        b, _, _ = dsq.dsq_conv2d(*args, w_offset=0.5, requant=(bits, 0.0, 1.5))
    finally:
        dsq.dsq_set_conv3_window(1)
    assert dsq.dsq_workspace_status(ws) == 0
    assert torch.equal(a, b)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("w_off", [0.3, -1.25, 2.0])
def test_general_weight_offset(dsq, bits, w_off):
    """Asymmetric learnt weight clips (Sec. 3.4: l_w and u_w are learnt
    separately) give a weight grid l_w + Delta_w q_w whose offset from the signed
    storage, o_w = l_w/Delta_w + 2^(b-1), is neither 0 nor 1/2: the epilogue then
    needs S_a next to the accumulator.  Dense convolutions on both tensor-core
    kernels and depthwise, against the oracle's general branch."""
    for geom in [(2, 9, 7, 64, 40, 3, 1, 1), (1, 12, 12, 128, 72, 3, 1, 1),
                 (2, 14, 14, 64, 128, 1, 2, 0), (1, 17, 13, 128, 300, 3, 2, 1),
                 (1, 12, 12, 960, 160, 1, 1, 0)]:
        conv_case(dsq, *geom, bits, w_off, residual=(geom[0] == 2), seed=geom[3])
    dw_case(dsq, 2, 9, 7, 144, 2, bits, w_off)
    dw_case(dsq, 1, 12, 12, 96, 1, bits, w_off, residual=True)
