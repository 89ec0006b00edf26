"""GPU parity, elementwise kernels: bit-exact against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import native
from gpu_util import T, N


@pytest.fixture(scope="module")
def dsq():
    import paper_1908_05033_b200 as d
    return d


SHAPES = [(1, 56, 56, 64), (2, 5, 7, 24), (1, 3, 3, 144), (3, 9, 9, 128),
          (1, 1, 1, 16), (1, 37, 41, 32), (2, 33, 65, 256), (1, 2, 2, 8)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("lo,hi", [(0.0, 2.0), (-0.7, 1.9)])
def test_quantize_act(dsq, bits, shape, lo, hi):
    rng = np.random.default_rng(bits * 100 + shape[3])
    x = (rng.standard_normal(shape) * 1.5).astype(np.float32)
    flat = x.reshape(-1)
    d = (np.float32(hi) - np.float32(lo)) / np.float32(2 ** bits - 1)
    special = [np.nan, np.inf, -np.inf, lo, hi, 0.0, -0.0, lo - 1, hi + 1]
    # exact levels and exact midpoints of the binary32 grid
    for q in range(2 ** bits):
        special += [np.float32(lo) + np.float32(q) * d,
                    np.float32(lo) + (np.float32(q) + np.float32(0.5)) * d]
    n = min(len(special), flat.size)
    flat[:n] = np.array(special[:n], np.float32)
    q = native.quantize(x, bits, lo, hi)
    ref = native.pack_rows(q.reshape(-1, shape[-1]), bits)
    got = N(dsq.dsq_quantize_act(T(x), bits, lo, hi)).reshape(ref.shape)
    assert np.array_equal(ref, got)


@pytest.mark.parametrize("bits", [2, 4])
def test_quantize_act_large_ragged_tail(dsq, bits):
    # several passes per warp plus a tail that is not a multiple of 32 lines
    shape = (3, 101, 67, 64)
    rng = np.random.default_rng(bits)
    x = np.maximum(rng.standard_normal(shape), 0).astype(np.float32)
    q = native.quantize(x, bits, 0.0, 2.0)
    ref = native.pack_rows(q.reshape(-1, 64), bits)
    got = N(dsq.dsq_quantize_act(T(x), bits, 0.0, 2.0)).reshape(ref.shape)
    assert np.array_equal(ref, got)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("rows,k", [(1, 1), (37, 131), (5, 128), (64, 4096), (3, 43)])
def test_pack_unpack_codes(dsq, bits, rows, k):
    half = 1 << (bits - 1)
    rng = np.random.default_rng(k)
    for signed in (True, False):
        lo, hi = (-half, half) if signed else (0, 2 * half)
        c = rng.integers(lo, hi, (rows, k), dtype=np.int8)
        ref = native.pack_rows(c, bits)
        got = dsq.dsq_pack_codes(T(c), bits)
        assert np.array_equal(ref, N(got))
        back = N(dsq.dsq_unpack(got, rows, k, bits, signed))
        assert np.array_equal(back, c)
        # the library's unpack reads the oracle's packing too
        back2 = N(dsq.dsq_unpack(T(ref), rows, k, bits, signed))
        assert np.array_equal(back2, c)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pack_weights_dense_and_depthwise(dsq, bits):
    ws = dsq.new_workspace()
    rng = np.random.default_rng(bits)
    for (Co, k, Ci) in [(64, 3, 64), (40, 3, 24), (24, 1, 144), (7, 1, 5)]:
        w = (rng.standard_normal((Co, k, k, Ci)) * 0.05).astype(np.float32)
        # scalar clip
        c = native.quantize_weights(w, bits, -0.1, 0.1)
        ref = native.pack_rows(c.reshape(Co * k * k, Ci), bits)
        blob, conv = dsq.dsq_pack_weights(T(w), bits, -0.1, 0.1, ws)
        assert np.array_equal(N(blob)[:ref.size].reshape(ref.shape), ref)
        # per-channel clip
        hi = (3 * w.reshape(Co, -1).std(1)).astype(np.float32)
        c = native.quantize_weights(w, bits, -hi, hi, per_row=True)
        ref = native.pack_rows(c.reshape(Co * k * k, Ci), bits)
        blob, conv = dsq.dsq_pack_weights(T(w), bits, T(-hi), T(hi), ws)
        assert np.array_equal(N(blob)[:ref.size].reshape(ref.shape), ref)
    for Cc in (32, 144, 20):
        w = (rng.standard_normal((Cc, 3, 3)) * 0.3).astype(np.float32)
        hi = np.abs(w).reshape(Cc, -1).max(1).astype(np.float32)
        c = native.quantize_weights(w, bits, -hi, hi, per_row=True)
        ref = native.pack_rows(c.reshape(Cc, 9).T.copy(), bits)   # [tap][C]
        blob, conv = dsq.dsq_pack_weights(T(w), bits, T(-hi), T(hi), ws,
                                          depthwise=True, pad=1)
        assert np.array_equal(N(blob)[:ref.size].reshape(ref.shape), ref)
    assert dsq.dsq_workspace_status(ws) == 0
    # a bad clip range is reported through the workspace
    w = np.zeros((4, 1, 1, 8), np.float32)
    dsq.dsq_pack_weights(T(w), bits, T(np.array([0, 0, 1, 0], np.float32)),
                         T(np.array([1, 1, 1, 1], np.float32)), ws)
    assert dsq.dsq_workspace_status(ws) == -6
    assert dsq.dsq_workspace_status(ws) == 0      # cleared by the read


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("shape", [(1, 4, 4, 64), (2, 6, 10, 24), (1, 8, 2, 144)])
def test_maxpool(dsq, bits, shape):
    rng = np.random.default_rng(bits + shape[3])
    q = rng.integers(0, 2 ** bits, shape, dtype=np.int8)
    ref = native.pack_rows(native.maxpool2x2(q).reshape(-1, shape[3]), bits)
    packed = T(native.pack_rows(q.reshape(-1, shape[3]), bits))
    got = N(dsq.dsq_maxpool2x2(packed, shape, bits)).reshape(ref.shape)
    assert np.array_equal(ref, got)
