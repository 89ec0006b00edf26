"""Pins of the oracle's packed-code format: element j of a row occupies bits
[j*b, j*b+b) of a little-endian bit stream; signed codes are b-bit two's
complement; the row pitch is the byte length rounded up to 16; spare bits are
zero.  The byte strings below were worked out by hand from that definition."""
import numpy as np
import pytest

from oracle import native


def test_hand_computed_byte_strings():
    p = native.pack_rows(np.array([[1, 2, 3, 4, 5, 6, 7, 8]], np.int8), 4)
    assert p.shape == (1, 16)
    assert bytes(p[0, :4]) == bytes([0x21, 0x43, 0x65, 0x87])
    assert not p[0, 4:].any()
    p = native.pack_rows(np.array([[0, 1, 2, 3, 3, 2, 1, 0]], np.int8), 2)
    assert bytes(p[0, :2]) == bytes([0xE4, 0x1B]) and not p[0, 2:].any()
    # 3-bit: sum(code_j << 3j) = 2054353 = 0x1F58D1
    p = native.pack_rows(np.array([[1, 2, 3, 4, 5, 6, 7, 0]], np.int8), 3)
    assert bytes(p[0, :3]) == bytes([0xD1, 0x58, 0x1F]) and not p[0, 3:].any()
    # signed two's complement fields
    p = native.pack_rows(np.array([[-8, -1, 0, 7]], np.int8), 4)
    assert bytes(p[0, :2]) == bytes([0xF8, 0x70])
    p = native.pack_rows(np.array([[-2, -1, 0, 1]], np.int8), 2)
    assert p[0, 0] == 0x4E
    p = native.pack_rows(np.array([[-4, -1, 3, 0]], np.int8), 3)
    assert bytes(p[0, :2]) == bytes([0xFC, 0x00])


def test_row_pitch():
    assert native.row_pitch(64, 4) == 32
    assert native.row_pitch(16, 4) == 16
    assert native.row_pitch(144, 4) == 80
    assert native.row_pitch(64, 2) == 16
    assert native.row_pitch(128, 3) == 48
    assert native.row_pitch(4096, 3) == 1536
    assert native.row_pitch(1, 2) == 16


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("signed", [False, True])
def test_round_trip_every_code_at_every_offset(bits, signed):
    half = 1 << (bits - 1)
    lo, hi = (-half, half - 1) if signed else (0, 2 * half - 1)
    for k in [1, 7, 8, 9, 31, 43, 128, 131]:
        # every code value at every position
        for v in range(lo, hi + 1):
            for j in range(min(k, 24)):
                row = np.zeros((1, k), np.int8)
                row[0, j] = v
                back = native.unpack_rows(native.pack_rows(row, bits), k,
                                          bits, signed)
                assert np.array_equal(back, row)
        rng = np.random.default_rng(k)
        codes = rng.integers(lo, hi + 1, size=(5, k), dtype=np.int8)
        packed = native.pack_rows(codes, bits)
        assert packed.shape[1] % 16 == 0
        assert np.array_equal(native.unpack_rows(packed, k, bits, signed),
                              codes)
        # spare bits are zero
        nbits = k * bits
        as_bits = np.unpackbits(packed, axis=1, bitorder="little")
        assert not as_bits[:, nbits:].any()
        # independent statement of the format through numpy bit arrays
        want = np.zeros_like(as_bits)
        u = codes.astype(np.int64) & (2 * half - 1)
        for t in range(bits):
            want[:, t:nbits:bits] = (u >> t) & 1
        assert np.array_equal(as_bits, want)
