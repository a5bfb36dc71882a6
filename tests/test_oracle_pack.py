"""Pins for the oracle's two packed layouts.

The paper fixes only the field content (k-bit two's complement, e.g. 1011 for -5 and 01101 for 13)
and, for its packed-bit tensor, 64 // k fields per unsigned 64-bit word.  The bit positions of the
sliced layout are this library's own; they are pinned by literal bytes worked out by hand from the
layout's prose definition (field widths 3, 4, 5, 6, 7 and 8), by the size function and by round trips.
"""
import numpy as np
import pytest

import oracle


def test_word64_field_counts_quoted_by_the_paper():
    # "twenty-one 3-bit weights ... twelve 5-bit weights" per unsigned INT64
    assert oracle.word64_fields_per_word(3) == 21
    assert oracle.word64_fields_per_word(5) == 12
    for k in range(3, 8):
        assert oracle.word64_fields_per_word(k) == 64 // k
        assert oracle.word64_row_words(1000, k) == -(-1000 // (64 // k))


def test_word64_fields_are_twos_complement():
    v = np.array([[-5, 13, -1, 7]], dtype=np.int8)
    w4 = oracle.pack_word64(np.array([[-5, 7]], dtype=np.int8), 4)
    assert int(w4[0, 0]) == (0b1011 | (0b0111 << 4))
    w5 = oracle.pack_word64(v, 5)
    assert int(w5[0, 0]) & 31 == 0b11011 and (int(w5[0, 0]) >> 5) & 31 == 0b01101
    assert np.array_equal(oracle.unpack_word64(w5, 4, 5), v)


@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("rows,cols", [(5, 1), (5, 31), (1, 128), (130, 147), (129, 300)])
def test_round_trips(bits, rows, cols):
    rng = np.random.default_rng(bits * 1000 + cols)
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1)
    v = rng.integers(lo, hi, size=(rows, cols)).astype(np.int8)
    p = oracle.pack_sliced(v, bits)
    assert p.shape == (-(-rows // 128) * 128, -(-cols // 128) * 16 * bits)
    assert np.array_equal(oracle.unpack_sliced(p, rows, cols, bits), v)
    if bits >= 2:
        w = oracle.pack_word64(v, bits)
        assert np.array_equal(oracle.unpack_word64(w, cols, bits), v)


def test_sliced_padding_is_zero_and_size_is_k_over_8_bytes_per_weight():
    v = np.full((2, 130), -1, dtype=np.int8)
    p = oracle.pack_sliced(v, 6)
    assert p.shape == (128, 2 * 96)
    back = oracle.unpack_sliced(p, 128, 256, 6)
    assert np.all(back[:2, :130] == -1) and np.all(back[:2, 130:] == 0) and np.all(back[2:] == 0)
    assert oracle.sliced_row_bytes(128 * 64, 5) * 8 == 128 * 64 * 5


def _packed_bytes(bits, placed, rows=1, cols=128):
    v = np.zeros((rows, cols), dtype=np.int8)
    for (r, c), val in placed.items():
        v[r, c] = val
    return oracle.pack_sliced(v, bits).reshape(-1)


def test_sliced_layout_literal_bytes():
    """Worked out by hand from the layout's prose: blocks of 128 rows x 128 columns, 2048 * k bytes each; inside a
    block the slice of width s takes 2048 * s bytes, row r of the block at r * 16 * s; inside a row's 16 * s bytes
    element e sits in byte ((e/32)*s + ((e%32)/4) / (8/s)) * 4 + e%4 at bits [8 - s*(sub+1), 8 - s*sub),
    sub = ((e%32)/4) % (8/s)."""
    # INT4 fields, element 0 = -5 (1011), element 4 = 7 (0111): they share byte 0 (lane 0 of word 0),
    # element 0 in the top nibble.  Element 1 = 3 goes to byte 1's top nibble.  Element 32 opens unit 1.
    p = _packed_bytes(4, {(0, 0): -5, (0, 4): 7, (0, 1): 3, (0, 32): -8})
    assert len(p) == 128 * 64
    assert p[0] == 0b1011_0111 and p[1] == 0b0011_0000 and p[16] == 0b1000_0000
    assert np.count_nonzero(p) == 3
    # INT5 = a 4-bit slice (8192 bytes of the block) then a 1-bit slice (2048 bytes): 13 = 0110|1
    p5 = _packed_bytes(5, {(0, 0): 13})
    assert p5[0] == 0b0110_0000 and p5[8192] == 0b1000_0000 and np.count_nonzero(p5) == 2
    # INT8 is the plain byte order of the block's rows
    v8 = np.arange(-64, 64, dtype=np.int8)[None, :]
    assert np.array_equal(oracle.pack_sliced(v8, 8).reshape(-1)[:128].view(np.int8), v8[0])
    # the second row of a block follows the first inside every slice: 16 * s bytes on
    p4 = _packed_bytes(4, {(1, 0): -1, (3, 127): -8}, rows=4)
    assert p4[64] == 0xF0 and p4[3 * 64 + 63] == 0x08 and np.count_nonzero(p4) == 2


def test_sliced_layout_literal_bytes_six_bit_fields():
    """INT(8|6) stores w_high in 6-bit fields: a 4-bit slice (bytes 0..8191 of a block) over a 2-bit slice
    (8192..12287)."""
    p = _packed_bytes(6, {(0, 0): -5, (0, 4): 13, (0, 13): -32, (0, 45): 31, (0, 127): -1, (0, 128): 1, (5, 0): 7, (130, 3): -2},
                      rows=131, cols=256)
    assert len(p) == 4 * 2048 * 6                                   # two row blocks x two column groups
    # e = 0: -5 = 111011 -> 1110 | 11;  e = 4: 13 = 001101 -> 0011 | 01 (same byte lane, next sub-position)
    assert p[0] == 0xE3 and p[8192] == 0xD0
    # e = 13: -32 = 100000 -> 1000 | 00: word 1, lane 1, low nibble; nothing in the 2-bit slice
    assert p[5] == 0x08
    # e = 45 (unit 1, element 13 of it): 31 = 011111 -> 0111 | 11
    assert p[21] == 0x07 and p[8192 + 9] == 0x03
    # e = 127, the row's last element of the group: -1 = 111111
    assert p[63] == 0x0F and p[8192 + 31] == 0x03
    # column 128 opens the second block, 12288 bytes on: 1 = 000001 -> 0000 | 01 in the top two bits
    assert p[12288] == 0x00 and p[12288 + 8192] == 0x40
    # row 5 of the first block: 64 bytes per row in the 4-bit slice, 32 in the 2-bit slice; 7 = 000111 -> 0001 | 11
    assert p[5 * 64] == 0x10 and p[8192 + 5 * 32] == 0xC0
    # row 130 = row 2 of the second row block (block number 2 of 4); column 3 = lane 3; -2 = 111110 -> 1111 | 10
    assert p[2 * 12288 + 2 * 64 + 3] == 0xF0 and p[2 * 12288 + 8192 + 2 * 32 + 3] == 0x80
    assert np.count_nonzero(p) == 12


def test_sliced_layout_literal_bytes_three_bit_fields():
    """INT(8|6) stores the compensated w_low in 3-bit fields: a 2-bit slice (bytes 0..4095 of a block) over a 1-bit
    slice (4096..6143)."""
    p = _packed_bytes(3, {(0, 0): -3, (0, 8): 3, (0, 30): -4, (0, 81): 2, (0, 127): -1, (127, 0): 1}, rows=128)
    assert len(p) == 2048 * 3
    # e = 0: -3 = 101 -> 10 | 1;  e = 8: 3 = 011 -> 01 | 1 (same lane, third sub-position of both slices)
    assert p[0] == 0x84 and p[4096] == 0xA0
    # e = 30 (quad 7, lane 2): -4 = 100 -> 10 | 0: word 1 of the 2-bit slice, last sub-position
    assert p[6] == 0x02
    # e = 81 (unit 2, element 17: quad 4, lane 1): 2 = 010 -> 01 | 0
    assert p[21] == 0x40
    # e = 127: -1 = 111
    assert p[31] == 0x03 and p[4096 + 15] == 0x01
    # the block's last row: 1 = 001 -> 00 | 1, top bit of byte 0 of that row's 16 bytes in the 1-bit slice
    assert p[4096 + 127 * 16] == 0x80
    assert np.count_nonzero(p) == 7


def test_sliced_layout_literal_bytes_seven_bit_fields():
    """Three slices: 4 bits (bytes 0..8191), 2 bits (8192..12287), 1 bit (12288..14335)."""
    p = _packed_bytes(7, {(0, 5): -64, (0, 6): 63})
    assert len(p) == 2048 * 7
    # e = 5 (quad 1, lane 1): -64 = 1000000 -> 1000 | 00 | 0;  e = 6 (quad 1, lane 2): 63 = 0111111 -> 0111 | 11 | 1
    assert p[1] == 0x08 and p[2] == 0x07 and p[8192 + 2] == 0x30 and p[12288 + 2] == 0x40
    assert np.count_nonzero(p) == 4
