"""Pins for the oracle's two packed layouts.

The paper fixes only the field content (k-bit two's complement, e.g. 1011 for -5 and 01101 for 13)
and, for its packed-bit tensor, 64 // k fields per unsigned 64-bit word.  The bit positions of the
sliced layout are this library's own; they are pinned by a hand-laid example written out below from
the layout's prose definition, by the size function and by round trips.
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
@pytest.mark.parametrize("cols", [1, 31, 128, 147, 300])
def test_round_trips(bits, cols):
    rng = np.random.default_rng(bits * 1000 + cols)
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1)
    v = rng.integers(lo, hi, size=(5, cols)).astype(np.int8)
    p = oracle.pack_sliced(v, bits)
    assert p.shape == (5, -(-cols // 128) * 16 * bits)
    assert np.array_equal(oracle.unpack_sliced(p, cols, bits), v)
    if bits >= 2:
        w = oracle.pack_word64(v, bits)
        assert np.array_equal(oracle.unpack_word64(w, cols, bits), v)


def test_sliced_padding_is_zero_and_size_is_k_over_8_bytes_per_weight():
    v = np.full((2, 130), -1, dtype=np.int8)
    p = oracle.pack_sliced(v, 6)
    assert p.shape[1] == 2 * 96
    back = oracle.unpack_sliced(p, 256, 6)
    assert np.all(back[:, :130] == -1) and np.all(back[:, 130:] == 0)
    assert oracle.sliced_row_bytes(128 * 64, 5) * 8 == 128 * 64 * 5


def _lay_by_hand(values, bits):
    """The sliced layout written out again, straight from its prose definition, bit by bit."""
    widths = [s for s in (8, 4, 2, 1) if bits & s]
    out = np.zeros(16 * bits, dtype=np.uint8)
    for e, val in enumerate(values):
        field = int(val) & ((1 << bits) - 1)
        text = format(field, f"0{bits}b")            # most significant bit first
        base, used = 0, 0
        for s in widths:
            piece = int(text[used:used + s], 2)
            unit, quad, lane = e // 32, (e % 32) // 4, e % 4
            per_byte = 8 // s
            word, sub = quad // per_byte, quad % per_byte
            byte = base + (unit * s + word) * 4 + lane
            out[byte] |= piece << (8 - s * (sub + 1))
            base += 16 * s
            used += s
    return out


@pytest.mark.parametrize("bits", range(1, 9))
def test_sliced_layout_against_a_hand_laid_group(bits):
    rng = np.random.default_rng(99 + bits)
    v = rng.integers(-(2 ** (bits - 1)), 2 ** (bits - 1), size=(1, 128)).astype(np.int8)
    assert np.array_equal(oracle.pack_sliced(v, bits)[0], _lay_by_hand(v[0], bits))


def test_sliced_layout_literal_bytes():
    # INT4 fields, element 0 = -5 (1011), element 4 = 7 (0111): they share byte 0 (lane 0 of word 0),
    # element 0 in the top nibble.  Element 1 = 3 goes to byte 1's top nibble.  Element 32 opens unit 1.
    v = np.zeros((1, 128), dtype=np.int8)
    v[0, 0], v[0, 4], v[0, 1], v[0, 32] = -5, 7, 3, -8
    p = oracle.pack_sliced(v, 4)[0]
    assert p[0] == 0b1011_0111 and p[1] == 0b0011_0000 and p[16] == 0b1000_0000
    assert np.count_nonzero(p) == 3
    # INT5 = a 4-bit slice (64 bytes) then a 1-bit slice (16 bytes): 13 = 0110|1
    v5 = np.zeros((1, 128), dtype=np.int8)
    v5[0, 0] = 13
    p5 = oracle.pack_sliced(v5, 5)[0]
    assert p5[0] == 0b0110_0000 and p5[64] == 0b1000_0000 and np.count_nonzero(p5) == 2
    # INT8 is the plain byte order
    v8 = np.arange(-64, 64, dtype=np.int8)[None, :]
    assert np.array_equal(oracle.pack_sliced(v8, 8)[0].view(np.int8), v8[0])
