"""Pins for the oracle's decompose / recompose / drop-low against what the paper prints.

None of these re-type the oracle's formula: they compare it with the paper's worked example,
with every entry of its numerical-error table, with the ranges it states, and with the exactness
claim of the compensation ("all the part-bit models can upgrade to the full-bit ones without any
performance degradation").
"""
from pathlib import Path

import numpy as np
import pytest

import oracle

GOLDEN = Path(__file__).parent / "golden"
ALL_INT8 = np.arange(-128, 128, dtype=np.int16).astype(np.int8)


def _read_rows(name):
    rows = []
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line.split())
    return rows


def _bits(value, width):
    return format(int(value) & ((1 << width) - 1), f"0{width}b")


def test_worked_example_of_the_compensation_figure():
    g = {k: v for k, v in _read_rows("worked_example.txt")}
    w = np.array([int(g["w_int"])], dtype=np.int8)
    zero = np.zeros(1, dtype=np.uint8)                       # BitShift = round down
    wh, wl = oracle.decompose(w, zero, 8, 4, compensate=False)
    assert int(wh[0]) == int(g["w_high"])
    assert _bits(wh[0], 4) == g["w_high_bits"]
    assert int(wl[0]) == int(g["w_low_clipped"])
    assert _bits(wl[0], 4) == g["w_low_clipped_bits"]
    rec = oracle.recompose(wh, wl, 8, 4)
    assert int(rec[0]) == int(g["recomposed_clipped"])
    assert int(w[0]) - int(rec[0]) == int(g["numerical_error"])
    wh2, wl2 = oracle.decompose(w, zero, 8, 4, compensate=True)
    assert int(wh2[0]) == int(g["w_high"])
    assert int(wl2[0]) == int(g["w_low_compensated"])
    assert _bits(wl2[0], 5) == g["w_low_compensated_bits"]
    assert int(oracle.recompose(wh2, wl2, 8, 4)[0]) == int(g["recomposed_compensated"])


def _mask_for(method, h):
    if method in ("bitshift", "down"):
        return np.zeros(256, dtype=np.uint8)
    if method == "up":
        return np.ones(256, dtype=np.uint8)
    if method == "rtn":
        return oracle.mask_rtn(ALL_INT8, 8, h)
    raise AssertionError(method)


@pytest.mark.parametrize("row", _read_rows("numerical_error_table.txt"), ids=lambda r: f"{r[0]}-h{r[1]}")
def test_numerical_error_table(row):
    method, h, nonzero, lo, hi = row[0], int(row[1]), int(row[2]), int(row[3]), int(row[4])
    wh, wl = oracle.decompose(ALL_INT8, _mask_for(method, h), 8, h, compensate=False)
    rec = oracle.recompose(wh, wl, 8, h)
    err = ALL_INT8.astype(np.int32) - rec.astype(np.int32)
    assert int(np.count_nonzero(err)) == nonzero
    assert int(err.min()) == lo and int(err.max()) == hi


def test_rtn_mask_is_nearest_integer():
    # independent statement of round-to-nearest: |w/2^l - w_high| <= 1/2 before clipping
    for h in range(3, 8):
        l = 8 - h
        m = oracle.mask_rtn(ALL_INT8, 8, h)
        wh, _ = oracle.decompose(ALL_INT8, m, 8, h, compensate=True)
        unclipped = ALL_INT8.astype(np.float64) / 2 ** l
        inside = unclipped <= 2 ** (h - 1) - 1          # where the clip cannot bind
        assert np.all(np.abs(unclipped - wh)[inside] <= 0.5)


NESTINGS = [(8, h) for h in range(1, 8)] + [(6, h) for h in range(1, 6)]


@pytest.mark.parametrize("n,h", NESTINGS)
def test_compensated_recomposition_is_exact_for_every_value_and_mask(n, h):
    vals = np.arange(-(2 ** (n - 1)), 2 ** (n - 1), dtype=np.int16).astype(np.int8)
    for bit in (0, 1):
        mask = np.full(vals.shape, bit, dtype=np.uint8)
        wh, wl = oracle.decompose(vals, mask, n, h, compensate=True)
        assert np.array_equal(oracle.recompose(wh, wl, n, h), vals)
        assert np.array_equal(oracle.drop_low(vals, wl, n, h), wh)


@pytest.mark.parametrize("n,h", NESTINGS)
def test_ranges_stated_by_the_paper(n, h):
    l = n - h
    vals = np.arange(-(2 ** (n - 1)), 2 ** (n - 1), dtype=np.int16).astype(np.int8)
    seen_low = set()
    for bit in (0, 1):
        mask = np.full(vals.shape, bit, dtype=np.uint8)
        wh, wl = oracle.decompose(vals, mask, n, h, compensate=True)
        # w_high within the signed INTh range (Eq. 6)
        assert wh.min() >= -(2 ** (h - 1)) and wh.max() <= 2 ** (h - 1) - 1
        # compensated w_low within [-2^l + 1, 2^l - 1], inside signed INT(l+1)
        assert wl.min() >= -(2 ** l) + 1 and wl.max() <= 2 ** l - 1
        seen_low.update(int(v) for v in wl)
        whc, wlc = oracle.decompose(vals, mask, n, h, compensate=False)
        assert np.array_equal(whc, wh)
        # clipped w_low within the signed INTl range (Eq. 10)
        assert wlc.min() >= -(2 ** (l - 1)) and wlc.max() <= 2 ** (l - 1) - 1
        # errors of the uncompensated round trip within [-2^(l-1)+1, 2^(l-1)]
        err = vals.astype(np.int32) - oracle.recompose(whc, wlc, n, h).astype(np.int32)
        assert err.min() >= -(2 ** (l - 1)) + 1 and err.max() <= 2 ** (l - 1)
    # the union over both rounding directions needs all 2^(l+1) - 1 values: l bits cannot hold it
    assert len(seen_low) == 2 ** (l + 1) - 1


@pytest.mark.parametrize("n,h", NESTINGS)
def test_part_bit_weight_is_the_masked_rounding_of_w_over_2l(n, h):
    l = n - h
    rng = np.random.default_rng(7)
    vals = rng.integers(-(2 ** (n - 1)), 2 ** (n - 1), size=4096).astype(np.int8)
    mask = rng.integers(0, 2, size=4096).astype(np.uint8)
    wh, _ = oracle.decompose(vals, mask, n, h)
    x = vals.astype(np.float64) / 2 ** l
    want = np.where(mask == 1, np.ceil(x), np.floor(x))
    want = np.clip(want, -(2 ** (h - 1)), 2 ** (h - 1) - 1)
    assert np.array_equal(wh.astype(np.float64), want)


def test_bitshift_rounding_equals_arithmetic_right_shift():
    for h in range(1, 8):
        wh, _ = oracle.decompose(ALL_INT8, np.zeros(256, np.uint8), 8, h)
        assert np.array_equal(wh, (ALL_INT8.astype(np.int32) >> (8 - h)).astype(np.int8))


def test_recompose_adds_a_signed_low_part_not_a_bit_or():
    # -67 rounded up in INT(8|4): w_high = -4, w_low = -3, whose 5-bit field is 11101 (29).
    # Shift-and-add gives -67 back; OR-ing the bit fields, as a pure BitShift scheme would, does not.
    w = np.array([-67], dtype=np.int8)
    wh, wl = oracle.decompose(w, np.ones(1, np.uint8), 8, 4)
    assert (int(wh[0]), int(wl[0])) == (-4, -3)
    assert int(oracle.recompose(wh, wl, 8, 4)[0]) == -67
    assert ((-4 << 4) | (-3 & 31)) != -67
    assert int(oracle.recompose(np.array([3], np.int8), np.array([-3], np.int8), 8, 6)[0]) == 9


def test_recompose_clips_to_intn_on_arbitrary_inputs():
    assert int(oracle.recompose(np.array([31], np.int8), np.array([3], np.int8), 6, 4)[0]) == 31
    assert int(oracle.recompose(np.array([7], np.int8), np.array([15], np.int8), 8, 4)[0]) == 127


def test_unsupported_nesting_is_rejected():
    w = np.zeros(4, np.int8)
    m = np.zeros(4, np.uint8)
    for n, h in [(8, 8), (8, 0), (9, 4), (1, 1)]:
        with pytest.raises(ValueError):
            oracle.decompose(w, m, n, h)


def test_ideal_storage_reduction_table():
    # bits kept by a nested model (h + l + 1) against an INTn plus an INTh model (n + h),
    # counted from the oracle's own packed sizes on a long row
    cols = 128 * 1000
    for n, h, pct in [(int(a), int(b), int(c)) for a, b, c in _read_rows("ideal_storage_reduction.txt")]:
        l = n - h
        nested = oracle.sliced_row_bytes(cols, h) + oracle.sliced_row_bytes(cols, l + 1)
        diverse = oracle.sliced_row_bytes(cols, n) + oracle.sliced_row_bytes(cols, h)
        reduction = 100.0 * (1.0 - nested / diverse)
        assert abs(reduction - pct) < 0.75, (n, h, reduction, pct)
