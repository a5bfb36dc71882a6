"""The C-ABI library loads without a GPU and exports every symbol include/nq.h declares."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import build as nq_build

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def library():
    nq_build.build()
    return nq.lib()


def declared_symbols():
    text = (ROOT / "include" / "nq.h").read_text()
    return sorted(set(re.findall(r"NQ_API\s+[\w\s\*]+?\b(nq_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(library):
    names = declared_symbols()
    assert len(names) >= 18
    for name in names:
        assert hasattr(library, name), name
    assert sorted(nq.EXPORTS) == names


def test_host_side_size_functions(library):
    assert nq.nq_low_bits(8, 6, True) == 3 and nq.nq_low_bits(8, 6, False) == 2
    assert nq.nq_low_bits(8, 8, True) == -1 and nq.nq_low_bits(9, 4, True) == -1
    assert nq.nq_packed_row_bytes(128, 6) == 96
    assert nq.nq_packed_row_bytes(147, 6) == 192
    assert nq.nq_packed_row_bytes(0, 6) == 0
    assert nq.nq_packed_row_bytes(10, 9) == -1
    assert nq.nq_packed_bytes(64, 576, 3) == 128 * 5 * 48          # rows padded to a whole 128-row block
    assert nq.nq_packed_bytes(129, 128, 8) == 256 * 128
    assert nq.status_str(0) == "ok" and "alignment" in nq.status_str(3)


def test_argument_errors_are_reported_before_any_launch(library):
    null = ctypes.c_void_p(0)
    i64 = ctypes.c_int64
    # unsupported nesting, negative sizes, null pointers: no CUDA call is reached
    assert library.nq_decompose(null, null, i64(4), i64(4), i64(4), 8, 8, 1, null, null, null) == 2
    assert library.nq_decompose(null, null, i64(-1), i64(4), i64(4), 8, 6, 1, null, null, null) == 1
    assert library.nq_decompose(null, null, i64(4), i64(4), i64(4), 8, 6, 1, null, null, null) == 1
    assert library.nq_recompose(null, null, i64(0), i64(0), 8, 6, 1, null, i64(0), null) == 0
    assert library.nq_unpack(null, 9, i64(1), i64(1), null, i64(1), null) == 2
