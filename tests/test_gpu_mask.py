"""Baseline rounding masks on the GPU (BitShift / round up / RTN): against the oracle's RTN helper, and through the
whole GPU path against the paper's table of nesting numerical errors (decompose without compensation, recompose,
count the 256 INT8 values that come back changed)."""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu

MODES = {"bitshift": nq.NQ_ROUND_DOWN, "down": nq.NQ_ROUND_DOWN, "up": nq.NQ_ROUND_UP, "rtn": nq.NQ_ROUND_NEAREST}


def _table():
    rows = []
    for line in (Path(__file__).parent / "golden" / "numerical_error_table.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            m, h, nz, lo, hi = line.split()
            rows.append((m, int(h), int(nz), int(lo), int(hi)))
    return rows


@pytest.mark.parametrize("row", _table(), ids=lambda r: f"{r[0]}-h{r[1]}")
def test_numerical_error_table_on_the_gpu(row):
    method, h, nonzero, lo, hi = row
    w = np.arange(-128, 128, dtype=np.int8).reshape(1, 256)
    wd = torch.from_numpy(w).cuda()
    mask = nq.nq_rounding_mask(wd, 8, h, MODES[method])
    p_hi, p_lo = nq.nq_decompose(wd, mask, 8, h, False)          # Eq. 10: low part clipped to l bits
    back = nq.nq_recompose(p_hi, p_lo, 1, 256, 8, h, False).cpu().numpy().astype(np.int32)
    err = w.astype(np.int32) - back
    assert (int(np.count_nonzero(err)), int(err.min()), int(err.max())) == (nonzero, lo, hi)


@pytest.mark.parametrize("n,h", [(8, 3), (8, 4), (8, 6), (8, 7), (6, 4), (6, 5), (4, 1)])
@pytest.mark.parametrize("rows,cols", [(7, 130), (64, 256), (3, 1000)])
def test_rtn_mask_matches_the_oracle(n, h, rows, cols):
    rng = wl.rng_for(94, n * 10 + h)
    lim = 1 << (n - 1)
    w = rng.integers(-lim, lim, size=(rows, cols)).astype(np.int8)
    got = nq.nq_rounding_mask(torch.from_numpy(w).cuda(), n, h, nq.NQ_ROUND_NEAREST).cpu().numpy()
    assert np.array_equal(got, oracle.mask_rtn(w, n, h))
    assert not nq.nq_rounding_mask(torch.from_numpy(w).cuda(), n, h, nq.NQ_ROUND_DOWN).any()
    assert nq.nq_rounding_mask(torch.from_numpy(w).cuda(), n, h, nq.NQ_ROUND_UP).all()


def test_rejected_arguments():
    w = torch.zeros((4, 16), dtype=torch.int8, device="cuda")
    with pytest.raises(nq.NqError):
        nq.nq_rounding_mask(w, 8, 8, nq.NQ_ROUND_NEAREST)
    with pytest.raises(nq.NqError):
        nq.nq_rounding_mask(w, 8, 4, 7)
