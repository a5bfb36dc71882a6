"""The MMA-issue-only measurement kernel: it runs, ends by itself, reports its operation count, and its rate is
plausible for the tensor path (above what the GEMMs reach, below twice the nominal dense INT8 figure)."""
import pytest
import torch

import paper_2506_17870_b200 as nq

pytestmark = pytest.mark.gpu


def test_ceiling_kernel_runs_and_counts_its_operations():
    pairs = torch.cuda.get_device_properties(0).multi_processor_count // 2
    ops = nq.nq_i8_mma_ceiling(500)
    assert ops == pairs * 500 * 4 * 2.0 * 256 * 256 * 32
    nq.nq_device_status()
    best = 0.0
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ops = nq.nq_i8_mma_ceiling(3700)
        b.record()
        torch.cuda.synchronize()
        best = max(best, ops / (a.elapsed_time(b) * 1e-3) / 1e12)
    nq.nq_device_status()
    assert 1500.0 < best < 9000.0, best


def test_ceiling_rejects_launches_that_could_outlast_the_bounded_wait():
    with pytest.raises(nq.NqError) as e:
        nq.nq_i8_mma_ceiling(1 << 22)
    assert e.value.status == 1
    with pytest.raises(nq.NqError):
        nq.nq_i8_mma_ceiling(0)
