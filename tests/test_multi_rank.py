"""The N > 1 arithmetic of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job throughput, and the
reference arm printing on rank 0 only.  The path shards as independent problems, so there is no data-path
collective to test: only the reduction of the timings."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]
sys.path.insert(0, str(ROOT))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        # rank r measured (10 + 5 r) ms for the step and (100 - 30 r) ms end to end
        got = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - 30.0 * rank], world)
        value = bench.whole_job_tops(world, 2.0e12, got[0])
        Path(out_dir, f"rank{rank}.json").write_text(json.dumps({"max": got, "value": value}))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_world2(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        r = json.loads(Path(tmp_path, f"rank{rank}.json").read_text())
        assert r["max"] == [15.0, 100.0]                    # slowest rank of each figure, the same on every rank
        # 2 ranks x 2e12 ops in 15 ms = 266.67 TOPS for the job
        assert r["value"] == pytest.approx(2 * 2.0e12 / 15.0e-3 / 1e12)


def test_world1_is_identity():
    import bench
    assert bench.max_over_ranks([3.5, 7.25], 1) == [3.5, 7.25]
    assert bench.whole_job_tops(1, 1.0e12, 1000.0) == pytest.approx(1.0)


def test_reference_arm_runs_on_rank0_only():
    """Under torchrun the oracle arm works and prints on rank 0; the other ranks exit 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
