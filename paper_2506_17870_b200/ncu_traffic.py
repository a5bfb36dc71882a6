"""DRAM traffic of the GEMM launches, from an ncu capture to a small tracked table.

The benchmark reports, next to the algorithmic bytes of a GEMM launch, what the launch really moved to and from
DRAM.  That figure is a hardware counter, so it cannot be taken in the timed run; it comes from one ncu pass over
the same command,

    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --clock-control none \\
        -k regex:contraction --csv --log-file <capture.csv> \\
        python bench.py --sizes 4096,8192 --steps 1 --warmup 1 --no-conv --no-cpu-baseline --no-model-switch --no-model-rows

and this module turns the capture into the table the benchmark reads:

    python -m paper_2506_17870_b200.ncu_traffic <capture.csv> --sizes 4096,8192 [--out profiles/gemm_dram_traffic.txt]

The table records a hash of the contraction kernels' sources.  `load` returns nothing once they have changed:
counters of another kernel version are not this kernel's traffic.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import statistics
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
KERNEL_SOURCES = ("nq_contraction.cuh", "nq_contraction_pair.cuh", "nq_sm100.cuh", "nq_gemm.cu")
HS = (4, 5, 6, 7)                      # part-bit launches of one size, in the benchmark's order; then one full-bit launch


def source_hash() -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        h.update((PKG / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def parse_capture(csv_path: Path, sizes, launches_per_step: int = 5):
    """{(size, h): [bytes of every repetition]} (h = 0: full-bit) and {(size, h): [duration ns]} from the capture.
    The capture holds whole steps; a step launches, per size, part-bit h = 4, 5, 6, 7 and then full-bit."""
    per_id = {}
    with open(csv_path, newline="") as f:
        rows = [r for r in csv.reader(f) if len(r) >= 15 and r[0].isdigit()]
    for r in rows:
        d = per_id.setdefault(int(r[0]), {})
        d[r[12]] = float(r[14].replace(",", ""))
    order = [(s, h) for s in sizes for h in list(HS) + [0]]
    traffic, duration = {}, {}
    ids = sorted(per_id)
    if len(ids) % len(order) != 0:
        raise ValueError(f"{len(ids)} captured launches are not whole steps of {len(order)} GEMM launches")
    for n, i in enumerate(ids):
        key = order[n % len(order)]
        m = per_id[i]
        traffic.setdefault(key, []).append(m["dram__bytes_read.sum"] + m["dram__bytes_write.sum"])
        duration.setdefault(key, []).append(m.get("gpu__time_duration.sum", 0.0))
    return traffic, duration


def write_table(csv_path: Path, sizes, out_path: Path, command: str = "") -> None:
    traffic, duration = parse_capture(csv_path, sizes)
    lines = ["# DRAM bytes (read + written) per GEMM launch, median over the captured repetitions; written by",
             "# python -m paper_2506_17870_b200.ncu_traffic from an ncu capture (see that module for the command).",
             f"# sources {source_hash()}",
             "# size h(0=full-bit) dram_bytes duration_us repetitions"]
    if command:
        lines.insert(2, "# capture: " + command)
    for (s, h), vals in sorted(traffic.items()):
        lines.append("%d %d %d %.1f %d" % (s, h, int(statistics.median(vals)),
                                           statistics.median(duration[(s, h)]) / 1e3, len(vals)))
    out_path.write_text("\n".join(lines) + "\n")


def load(path: Path):
    """({(size, h): bytes}, None), or (None, reason) when the table is absent or was taken on other kernel sources."""
    path = Path(path)
    if not path.exists():
        return None, "no capture on record"
    table, recorded = {}, None
    for line in path.read_text().splitlines():
        if line.startswith("# sources "):
            recorded = line.split()[2]
        if not line or line.startswith("#"):
            continue
        s, h, b = line.split()[:3]
        table[(int(s), int(h))] = float(b)
    if recorded != source_hash():
        return None, "the contraction kernels have changed since the counters were taken"
    return table, None


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("capture", type=Path)
    ap.add_argument("--sizes", default="4096,8192")
    ap.add_argument("--out", type=Path, default=PKG.parent / "profiles" / "gemm_dram_traffic.txt")
    ap.add_argument("--command", default="")
    a = ap.parse_args(argv)
    write_table(a.capture, tuple(int(x) for x in a.sizes.split(",")), a.out, a.command)
    print(a.out)
    return 0


if __name__ == "__main__":
    sys.exit(main())
