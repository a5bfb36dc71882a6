#!/usr/bin/env python
"""Benchmark of the nested-INT8 hot path on B200.

One "step" is one pass of the whole path over the large square GEMM sweep (M = N = K in
{4096, 8192, 16384}, INT8 nesting INTh for h in {4, 5, 6, 7}): for every size and h

    decompose -> drop-low (page-out) -> recompose (page-in) -> part-bit GEMM,   plus one full-bit GEMM per size,

followed by the ResNet-18-shaped convolution stack (config 2: 20 convolutions + classifier, batch 32, NCHW
int8 activations, implicit GEMM, both modes).  After the timed steps the whole-model page-out / page-in of a
ResNet-101-shaped and a ViT-B-shaped model (one batched launch each, cold L2) is timed separately and
reported under rows.model_switch, and configs 3 and 5 run layer by layer through both modes (the ResNet-101-shaped
stack at batch 128, the ViT-B/16 linears at 256 x 197 tokens): rows.resnet101_stack_int8_6, rows.vit_b16_linears_int8_4.
`value` is the integer-op throughput of the whole step (2*M*N*K per contraction; the codec kernels
add time but no ops) in TOPS, summed over ranks.  Per-row numbers (TOPS per mode, GB/s per codec
kernel) are reported under "rows".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sizes 4096,8192]

Under torchrun each rank runs the same per-GPU workload on its own GPU (independent problems, no
data-path collective: weak scaling); timing is max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

SIZES = (4096, 8192, 16384)
HS = (4, 5, 6, 7)
N_BITS = 8
ACT_SCALE = 0.05
METRIC = "nested_int8_gemm_tops"
CONV_H = 6


# DRAM bytes (read + written, MB) of one GEMM launch, from the ncu capture summarised in
# profiles/gemm_dram_traffic_4096_8192.md (tile-store epilogue, 40 ns barrier probes, packed-tile producer warp).  16384 was not captured (over
# a gigabyte per launch): it is taken as four times 8192, every operand and the output growing fourfold.  Must be set
# to None again when the contraction kernels change.
NCU_GEMM_DRAM_MB = {
    4096: {4: 25.7, 5: 27.8, 6: 30.0, 7: 32.2, 0: 34.3},
    8192: {4: 290.0, 5: 287.0, 6: 312.0, 7: 342.0, 0: 358.0},
}


def gemm_traffic_bytes_per_launch(sizes):
    """Mean DRAM traffic of the GEMM launches of one step (h = 4..7 part-bit + one full-bit per size), or None."""
    if NCU_GEMM_DRAM_MB is None:
        return None
    total, n = 0.0, 0
    for s in sizes:
        table, factor = NCU_GEMM_DRAM_MB.get(s), 1.0
        if table is None and s == 16384:
            table, factor = NCU_GEMM_DRAM_MB.get(8192), 4.0
        if table is None:
            return None
        for h in list(HS) + [0]:
            total += table[h] * factor * 1e6
            n += 1
    return total / n


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi in the background during the timed region: SM clock and throttle reasons."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for (_, l) in self.lines]
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- workload (host side, seeded)
def make_host_inputs(sizes):
    from paper_2506_17870_b200 import workloads as wl
    # W ~ clipped N(0, 40), X ~ clipped N(0, 32), Bernoulli(0.5) rounding mask, scales ~ U(1e-3, 1e-2)
    return {s: wl.gemm_inputs(4, i, s, s, s) for i, s in enumerate(sizes)}


def conv_bench_layers():
    """Config 2: the whole ResNet-18-shaped stack, 20 convolutions + the classifier."""
    from paper_2506_17870_b200 import workloads as wl
    return wl.resnet18_layers()


def _conv_available(nq, torch, dev):
    """True once nq_conv_implicit_gemm does work (probed with a tiny layer)."""
    try:
        d = nq.nq_conv_desc(1, 64, 8, 8, 64, 3, 3, 1, 1, 0)
        x = torch.zeros((1, 8, 8, 64), dtype=torch.int8, device=dev)
        w = torch.zeros((64, 576), dtype=torch.int8, device=dev)
        ws = torch.ones(64, device=dev)
        nq.nq_conv_implicit_gemm(x, w, d, ws, 1.0)
        torch.cuda.synchronize()
        return True
    except nq.NqError:
        return False


def _prepare_conv(nq, wl, torch, L, batch, index, dev):
    d = wl.conv_layer_inputs(2, index, L, batch)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    ldw = -(-L.K // 16) * 16
    w_mat = torch.from_numpy(wl.oihw_to_ohwi_matrix(d["W"], ldw)).to(dev)[:, :L.K]
    m_mat = torch.from_numpy(wl.oihw_to_ohwi_matrix(d["mask"], ldw)).to(dev)[:, :L.K]
    hi, lo = nq.nq_decompose(w_mat, m_mat, N_BITS, CONV_H, True)
    return {"desc": desc, "w": w_mat, "hi": hi, "ws": torch.from_numpy(d["w_scale"]).to(dev),
            "x": torch.from_numpy(d["X"]).to(dev), "act": d["act_scale"],
            "y": torch.empty((batch, L.Ho, L.Wo, L.Cout), dtype=torch.bfloat16, device=dev),
            "work": torch.empty(max(nq.nq_conv_workspace_bytes(desc), 0) + 2048, dtype=torch.uint8, device=dev)}


def _run_conv(nq, cs, part):
    if part:
        nq.nq_conv_implicit_gemm(cs["x"], cs["hi"], cs["desc"], cs["ws"], cs["act"], part_bit=True, n_bits=N_BITS,
                                 h_bits=CONV_H, workspace=cs["work"], y_out=cs["y"])
    else:
        nq.nq_conv_implicit_gemm(cs["x"], cs["w"], cs["desc"], cs["ws"], cs["act"], part_bit=False,
                                 workspace=cs["work"], y_out=cs["y"])


# --------------------------------------------------------------------------- multi-rank arithmetic
def max_over_ranks(values, world, device=None):
    """Element-wise maximum over the ranks of a list of per-rank figures (timings): one all-reduce, no data-path
    collective.  At world 1 the values come back unchanged.  Works on any initialised backend (nccl on GPUs,
    gloo in the CPU tests)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_tops(world, ops_per_gpu_per_step, ms_per_step):
    """Every rank runs the same per-GPU workload (independent problems, weak scaling): the job's throughput is
    the ops of all ranks over the slowest rank's time."""
    return world * ops_per_gpu_per_step / (ms_per_step * 1e-3) / 1e12


# --------------------------------------------------------------------------- our arm
def run_ours(args, rank, world, local_rank):
    import torch
    import paper_2506_17870_b200 as nq
    from paper_2506_17870_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    nq.lib()                                            # fail loudly if the extension is missing
    sizes = tuple(int(s) for s in args.sizes.split(","))
    host = make_host_inputs(sizes)
    stream = torch.cuda.current_stream()

    state = {}
    for s in sizes:
        d = {k: torch.from_numpy(host[s][k]).to(dev) for k in ("W", "X", "mask", "w_scale")}
        d["y"] = torch.empty((s, s), dtype=torch.bfloat16, device=dev)
        d["w_rec"] = torch.empty((s, s), dtype=torch.int8, device=dev)
        d["hi"] = {h: torch.empty((s, nq.nq_packed_row_bytes(s, h)), dtype=torch.uint8, device=dev) for h in HS}
        d["lo"] = {h: torch.empty((s, nq.nq_packed_row_bytes(s, N_BITS - h + 1)), dtype=torch.uint8, device=dev)
                   for h in HS}
        state[s] = d

    conv_layers, conv_state = [], []
    have_conv = args.conv and _conv_available(nq, torch, dev)
    if have_conv:
        conv_layers = conv_bench_layers()
        conv_state = [_prepare_conv(nq, wl, torch, L, args.conv_batch, i, dev) for i, L in enumerate(conv_layers)]

    launches = [0]
    events = {}

    def timed(key, fn, record, n_kernels=1):
        if record:
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            events.setdefault(key, []).append((a, b))
        else:
            fn()
        launches[0] += n_kernels

    def step(record):
        for s in sizes:
            d = state[s]
            for h in HS:
                timed(("decompose", s, h), lambda: nq.nq_decompose(d["W"], d["mask"], N_BITS, h, True, out_high=d["hi"][h], out_low=d["lo"][h]), record)
                timed(("page_out", s, h), lambda: nq.nq_drop_low(d["W"], d["lo"][h], N_BITS, h, True, out_high=d["hi"][h]), record)
                timed(("page_in", s, h), lambda: nq.nq_recompose(d["hi"][h], d["lo"][h], s, s, N_BITS, h, True, out=d["w_rec"]), record)
                timed(("gemm_part", s, h), lambda: nq.nq_gemm_part(d["X"], d["hi"][h], s, N_BITS, h, d["w_scale"], ACT_SCALE, y_out=d["y"]), record)
            timed(("gemm_full", s, 0), lambda: nq.nq_gemm_full(d["X"], d["w_rec"], d["w_scale"], ACT_SCALE, y_out=d["y"]), record)
        for L, cs in zip(conv_layers, conv_state):
            timed(("conv_full", L.name, 0), lambda: _run_conv(nq, cs, False), record, 2)   # layout pre-pass + contraction
            timed(("conv_part", L.name, 0), lambda: _run_conv(nq, cs, True), record, 2)

    ops_step = sum(2.0 * s ** 3 * (len(HS) + 1) for s in sizes)
    for L in conv_layers:
        M, N, K = L.gemm_view(args.conv_batch)
        ops_step += 2 * 2.0 * M * N * K

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    nq.nq_device_status()

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches[0] = 0
    barrier()
    t_wall0 = time.time()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step(True)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    total_ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t_wall0, t_wall1)
    nq.nq_device_status()
    gpu_launches = launches[0]

    e2e = _run_e2e(nq, torch, sizes, host, state, args, world)
    model_switch = _model_switch(nq, torch, wl, dev) if (rank == 0 and args.model_switch) else None
    model_rows = _model_rows(nq, torch, wl, dev, args.model_batch) if (rank == 0 and args.model_rows and have_conv) else None

    total_ms, e2e["ms_per_step"] = max_over_ranks([total_ms, e2e["ms_per_step"]], world, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_tops(world, ops_step, ms_per_step)
    if rank != 0:
        return None

    peaks = measured_peaks()
    rows = _summarise_rows(events, conv_layers, args.conv_batch, peaks)
    gemm_ms, gemm_ops, gemm_n = 0.0, 0.0, 0
    for (kind, s, h), pairs in events.items():
        if kind in ("gemm_full", "gemm_part"):
            for a, b in pairs:
                gemm_ms += a.elapsed_time(b)
                gemm_ops += 2.0 * s ** 3
                gemm_n += 1
    int8_peak = 2.0 * peaks["bf16_tflops"]
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    roofline = {
        "bound": "tensor", "kernel": "contraction_pair_kernel / contraction_kernel (tcgen05 kind::i8): every GEMM launch of the timed steps",
        "achieved": round(achieved, 1), "peak": round(int8_peak, 1), "unit": "TOP/s",
        "frac": round(achieved / int8_peak, 4),
        "peak_source": "2 x the %s bf16 burst figure (dense INT8 : bf16 nominal ratio 4.5 : 2.25)" % peaks["source"],
        "launches": gemm_n, "avg_launch_ms": round(gemm_ms / max(gemm_n, 1), 4),
        "traffic": gemm_traffic_bytes_per_launch(sizes),
        "traffic_unit": "DRAM bytes per launch, mean over the step's GEMM launches (ncu, profiles/gemm_dram_traffic_4096_8192.md)",
        "algorithmic_bytes_per_launch": float(np.mean([s * s * (1 + (h / 8.0 if h else 1.0) + 2) for s in sizes for h in list(HS) + [0]])),
    }
    conv_note = (", + config 2: the ResNet-18-shaped stack (%d layers), batch %d, NCHW int8 in, both modes"
                 % (len(conv_layers), args.conv_batch) if have_conv else "")
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "TOPS", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "config 4: square nested GEMM sweep M=N=K in {%s}, INT8 nesting INTh, h in {4,5,6,7}: "
                               "decompose, page-out, page-in, part-bit GEMM per (size, h) + full-bit GEMM per size%s"
                               % (",".join(map(str, sizes)), conv_note),
                   "output": "bf16", "l2": "inputs larger than L2, no flush (every kernel of the step touches > 126 MB "
                                           "between two launches of the same kernel)",
                   "per_gpu_ops_per_step": ops_step},
        "clocks": clocks, "gpu_launches": gpu_launches,
        "e2e": {"value": round(whole_job_tops(world, ops_step, e2e["ms_per_step"]), 3), "unit": "TOPS",
                "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": round(e2e["ms_per_step"], 3), "covers": "the GEMM sweep (codec + both GEMM modes)"},
        "roofline": roofline, "rows": rows,
    }
    if model_switch is not None:
        line["rows"]["model_switch"] = model_switch
        line["rows"]["word64_convert_8192"] = _word64_rows(nq, torch, dev)
        line["rows"]["gemm_nested_8192"] = _nested_rows(nq, torch, dev)
    if model_rows is not None:
        line["rows"].update(model_rows)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(sizes, host, args.cpu_rows)
    return line


def _summarise_rows(events, conv_layers, conv_batch, peaks):
    out = {"gemm_full": {}, "gemm_part": {}, "codec": {}}
    int8_peak = 2.0 * peaks["bf16_tflops"]
    hbm = peaks["hbm_gbs"]
    codec_bytes = {"decompose": 1 + 1 + 9 / 8, "page_out": 1 + 9 / 8, "page_in": 9 / 8 + 1}   # per weight, n = 8
    agg = {}
    for (kind, s, h), pairs in events.items():
        ms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
        if kind == "gemm_full":
            t = 2.0 * s ** 3 / (ms * 1e-3) / 1e12
            out["gemm_full"][str(s)] = {"tops": round(t, 1), "frac_int8_peak": round(t / int8_peak, 3), "ms": round(ms, 4)}
        elif kind == "gemm_part":
            t = 2.0 * s ** 3 / (ms * 1e-3) / 1e12
            out["gemm_part"].setdefault(str(s), {})[f"h{h}"] = {"tops": round(t, 1), "frac_int8_peak": round(t / int8_peak, 3),
                                                                "ms": round(ms, 4)}
        elif kind in codec_bytes:
            agg.setdefault((kind, s), []).append(codec_bytes[kind] * s * s / (ms * 1e-3) / 1e9)
        elif kind in ("conv_full", "conv_part"):
            L = next(l for l in conv_layers if l.name == s)
            M, N, K = L.gemm_view(conv_batch)
            t = 2.0 * M * N * K / (ms * 1e-3) / 1e12
            out.setdefault(kind, {})[s] = {"tops": round(t, 1), "ms": round(ms, 4), "gemm_view": [M, N, K]}
    for kind in ("conv_full", "conv_part"):
        if kind in out:
            tot_ms = sum(v["ms"] for v in out[kind].values())
            tot_ops = sum(2.0 * v["gemm_view"][0] * v["gemm_view"][1] * v["gemm_view"][2] for v in out[kind].values())
            out[kind + "_stack"] = {"ms": round(tot_ms, 4), "tops": round(tot_ops / (tot_ms * 1e-3) / 1e12, 1),
                                    "layers": len(out[kind])}
    for (kind, s), vals in agg.items():
        g = float(np.mean(vals))
        out["codec"].setdefault(kind, {})[str(s)] = {"gbs": round(g, 0), "frac_hbm": round(g / hbm, 3)}
    out["codec"]["algorithmic_bytes_per_weight"] = codec_bytes
    out["peaks"] = {"int8_tops": int8_peak, "hbm_gbs": hbm, "source": peaks["source"]}
    return out


def _model_switch(nq, torch, wl, dev):
    """Whole-model page-out and page-in as one batched launch each, INT(8|6) ResNet-101 (105 tensors) and INT(8|4)
    ViT-B/16 blocks (48 tensors).  Three copies of each model are rotated so that every launch finds its data in
    HBM, not in the 126 MB L2; CUDA events around three back-to-back launches (one per copy), median of 12."""
    peaks = measured_peaks()
    out = {}
    models = {
        "resnet101_int8_6": (6, [(L.Cout, L.K) for L in wl.resnet101_layers()]),
        "vit_b16_int8_4": (4, [(n, k) for _, k, n in wl.vit_b16_linears()]),
    }
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.BASE_SEED)
    for name, (h, shapes) in models.items():
        copies = []
        for c in range(3):
            tensors = []
            for rows, cols in shapes:
                ld = -(-cols // 16) * 16
                w = torch.randint(-128, 128, (rows, ld), dtype=torch.int8, device=dev, generator=gen)[:, :cols]
                m = torch.randint(0, 2, (rows, ld), dtype=torch.uint8, device=dev, generator=gen)[:, :cols]
                hi, lo = nq.nq_decompose(w, m, N_BITS, h, True)
                tensors.append({"w_int": w, "packed_high": hi, "packed_low": lo})
            copies.append(nq.nq_batch_plan(tensors))
        weights = sum(r * c for r, c in shapes)
        nbytes = weights * 2.125
        res = {}
        for kind, fn in (("page_out", nq.nq_drop_low_batched), ("page_in", nq.nq_recompose_batched)):
            for i in range(3):
                fn(copies[i], N_BITS, h, True)
            torch.cuda.synchronize()
            ts = []
            for i in range(12):                       # one launch per copy inside each event pair
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                for c in range(3):
                    fn(copies[c], N_BITS, h, True)
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) / 3)
            ms = float(np.median(ts))
            gbs = nbytes / (ms * 1e-3) / 1e9
            res[kind] = {"us": round(ms * 1e3, 1), "gbs": round(gbs, 0), "frac_hbm": round(gbs / peaks["hbm_gbs"], 3)}
        res["weights"] = weights
        res["tensors"] = len(shapes)
        res["algorithmic_mb"] = round(nbytes / 1e6, 1)
        out[name] = res
    return out


def _nested_rows(nq, torch, dev):
    """The full-bit layer computed straight from packed w_high and compensated w_low (no INT8 copy of the weights):
    8192^3, median of 5 launches per nesting, against the int8 peak; outputs checked equal to the full-bit GEMM's."""
    peaks = measured_peaks()
    int8_peak = 2.0 * peaks["bf16_tflops"]
    S = 8192
    gen = torch.Generator(device=dev)
    gen.manual_seed(11)
    W = torch.randint(-128, 128, (S, S), dtype=torch.int8, device=dev, generator=gen)
    X = torch.randint(-128, 128, (S, S), dtype=torch.int8, device=dev, generator=gen)
    mask = torch.randint(0, 2, (S, S), dtype=torch.uint8, device=dev, generator=gen)
    ws = torch.rand(S, device=dev, generator=gen) * 0.01 + 0.001
    y = torch.empty((S, S), dtype=torch.float32, device=dev)
    nq.nq_gemm_full(X, W, ws, ACT_SCALE, y_out=y)
    ref = y.clone()
    out = {}
    for h in HS:
        hi, lo = nq.nq_decompose(W, mask, N_BITS, h, True)
        ts = []
        for rep in range(6):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            nq.nq_gemm_nested(X, hi, lo, S, N_BITS, h, ws, ACT_SCALE, y_out=y)
            b.record()
            torch.cuda.synchronize()
            if rep:
                ts.append(a.elapsed_time(b))
        ms = float(np.median(ts))
        t = 2.0 * S * S * S / (ms * 1e-3) / 1e12
        out[f"h{h}"] = {"tops": round(t, 1), "frac_int8_peak": round(t / int8_peak, 3), "ms": round(ms, 4),
                        "weight_bytes_per_element": (N_BITS + 1) / 8, "equals_full_bit": bool(torch.equal(y, ref))}
    return out


def _word64_rows(nq, torch, dev):
    """The paper's packed-bit tensors (64 // k fields per 64-bit word) converted to the sliced layout and back on the
    device: one 8192 x 8192 tensor per field width, bytes read + written over the median of 5 launches."""
    peaks = measured_peaks()
    out = {}
    rows = cols = 8192
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    for bits in (4, 5, 6):
        lim = 1 << (bits - 1)
        v = torch.randint(-lim, lim, (rows, cols), dtype=torch.int8, device=dev, generator=gen)
        sliced = nq.nq_pack(v, bits)
        words = nq.nq_sliced_to_word64(sliced, bits, rows, cols)
        nbytes = sliced.numel() + words.numel() * 8
        row = {}
        for name, fn in (("to_sliced", lambda: nq.nq_word64_to_sliced(words, bits, cols)),
                         ("to_word64", lambda: nq.nq_sliced_to_word64(sliced, bits, rows, cols))):
            ts = []
            for rep in range(6):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                if rep:
                    ts.append(a.elapsed_time(b))
            ms = float(np.median(ts))
            g = nbytes / (ms * 1e-3) / 1e9
            row[name] = {"us": round(ms * 1e3, 1), "gbs": round(g, 0), "frac_hbm": round(g / peaks["hbm_gbs"], 3)}
        out[f"k{bits}"] = row
    return out


def _device_conv_weights(torch, L, dev, gen):
    """[Cout, K] int8 weights of a layer, Gaussian fit then per-channel INT8 quantisation (Eq. 1), generated on the
    device for the timing-only rows (the parity tests use the seeded host generators)."""
    ldw = -(-L.K // 16) * 16
    w = torch.randn((L.Cout, ldw), device=dev, generator=gen) * (2.0 / L.K) ** 0.5
    s = w[:, :L.K].abs().amax(dim=1).clamp_min(1e-12) / 127.0
    q = torch.clamp(torch.round(w / s[:, None]), -128, 127).to(torch.int8)
    q[:, L.K:] = 0
    return q[:, :L.K], s.float()


def _model_rows(nq, torch, wl, dev, conv_batch):
    """Configs 3 and 5 through both modes, layer by layer on seeded device-side inputs of the stated shapes and
    distributions: the ResNet-101-shaped stack (104 convolutions + classifier, batch `conv_batch`, NCHW int8
    activations ~ U{0..127}, INT8 nesting INT6, bf16 out) and the ViT-B/16 linears (M = 256 * 197 tokens, INT8
    nesting INT4).  Each layer is timed with its own pair of CUDA events, median of 3 passes; inputs of one pass
    exceed L2, so nothing is flushed."""
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.BASE_SEED + 3000)
    out = {}
    # ---- config 3
    layers = wl.resnet101_layers()
    xs, prepared = {}, []
    y_elems = max(conv_batch * L.Ho * L.Wo * L.Cout for L in layers)
    ybuf = torch.empty(y_elems, dtype=torch.bfloat16, device=dev)
    work_bytes = 0
    for L in layers:
        key = (L.Cin, L.H, L.W)
        if key not in xs:
            xs[key] = torch.randint(0, 128, (conv_batch, L.Cin, L.H, L.W), dtype=torch.int8, device=dev, generator=gen)
        desc = nq.nq_conv_desc(conv_batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
        w, ws = _device_conv_weights(torch, L, dev, gen)
        m = torch.randint(0, 2, (L.Cout, w.stride(0)), dtype=torch.uint8, device=dev, generator=gen)[:, :L.K]
        hi, lo = nq.nq_decompose(w, m, N_BITS, CONV_H, True)
        work_bytes = max(work_bytes, nq.nq_conv_workspace_bytes(desc))
        prepared.append({"desc": desc, "w": w, "hi": hi, "lo": lo, "ws": ws, "x": xs[key], "act": 0.02,
                         "y": ybuf[:conv_batch * L.Ho * L.Wo * L.Cout].view(conv_batch, L.Ho, L.Wo, L.Cout)})
    work = torch.empty(work_bytes + 2048, dtype=torch.uint8, device=dev)
    for cs in prepared:
        cs["work"] = work
    ops = sum(2.0 * float(np.prod(L.gemm_view(conv_batch))) for L in layers)
    res = {}
    for part in (False, True):
        per_layer = []
        for rep in range(4):
            evs = []
            for cs in prepared:
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                _run_conv(nq, cs, part)
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            if rep:
                per_layer.append([a.elapsed_time(b) for a, b in evs])
        ms = float(np.sum(np.median(np.array(per_layer), axis=0)))
        res["part_bit" if part else "full_bit"] = {"ms": round(ms, 3), "tops": round(ops / (ms * 1e-3) / 1e12, 1)}
    # the full-bit stack again with no INT8 copy of the weights: every layer rebuilds them from the two packed parts
    per_layer = []
    for rep in range(4):
        evs = []
        for cs in prepared:
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            nq.nq_conv_implicit_gemm_nested(cs["x"], cs["hi"], cs["lo"], cs["desc"], cs["ws"], cs["act"], n_bits=N_BITS,
                                            h_bits=CONV_H, workspace=cs["work"], y_out=cs["y"])
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        if rep:
            per_layer.append([a.elapsed_time(b) for a, b in evs])
    ms = float(np.sum(np.median(np.array(per_layer), axis=0)))
    res["nested_full_bit"] = {"ms": round(ms, 3), "tops": round(ops / (ms * 1e-3) / 1e12, 1)}
    res.update({"layers": len(layers), "batch": conv_batch, "weights": sum(L.weights for L in layers),
                "tera_ops_per_pass": round(ops / 1e12, 3)})
    # the same stack in chained form: NHWC int8 activations in, the next layer's INT8 activations out (requantising
    # epilogue with ReLU), no layout pre-pass; every layer still runs on its own input
    yq = torch.empty(y_elems, dtype=torch.int8, device=dev)
    for cs, L in zip(prepared, layers):
        key = ("nhwc", L.Cin, L.H, L.W)
        if key not in xs:
            xs[key] = cs["x"].permute(0, 2, 3, 1).contiguous()
        cs["x_nhwc"] = xs[key]
        cs["desc_nhwc"] = nq.nq_conv_desc(conv_batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 0)
        cs["yq"] = yq[:conv_batch * L.Ho * L.Wo * L.Cout].view(conv_batch, L.Ho, L.Wo, L.Cout)
    for part in (False, True):
        per_layer = []
        for rep in range(4):
            evs = []
            for cs in prepared:
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                nq.nq_conv_implicit_gemm_q8(cs["x_nhwc"], cs["hi"] if part else cs["w"], cs["desc_nhwc"], cs["ws"], cs["act"],
                                            0.5, relu=True, part_bit=part, n_bits=N_BITS, h_bits=CONV_H,
                                            workspace=cs["work"], y_out=cs["yq"])
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            if rep:
                per_layer.append([a.elapsed_time(b) for a, b in evs])
        ms = float(np.sum(np.median(np.array(per_layer), axis=0)))
        res["chained_int8_out_" + ("part_bit" if part else "full_bit")] = {"ms": round(ms, 3), "tops": round(ops / (ms * 1e-3) / 1e12, 1)}
    per_layer = []
    for rep in range(4):
        evs = []
        for cs in prepared:
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            nq.nq_conv_implicit_gemm_nested_q8(cs["x_nhwc"], cs["hi"], cs["lo"], cs["desc_nhwc"], cs["ws"], cs["act"], 0.5,
                                               relu=True, n_bits=N_BITS, h_bits=CONV_H, workspace=cs["work"], y_out=cs["yq"])
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        if rep:
            per_layer.append([a.elapsed_time(b) for a, b in evs])
    ms = float(np.sum(np.median(np.array(per_layer), axis=0)))
    res["chained_int8_out_nested_full_bit"] = {"ms": round(ms, 3), "tops": round(ops / (ms * 1e-3) / 1e12, 1)}
    del yq
    out["resnet101_stack_int8_6"] = res
    nq.nq_device_status()
    del prepared, xs, ybuf, work
    torch.cuda.empty_cache()
    # ---- config 5
    M = 256 * wl.VIT_TOKENS
    res = {}
    for _, k, n in wl.vit_b16_linears(1):
        x = torch.clamp(torch.round(torch.randn((M, k), device=dev, generator=gen) * 32.0), -128, 127).to(torch.int8)
        wf = torch.randn((n, k), device=dev, generator=gen) * 0.02
        hit = torch.rand((n, k), device=dev, generator=gen) < 1e-3
        sign = torch.where(torch.rand((n, k), device=dev, generator=gen) < 0.5, -1.0, 1.0)
        wf = torch.where(hit, sign * 0.12, wf)
        sc = wf.abs().amax(dim=1) / 127.0
        w = torch.clamp(torch.round(wf / sc[:, None]), -128, 127).to(torch.int8)
        m = torch.randint(0, 2, w.shape, dtype=torch.uint8, device=dev, generator=gen)
        hi, _ = nq.nq_decompose(w, m, N_BITS, 4, True)
        y = torch.empty((M, n), dtype=torch.bfloat16, device=dev)
        row = {}
        for name, fn in (("full_bit", lambda: nq.nq_gemm_full(x, w, sc, ACT_SCALE, y_out=y)),
                         ("part_bit", lambda: nq.nq_gemm_part(x, hi, n, N_BITS, 4, sc, ACT_SCALE, y_out=y))):
            ts = []
            for rep in range(5):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                if rep:
                    ts.append(a.elapsed_time(b))
            ms = float(np.median(ts))
            row[name] = {"ms": round(ms, 4), "tops": round(2.0 * M * n * k / (ms * 1e-3) / 1e12, 1)}
        res[f"K{k}_N{n}"] = row
    res["M"] = M
    out["vit_b16_linears_int8_4"] = res
    nq.nq_device_status()
    return out


def _run_e2e(nq, torch, sizes, host, state, args, world):
    """The GEMM sweep fed from pinned host buffers, every GEMM result read back: H2D + kernels + D2H timed.  The
    result copies run on a second stream beside the following kernels; the step ends after the last copy."""
    pinned = {s: {k: torch.from_numpy(host[s][k]).pin_memory() for k in ("W", "X", "mask", "w_scale")} for s in sizes}
    ybuf = {s: torch.empty((s, s), dtype=torch.bfloat16).pin_memory() for s in sizes}     # contiguous: plain 1-D copies
    steps = max(1, min(args.steps, args.e2e_steps))
    stream = torch.cuda.current_stream()
    counts = {"h2d": 0, "d2h": 0}
    # results leave on a copy stream while the next kernels run: two device result buffers per size take turns, a
    # kernel may only overwrite a buffer once the copy that read it has finished
    copy_stream = torch.cuda.Stream()
    ydev = {s: [state[s]["y"], torch.empty_like(state[s]["y"])] for s in sizes}
    copied = {s: [None, None] for s in sizes}
    turn = {s: 0 for s in sizes}

    def result_out(s, launch):
        i = turn[s]
        turn[s] ^= 1
        if copied[s][i] is not None:
            stream.wait_event(copied[s][i])
        launch(ydev[s][i])
        done = torch.cuda.Event()
        done.record(stream)
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(done)
            ybuf[s].copy_(ydev[s][i], non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(copy_stream)
        copied[s][i] = ev
        counts["d2h"] += s * s * 2

    def one():
        counts["h2d"] = counts["d2h"] = 0
        for s in sizes:
            d = state[s]
            for k in ("W", "X", "mask", "w_scale"):
                d[k].copy_(pinned[s][k], non_blocking=True)
                counts["h2d"] += pinned[s][k].numel() * pinned[s][k].element_size()
            for h in HS:
                nq.nq_decompose(d["W"], d["mask"], N_BITS, h, True, out_high=d["hi"][h], out_low=d["lo"][h])
                nq.nq_drop_low(d["W"], d["lo"][h], N_BITS, h, True, out_high=d["hi"][h])
                nq.nq_recompose(d["hi"][h], d["lo"][h], s, s, N_BITS, h, True, out=d["w_rec"])
                result_out(s, lambda y: nq.nq_gemm_part(d["X"], d["hi"][h], s, N_BITS, h, d["w_scale"], ACT_SCALE, y_out=y))
            result_out(s, lambda y: nq.nq_gemm_full(d["X"], d["w_rec"], d["w_scale"], ACT_SCALE, y_out=y))
        stream.wait_stream(copy_stream)               # the step ends when its last result is on the host

    one()
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        one()
    b.record(stream)
    torch.cuda.synchronize()
    return {"ms_per_step": a.elapsed_time(b) / steps, "h2d": counts["h2d"], "d2h": counts["d2h"]}


# --------------------------------------------------------------------------- oracle arm / CPU baseline
def oracle_sample(sizes, host, budget_rows):
    """The oracle as it stands on a bounded sample of the same workload: for one size, `budget_rows`
    rows of X through both GEMM modes + dequantisation, plus the three codec functions on a row band."""
    import oracle
    s = sizes[min(1, len(sizes) - 1)]
    d = host[s]
    rows = min(budget_rows, s)
    band = min(1024, s)
    t0 = time.time()
    wh, wl_ = oracle.decompose(d["W"][:band], d["mask"][:band], N_BITS, 6, True)
    oracle.recompose(wh, wl_, N_BITS, 6)
    oracle.drop_low(d["W"][:band], wl_, N_BITS, 6)
    t_codec = time.time() - t0
    wh_full, _ = oracle.decompose(d["W"], d["mask"], N_BITS, 6, True)      # set-up for the part-bit sample, untimed
    t1 = time.time()
    acc = oracle.gemm_acc(d["X"][:rows], d["W"])
    oracle.dequant(acc, d["w_scale"], ACT_SCALE, 0)
    accp = oracle.gemm_acc(d["X"][:rows], wh_full)
    oracle.dequant(accp, d["w_scale"], ACT_SCALE, 2)
    t_gemm = time.time() - t1
    return {"ops": 2 * 2.0 * rows * s * s, "seconds": t_gemm + t_codec, "cores": oracle.num_threads(),
            "sample": f"size {s}: {rows} of {s} rows of X through full-bit and part-bit (h=6) GEMM + dequant, and "
                      f"decompose / recompose / drop-low on a {band}-row band of W"}


def cpu_baseline(sizes, host, budget_rows):
    r = oracle_sample(sizes, host, budget_rows)
    return {"value": round(r["ops"] / r["seconds"] / 1e12, 6), "unit": "TOPS", "cores": r["cores"], "kind": "oracle",
            "sample": r["sample"], "seconds": round(r["seconds"], 2)}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    sizes = tuple(int(s) for s in args.sizes.split(","))[:2]
    host = make_host_inputs(sizes)
    rows = max(8, args.cpu_rows // 4)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(sizes, host, 8)
    t_ops, t_sec, last = 0.0, 0.0, None
    for _ in range(args.steps):
        last = oracle_sample(sizes, host, rows)
        t_ops += last["ops"]
        t_sec += last["seconds"]
    value = t_ops / t_sec / 1e12
    return {
        "impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(1e3 * t_sec / args.steps, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "config 4: square nested GEMM sweep; each step is a bounded sample run by the CPU oracle"},
        "cpu_baseline": {"value": round(value, 6), "unit": "TOPS", "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"]},
        "e2e": {"value": round(value, 6), "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--sizes", default=",".join(map(str, SIZES)))
    ap.add_argument("--cpu-rows", type=int, default=256)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--conv-batch", type=int, default=32)
    ap.add_argument("--no-conv", dest="conv", action="store_false")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-model-switch", dest="model_switch", action="store_false")
    ap.add_argument("--no-model-rows", dest="model_rows", action="store_false",
                    help="skip the ResNet-101-shaped stack and the ViT-B linears (timed after the steps)")
    ap.add_argument("--model-batch", type=int, default=128)
    ap.add_argument("--nested-only", action="store_true",
                    help="time only the nested full-bit GEMM rows (8192^3, h in {4..7}) and print them")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        line = run_reference(args, rank, world)
        if line is not None:
            print(json.dumps(line), flush=True)
        return

    if args.nested_only:
        if rank == 0:
            import torch
            import paper_2506_17870_b200 as nq
            torch.cuda.set_device(local_rank)
            print(json.dumps({"rows": {"gemm_nested_8192": _nested_rows(nq, torch, torch.device("cuda", local_rank))}}), flush=True)
        return

    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        line = run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
