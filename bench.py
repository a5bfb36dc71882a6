#!/usr/bin/env python
"""Benchmark of the nested-INT8 hot path on B200.

One "step" is one pass of the whole path over the large square GEMM sweep (M = N = K in
{4096, 8192, 16384}, INT8 nesting INTh for h in {4, 5, 6, 7}): for every size and h

    decompose -> drop-low (page-out) -> recompose (page-in) -> part-bit GEMM,   plus one full-bit GEMM per size,

followed by the ResNet-18-shaped convolution stack (config 2: 20 convolutions + classifier, batch 32, NCHW
int8 activations, implicit GEMM, both modes; each mode's stack is replayed as one CUDA graph).  Before the warm-up
the INT8 tensor ceiling is measured (nq_i8_mma_ceiling: the GEMMs' tensor instruction issued from shared memory with
no loads, burst and sustained): roofline.frac is the GEMM launches' rate over the sustained ceiling.  After the timed steps the whole-model page-out / page-in of a
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


# DRAM traffic of the GEMM launches comes from an ncu capture, never from this file: profiles/gemm_dram_traffic.txt is
# written by `python -m paper_2506_17870_b200.ncu_traffic` from the capture's CSV and carries a hash of the kernel
# sources it was taken on.  When the sources have changed since, or a size was not captured, traffic is null.
TRAFFIC_FILE = ROOT / "profiles" / "gemm_dram_traffic.txt"


def gemm_traffic_bytes_per_launch(sizes):
    """(mean DRAM bytes of the GEMM launches of one step, note).  The mean runs over the captured sizes among
    `sizes` (h = 4..7 part-bit + one full-bit launch each); None with the reason when there is nothing valid."""
    from paper_2506_17870_b200 import ncu_traffic
    table, why = ncu_traffic.load(TRAFFIC_FILE)
    if table is None:
        return None, why
    have = [s for s in sizes if all((s, h) in table for h in list(HS) + [0])]
    if not have:
        return None, "no size of this run was captured"
    vals = [table[(s, h)] for s in have for h in list(HS) + [0]]
    note = "ncu dram__bytes_read + dram__bytes_write, mean over the GEMM launches of sizes %s" % ",".join(map(str, have))
    if len(have) < len(sizes):
        note += " only (%s not captured: over a gigabyte per launch)" % ",".join(str(s) for s in sizes if s not in have)
    return float(np.mean(vals)), note


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


# --------------------------------------------------------------------------- measured INT8 tensor ceiling
def measure_int8_ceiling(nq, torch, gpu_index, seconds=2.0):
    """The issue-only rate of the tensor instruction the GEMMs use (nq_i8_mma_ceiling: tcgen05.mma kind::i8 on CTA
    pairs, operands parked in shared memory, accumulators in tensor memory, no loads, no epilogue), in TOP/s.
    burst      best of five 1 ms launches after the GPU has idled for half a second (a kernel timed alone)
    sustained  median over the second half of about `seconds` of back-to-back 10 ms launches (a kernel inside a
               long hot step: the 1 kW power limit has pulled the clock down by then)
    with the median SM clock sampled during the sustained run."""
    stream = torch.cuda.current_stream()

    def launch(iters):
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ops = nq.nq_i8_mma_ceiling(iters)
        b.record(stream)
        return a, b, ops

    launch(400)
    torch.cuda.synchronize()
    nq.nq_device_status()
    time.sleep(0.5)
    burst = 0.0
    for _ in range(5):
        a, b, ops = launch(3700)
        torch.cuda.synchronize()
        burst = max(burst, ops / (a.elapsed_time(b) * 1e-3) / 1e12)
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.2)
    t0 = time.time()
    evs = []
    while time.time() - t0 < seconds and len(evs) < 400:
        for _ in range(8):
            evs.append(launch(37000))
        evs[-1][1].synchronize()
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0 + 0.5 * (t1 - t0), t1)
    rates = [ops / (a.elapsed_time(b) * 1e-3) / 1e12 for a, b, ops in evs[len(evs) // 2:]]
    nq.nq_device_status()
    return {"burst_tops": round(burst, 1), "sustained_tops": round(float(np.median(rates)), 1),
            "sustained_sm_mhz": clocks.get("sm_mhz"), "sustained_reasons": clocks.get("reasons"),
            "launches": len(evs), "how": "nq_i8_mma_ceiling: 74 CTA pairs issuing tcgen05.mma.cta_group::2.kind::i8 "
                                         "256x256x32 from shared memory into tensor memory, no loads"}


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

    conv_graphs = {}
    if have_conv and args.graphs:
        for part in (False, True):
            g = capture_stack(torch, conv_state, lambda cs: _run_conv(nq, cs, part))
            if g is not None:
                conv_graphs[part] = g

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
        # config 2: each stack is one CUDA-graph launch (layout pre-pass + contraction of every layer, in order) when
        # the capture succeeded, otherwise layer by layer
        if len(conv_graphs) == 2:
            timed(("conv_stack_graph", "full_bit", 0), lambda: conv_graphs[False].replay(), record, 2 * len(conv_layers))
            timed(("conv_stack_graph", "part_bit", 0), lambda: conv_graphs[True].replay(), record, 2 * len(conv_layers))
        else:
            for L, cs in zip(conv_layers, conv_state):
                timed(("conv_full", L.name, 0), lambda: _run_conv(nq, cs, False), record, 2)   # layout pre-pass + contraction
                timed(("conv_part", L.name, 0), lambda: _run_conv(nq, cs, True), record, 2)

    ops_gemm_sweep = sum(2.0 * s ** 3 * (len(HS) + 1) for s in sizes)
    ops_step = ops_gemm_sweep
    for L in conv_layers:
        M, N, K = L.gemm_view(args.conv_batch)
        ops_step += 2 * 2.0 * M * N * K

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    ceiling = measure_int8_ceiling(nq, torch, local_rank) if args.ceiling else None
    peaks = measured_peaks()
    peaks["int8_tops"] = ceiling["sustained_tops"] if ceiling else 2.0 * peaks["bf16_tflops_sustained"]
    peaks["int8_source"] = "measured ceiling (sustained)" if ceiling else "2 x bf16 sustained"
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
    model_rows = _model_rows(nq, torch, wl, dev, args.model_batch, peaks) if (rank == 0 and args.model_rows and have_conv) else None

    total_ms, e2e["ms_per_step"] = max_over_ranks([total_ms, e2e["ms_per_step"]], world, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_tops(world, ops_step, ms_per_step)
    if rank != 0:
        return None

    rows = _summarise_rows(events, conv_layers, args.conv_batch, peaks)
    if have_conv:
        rows.update(_config2_rows(nq, torch, wl, conv_layers, conv_state, args.conv_batch, peaks, events))
    gemm_ms, gemm_ops, gemm_n = 0.0, 0.0, 0
    for (kind, s, h), pairs in events.items():
        if kind in ("gemm_full", "gemm_part"):
            for a, b in pairs:
                gemm_ms += a.elapsed_time(b)
                gemm_ops += 2.0 * s ** 3
                gemm_n += 1
    # Denominator: the measured ceiling of the INT8 tensor instruction on this GPU (sustained: these launches run
    # inside a long hot step).  Alongside: its burst figure, 2 x the measured bf16 cuBLAS figures (dense INT8 :
    # bf16 nominal ratio 4.5 : 2.25) and the nominal 4.5 POP/s.
    derived_burst, derived_sustained = 2.0 * peaks["bf16_tflops"], 2.0 * peaks["bf16_tflops_sustained"]
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    if ceiling is not None:
        int8_peak, peak_source = ceiling["sustained_tops"], "measured in this run: sustained issue-only rate of tcgen05.mma kind::i8 (nq_i8_mma_ceiling)"
    else:
        int8_peak, peak_source = derived_sustained, "derived: 2 x the %s bf16 sustained figure" % peaks["source"]
    traffic, traffic_note = gemm_traffic_bytes_per_launch(sizes)
    roofline = {
        "bound": "tensor", "kernel": "contraction_pair_kernel / contraction_kernel (tcgen05 kind::i8): every GEMM launch of the timed steps",
        "achieved": round(achieved, 1), "peak": round(int8_peak, 1), "unit": "TOP/s",
        "frac": round(achieved / int8_peak, 4), "peak_source": peak_source,
        "int8_ceiling": ceiling,
        "frac_vs_measured_burst": round(achieved / ceiling["burst_tops"], 4) if ceiling else None,
        "frac_vs_2x_bf16_burst": round(achieved / derived_burst, 4),
        "frac_vs_2x_bf16_sustained": round(achieved / derived_sustained, 4),
        "frac_vs_nominal_4500": round(achieved / 4500.0, 4),
        "launches": gemm_n, "avg_launch_ms": round(gemm_ms / max(gemm_n, 1), 4),
        "traffic": traffic, "traffic_note": traffic_note,
        "algorithmic_bytes_per_launch": float(np.mean([s * s * (1 + (h / 8.0 if h else 1.0) + 2) for s in sizes for h in list(HS) + [0]])),
    }
    conv_note = (", + config 2: the ResNet-18-shaped stack (%d layers), batch %d, NCHW int8 in, both modes%s"
                 % (len(conv_layers), args.conv_batch, ", each stack one CUDA-graph launch" if len(conv_graphs) == 2 else "")
                 if have_conv else "")
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
        "e2e": {"value": round(whole_job_tops(world, ops_gemm_sweep, e2e["ms_per_step"]), 3), "unit": "TOPS",
                "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": round(e2e["ms_per_step"], 3), "ops_per_step": ops_gemm_sweep,
                "covers": "the GEMM sweep (codec + both GEMM modes), whose ops alone are counted; no convolution stack"},
        "roofline": roofline, "rows": rows,
    }
    if model_switch is not None:
        line["rows"]["model_switch"] = model_switch
        line["rows"]["word64_convert_8192"] = _word64_rows(nq, torch, dev)
        line["rows"]["gemm_nested_8192"] = _nested_rows(nq, torch, dev, peaks)
        line["rows"]["gemm_output_types_config4"] = _output_type_rows(nq, torch, state, sizes, peaks)
    if model_rows is not None:
        line["rows"].update(model_rows)
    if have_conv and args.chains:
        line["rows"]["resnet18_chain_int8_6"] = _chain_rows(nq, torch, wl, dev, peaks, wl.resnet18_layers(), 2, args.conv_batch)
        if args.model_rows:
            line["rows"]["resnet101_chain_int8_6"] = _chain_rows(nq, torch, wl, dev, peaks, wl.resnet101_layers(), 3, args.model_batch)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(sizes, host, args.cpu_rows)
    return line


def layer_roofline_us(M, N, K, in_bytes, weight_bytes, out_bytes, peaks):
    """Lower bound of one layer's time: max(integer ops / INT8 tensor ceiling, algorithmic bytes / HBM copy bandwidth),
    the activations read once, the weights once, the output written once."""
    t_ops = 2.0 * M * N * K / (peaks["int8_tops"] * 1e12)
    t_mem = (in_bytes + weight_bytes + out_bytes) / (peaks["hbm_gbs"] * 1e9)
    return 1e6 * max(t_ops, t_mem)


def conv_roofline_us(L, batch, part, h, out_esize, peaks):
    M, N, K = L.gemm_view(batch)
    return layer_roofline_us(M, N, K, batch * L.Cin * L.H * L.W, N * K * (h / 8.0 if part else 1.0), M * N * out_esize, peaks)


def _frac(t, peaks):
    return {"frac_int8_ceiling": round(t / peaks["int8_tops"], 3),
            "frac_2x_bf16_burst": round(t / (2.0 * peaks["bf16_tflops"]), 3),
            "frac_nominal_4500": round(t / 4500.0, 3)}


def _summarise_rows(events, conv_layers, conv_batch, peaks):
    out = {"gemm_full": {}, "gemm_part": {}, "codec": {}}
    hbm = peaks["hbm_gbs"]
    codec_bytes = {"decompose": 1 + 1 + 9 / 8, "page_out": 1 + 9 / 8, "page_in": 9 / 8 + 1}   # per weight, n = 8
    agg = {}
    for (kind, s, h), pairs in events.items():
        ms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
        if kind == "gemm_full":
            t = 2.0 * s ** 3 / (ms * 1e-3) / 1e12
            out["gemm_full"][str(s)] = {"tops": round(t, 1), "ms": round(ms, 4), **_frac(t, peaks)}
        elif kind == "gemm_part":
            t = 2.0 * s ** 3 / (ms * 1e-3) / 1e12
            out["gemm_part"].setdefault(str(s), {})[f"h{h}"] = {"tops": round(t, 1), "ms": round(ms, 4), **_frac(t, peaks)}
        elif kind in codec_bytes:
            agg.setdefault((kind, s), []).append((codec_bytes[kind] * s * s / (ms * 1e-3) / 1e9, h, ms))
        elif kind in ("conv_full", "conv_part"):
            L = next(l for l in conv_layers if l.name == s)
            M, N, K = L.gemm_view(conv_batch)
            t = 2.0 * M * N * K / (ms * 1e-3) / 1e12
            roof = conv_roofline_us(L, conv_batch, kind == "conv_part", CONV_H, 2, peaks)
            out.setdefault(kind, {})[s] = {"tops": round(t, 1), "ms": round(ms, 4), "gemm_view": [M, N, K],
                                           "roofline_us": round(roof, 2), "frac_roofline": round(roof / (ms * 1e3), 3)}
    for kind in ("conv_full", "conv_part"):
        if kind in out:
            tot_ms = sum(v["ms"] for v in out[kind].values())
            tot_ops = sum(2.0 * v["gemm_view"][0] * v["gemm_view"][1] * v["gemm_view"][2] for v in out[kind].values())
            roof = sum(v["roofline_us"] for v in out[kind].values())
            out[kind + "_stack"] = {"ms": round(tot_ms, 4), "tops": round(tot_ops / (tot_ms * 1e-3) / 1e12, 1),
                                    "layers": len(out[kind]), "roofline_sum_us": round(roof, 1),
                                    "frac_roofline": round(roof / (tot_ms * 1e3), 3),
                                    "roofline": "per layer max(ops / INT8 ceiling, (activations + weights + bf16 output) / HBM), summed"}
    for (kind, s), vals in agg.items():
        g = float(np.mean([v[0] for v in vals]))
        row = {"gbs": round(g, 0), "frac_hbm": round(g / hbm, 3)}
        if kind == "page_in":
            # the paper's switching-overhead model counts only the bytes paged in, P_low = (l + 1) / 8 per weight
            row["paper_model_p_low_gbs"] = {f"h{h}": round((N_BITS - h + 1) / 8.0 * s * s / (ms * 1e-3) / 1e9, 0) for _, h, ms in vals}
        out["codec"].setdefault(kind, {})[str(s)] = row
    out["codec"]["algorithmic_bytes_per_weight"] = codec_bytes
    out["peaks"] = {"int8_tops": peaks["int8_tops"], "int8_source": peaks["int8_source"], "hbm_gbs": hbm,
                    "bf16_tflops": peaks["bf16_tflops"], "source": peaks["source"]}
    return out


def _config2_rows(nq, torch, wl, conv_layers, conv_state, conv_batch, peaks, events):
    """Config 2 layer by layer (outside the timed steps: own CUDA events per layer, median of 3 passes), each layer
    against its roofline max(ops / INT8 ceiling, algorithmic bytes / HBM); the stack with NHWC input (no layout
    pre-pass) and with fp32 output; and the graph launches of the timed steps."""
    out = {}
    ops = sum(2.0 * float(np.prod(L.gemm_view(conv_batch))) for L in conv_layers)
    for part in (False, True):
        kind = "conv_part" if part else "conv_full"
        ms_l = time_layers(torch, conv_state, lambda cs: _run_conv(nq, cs, part))
        rows, roof_sum = {}, 0.0
        for L, ms in zip(conv_layers, ms_l):
            M, N, K = L.gemm_view(conv_batch)
            roof = conv_roofline_us(L, conv_batch, part, CONV_H, 2, peaks)
            roof_sum += roof
            rows[L.name] = {"tops": round(2.0 * M * N * K / (float(ms) * 1e-3) / 1e12, 1), "us": round(float(ms) * 1e3, 1),
                            "gemm_view": [M, N, K], "roofline_us": round(roof, 2), "frac_roofline": round(roof / (float(ms) * 1e3), 3)}
        out[kind] = rows
        tot = float(ms_l.sum())
        stack = {"ms": round(tot, 4), "tops": round(ops / (tot * 1e-3) / 1e12, 1), "layers": len(conv_layers),
                 "roofline_sum_us": round(roof_sum, 1), "frac_roofline": round(roof_sum / (tot * 1e3), 3),
                 "roofline": "per layer max(ops / INT8 ceiling, (activations + weights + bf16 output) / HBM), summed"}
        pairs = events.get(("conv_stack_graph", "part_bit" if part else "full_bit", 0))
        if pairs:
            gms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
            stack["graph_ms_in_step"] = round(gms, 4)
            stack["graph_frac_roofline"] = round(roof_sum / (gms * 1e3), 3)
        out[kind + "_stack"] = stack
    # the same stack fed NHWC activations (no transposing pre-pass; the stem still builds its patch matrix), and with fp32 output
    nhwc = []
    for L, cs in zip(conv_layers, conv_state):
        c = dict(cs)
        c["x"] = cs["x"].permute(0, 2, 3, 1).contiguous()
        c["desc"] = nq.nq_conv_desc(conv_batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 0)
        c["y32"] = torch.empty(cs["y"].shape, dtype=torch.float32, device=cs["y"].device)
        nhwc.append(c)
    for part in (False, True):
        roof = sum(conv_roofline_us(L, conv_batch, part, CONV_H, 2, peaks) for L in conv_layers)
        row, _ = stack_row(torch, nhwc, lambda cs: _run_conv(nq, cs, part), ops, roof)
        out[("conv_part" if part else "conv_full") + "_stack_nhwc_in"] = row
        base = out[("conv_part" if part else "conv_full") + "_stack"]
        base["nchw_prepass_ms"] = round(base["ms"] - row["ms"], 4)
    roof = sum(conv_roofline_us(L, conv_batch, False, CONV_H, 4, peaks) for L in conv_layers)
    out["conv_full_stack_nhwc_in_fp32_out"], _ = stack_row(
        torch, nhwc, lambda cs: nq.nq_conv_implicit_gemm(cs["x"], cs["w"], cs["desc"], cs["ws"], cs["act"], part_bit=False,
                                                         workspace=cs["work"], y_out=cs["y32"]), ops, roof)
    return out


def _chain_rows(nq, torch, wl, dev, peaks, layers, config, batch):
    """A ResNet-shaped model as ONE dependent chain on the device (stem, max pooling, residual blocks with the skip
    tensor added in the epilogue, global average pooling, classifier): INT8 activations hand over between layers, NCHW
    int8 input.  Scales are calibrated on the device first (set-up).  Timed per pass, layer by layer launches and as
    one CUDA-graph launch, in full-bit, part-bit and nested full-bit mode; the roofline of a pass is the sum over layers
    of max(ops / INT8 ceiling, (input + weights + INT8 output + skip tensor) / HBM) plus the pooling passes' bytes."""
    from paper_2506_17870_b200.chain import ResNetChain
    plan = wl.resnet_chain_plan(layers)
    weights = wl.chain_weights(config, layers)
    model = ResNetChain(layers, plan, weights, batch, 0.02, n_bits=N_BITS, h_bits=CONV_H, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.BASE_SEED + 7000 + config)
    x = torch.randint(0, 128, (batch, 3, 224, 224), dtype=torch.int8, device=dev, generator=gen)
    by = {L.name: L for L in layers}
    ops = 0.0
    out = {"batch": batch, "steps": len(plan), "kernels_per_pass": model.kernels_per_pass()}
    for mode in ("full", "part", "nested"):
        model.calibrate(x, "part" if mode == "part" else "full")
        wbytes = {"full": 1.0, "part": CONV_H / 8.0, "nested": (N_BITS + 1) / 8.0}[mode]
        roof, ops = 0.0, 0.0
        for st in plan:
            if st["op"] in ("conv", "fc"):
                L = by[st["layer"]]
                M, N, K = L.gemm_view(batch)
                ops += 2.0 * M * N * K
                out_b = M * N * (4 if st["op"] == "fc" else 1) + (M * N if st.get("skip") else 0)
                roof += layer_roofline_us(M, N, K, batch * L.Cin * L.H * L.W, N * K * wbytes, out_b, peaks)
            else:
                roof += 1e6 * (model.t[st["src"]].numel() + model.t[st["dst"]].numel()) / (peaks["hbm_gbs"] * 1e9)
        ts = []
        for rep in range(5):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            model.run(x, mode)
            b.record()
            torch.cuda.synchronize()
            if rep:
                ts.append(a.elapsed_time(b))
        ms = float(np.median(ts))
        row = {"ms": round(ms, 3), "tops": round(ops / (ms * 1e-3) / 1e12, 1), "roofline_sum_ms": round(roof / 1e3, 3),
               "frac_roofline": round(roof / 1e3 / ms, 3)}
        g = capture_stack(torch, [None], lambda _: model.run(x, mode))
        if g is not None:
            gms = time_graph(torch, g)
            row["graph_ms"] = round(gms, 3)
            row["graph_frac_roofline"] = round(roof / 1e3 / gms, 3)
            del g
        out[mode] = row
    nq.nq_device_status()
    out["tera_ops_per_pass"] = round(ops / 1e12, 3)
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
            if kind == "page_in":       # the paper's switching-overhead model counts only the paged bytes, P_low
                res[kind]["paper_model_p_low_gbs"] = round(weights * (N_BITS - h + 1) / 8.0 / (ms * 1e-3) / 1e9, 0)
        res["weights"] = weights
        res["tensors"] = len(shapes)
        res["algorithmic_mb"] = round(nbytes / 1e6, 1)
        out[name] = res
    return out


def _nested_rows(nq, torch, dev, peaks):
    """The full-bit layer computed straight from packed w_high and compensated w_low (no INT8 copy of the weights):
    8192^3, median of 5 launches per nesting, against the INT8 ceiling; outputs checked equal to the full-bit GEMM's."""
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
        out[f"h{h}"] = {"tops": round(t, 1), "ms": round(ms, 4), **_frac(t, peaks),
                        "weight_bytes_per_element": (N_BITS + 1) / 8, "equals_full_bit": bool(torch.equal(y, ref))}
    return out


def _output_type_rows(nq, torch, state, sizes, peaks):
    """Config 4 with the other two output types, timed once each (median of 3 launches after a warm-up launch):
    fp32 Y, and the raw INT32 accumulators with no Y.  Full-bit and part-bit h = 6."""
    out = {}
    for s in sizes:
        d = state[s]
        y32 = torch.empty((s, s), dtype=torch.float32, device=d["X"].device)
        acc = torch.empty((s, s), dtype=torch.int32, device=d["X"].device)
        row = {}
        for name, fn in (
                ("full_fp32", lambda: nq.nq_gemm_full(d["X"], d["w_rec"], d["w_scale"], ACT_SCALE, y_out=y32)),
                ("part_h6_fp32", lambda: nq.nq_gemm_part(d["X"], d["hi"][6], s, N_BITS, 6, d["w_scale"], ACT_SCALE, y_out=y32)),
                ("full_int32", lambda: nq.nq_gemm_full(d["X"], d["w_rec"], d["w_scale"], ACT_SCALE, acc_out=acc, y_dtype=None)),
                ("part_h6_int32", lambda: nq.nq_gemm_part(d["X"], d["hi"][6], s, N_BITS, 6, d["w_scale"], ACT_SCALE, acc_out=acc, y_dtype=None))):
            ts = []
            for rep in range(4):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                if rep:
                    ts.append(a.elapsed_time(b))
            ms = float(np.median(ts))
            t = 2.0 * s ** 3 / (ms * 1e-3) / 1e12
            row[name] = {"tops": round(t, 1), "ms": round(ms, 4), **_frac(t, peaks)}
        out[str(s)] = row
        del y32, acc
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


def time_layers(torch, prepared, call, reps=4):
    """ms per layer: every layer between its own pair of CUDA events, median over reps - 1 passes (first discarded)."""
    per_layer = []
    for rep in range(reps):
        evs = []
        for cs in prepared:
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            call(cs)
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        if rep:
            per_layer.append([a.elapsed_time(b) for a, b in evs])
    return np.median(np.array(per_layer), axis=0)


def capture_stack(torch, prepared, call):
    """The whole stack as ONE CUDA graph (every launch of every layer, in order), or None when capture fails.  The
    library calls only enqueue kernels on the current stream, so they can be recorded once and replayed."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for cs in prepared:
                call(cs)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for cs in prepared:
                call(cs)
        return g
    except Exception:
        torch.cuda.synchronize()
        return None


def time_graph(torch, g, reps=6):
    ts = []
    for rep in range(reps):
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        if rep:
            ts.append(a.elapsed_time(b))
    return float(np.median(ts))


def stack_row(torch, prepared, call, ops, roofline_us, graph=True):
    """One variant of a stack: layer by layer (sum of per-layer medians) and as one graph launch."""
    ms_layers = time_layers(torch, prepared, call)
    row = {"ms": round(float(ms_layers.sum()), 3), "tops": round(ops / (float(ms_layers.sum()) * 1e-3) / 1e12, 1),
           "roofline_sum_ms": round(roofline_us / 1e3, 3), "frac_roofline": round(roofline_us / 1e3 / float(ms_layers.sum()), 3)}
    if graph:
        g = capture_stack(torch, prepared, call)
        if g is not None:
            gms = time_graph(torch, g)
            row["graph_ms"] = round(gms, 3)
            row["graph_frac_roofline"] = round(roofline_us / 1e3 / gms, 3)
            del g
    return row, ms_layers


def _model_rows(nq, torch, wl, dev, conv_batch, peaks):
    """Configs 3 and 5 through both modes on seeded device-side inputs of the stated shapes and distributions: the
    ResNet-101-shaped stack (104 convolutions + classifier, batch `conv_batch`, int8 activations ~ U{0..127}, INT8
    nesting INT6) and the ViT-B/16 linears (M = 256 * 197 tokens, INT8 nesting INT4).  Every variant is timed layer by
    layer (own pair of CUDA events per layer, median of 3 passes) and as one CUDA-graph launch of the whole stack;
    inputs of one pass exceed L2, so nothing is flushed.  `frac_roofline` = sum over layers of max(ops / INT8 ceiling,
    algorithmic bytes / HBM copy bandwidth) over the measured time."""
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.BASE_SEED + 3000)
    out = {}
    # ---- config 3
    layers = wl.resnet101_layers()
    xs, prepared = {}, []
    y_elems = max(conv_batch * L.Ho * L.Wo * L.Cout for L in layers)
    ybuf = torch.empty(y_elems, dtype=torch.float32, device=dev)
    work_bytes = 0
    for L in layers:
        key = (L.Cin, L.H, L.W)
        if key not in xs:
            xs[key] = torch.randint(0, 128, (conv_batch, L.Cin, L.H, L.W), dtype=torch.int8, device=dev, generator=gen)
            xs[("nhwc",) + key] = xs[key].permute(0, 2, 3, 1).contiguous()
        args5 = (conv_batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad)
        desc = nq.nq_conv_desc(*args5, 1)
        desc_nhwc = nq.nq_conv_desc(*args5, 0)
        w, ws = _device_conv_weights(torch, L, dev, gen)
        m = torch.randint(0, 2, (L.Cout, w.stride(0)), dtype=torch.uint8, device=dev, generator=gen)[:, :L.K]
        hi, lo = nq.nq_decompose(w, m, N_BITS, CONV_H, True)
        work_bytes = max(work_bytes, nq.nq_conv_workspace_bytes(desc), nq.nq_conv_workspace_bytes(desc_nhwc))
        n_out = conv_batch * L.Ho * L.Wo * L.Cout
        shape = (conv_batch, L.Ho, L.Wo, L.Cout)
        prepared.append({"L": L, "desc": desc, "desc_nhwc": desc_nhwc, "w": w, "hi": hi, "lo": lo, "ws": ws, "x": xs[key],
                         "x_nhwc": xs[("nhwc",) + key], "act": 0.02,
                         "y": ybuf.view(torch.bfloat16)[:n_out].view(shape), "y32": ybuf[:n_out].view(shape),
                         "yq": ybuf.view(torch.int8)[:n_out].view(shape)})
    work = torch.empty(work_bytes + 2048, dtype=torch.uint8, device=dev)
    for cs in prepared:
        cs["work"] = work
    ops = sum(2.0 * float(np.prod(L.gemm_view(conv_batch))) for L in layers)

    def roof(part, esize):
        return sum(conv_roofline_us(L, conv_batch, part, CONV_H, esize, peaks) for L in layers)

    def conv(cs, part, nhwc, y):
        nq.nq_conv_implicit_gemm(cs["x_nhwc"] if nhwc else cs["x"], cs["hi"] if part else cs["w"],
                                 cs["desc_nhwc"] if nhwc else cs["desc"], cs["ws"], cs["act"], part_bit=part, n_bits=N_BITS,
                                 h_bits=CONV_H, workspace=cs["work"], y_out=cs[y])

    res = {}
    per_layer_nhwc = None
    for part in (False, True):
        mode = "part_bit" if part else "full_bit"
        res[mode], _ = stack_row(torch, prepared, lambda cs: conv(cs, part, False, "y"), ops, roof(part, 2))
        res[mode + "_nhwc_in"], ms_l = stack_row(torch, prepared, lambda cs: conv(cs, part, True, "y"), ops, roof(part, 2))
        if not part:
            per_layer_nhwc = ms_l
        # what the NCHW -> NHWC pre-pass (a transposing kernel in front of every layer) costs: the difference
        res[mode]["nchw_prepass_ms"] = round(res[mode]["ms"] - res[mode + "_nhwc_in"]["ms"], 3)
    res["full_bit_nhwc_in_fp32_out"], _ = stack_row(torch, prepared, lambda cs: conv(cs, False, True, "y32"), ops, roof(False, 4))
    # the full-bit stack again with no INT8 copy of the weights: every layer rebuilds them from the two packed parts
    res["nested_full_bit"], _ = stack_row(
        torch, prepared, lambda cs: nq.nq_conv_implicit_gemm_nested(cs["x"], cs["hi"], cs["lo"], cs["desc"], cs["ws"], cs["act"],
                                                                    n_bits=N_BITS, h_bits=CONV_H, workspace=cs["work"], y_out=cs["y"]),
        ops, roof(False, 2), graph=False)
    # chained form: NHWC int8 activations in, the next layer's INT8 activations out (requantising epilogue with ReLU),
    # no layout pre-pass; every layer still runs on its own input
    for part in (False, True):
        res["chained_int8_out_" + ("part_bit" if part else "full_bit")], _ = stack_row(
            torch, prepared, lambda cs: nq.nq_conv_implicit_gemm_q8(cs["x_nhwc"], cs["hi"] if part else cs["w"], cs["desc_nhwc"],
                                                                    cs["ws"], cs["act"], 0.5, relu=True, part_bit=part, n_bits=N_BITS,
                                                                    h_bits=CONV_H, workspace=cs["work"], y_out=cs["yq"]),
            ops, roof(part, 1))
    res["chained_int8_out_nested_full_bit"], _ = stack_row(
        torch, prepared, lambda cs: nq.nq_conv_implicit_gemm_nested_q8(cs["x_nhwc"], cs["hi"], cs["lo"], cs["desc_nhwc"], cs["ws"],
                                                                       cs["act"], 0.5, relu=True, n_bits=N_BITS, h_bits=CONV_H,
                                                                       workspace=cs["work"], y_out=cs["yq"]),
        ops, roof(False, 1), graph=False)
    # per distinct layer shape, full-bit, NHWC in, bf16 out: where the stack's time goes against each layer's roofline
    shapes = {}
    for cs, ms in zip(prepared, per_layer_nhwc):
        L = cs["L"]
        key = (L.Cin, L.H, L.Cout, L.R, L.stride)
        e = shapes.setdefault(key, {"first": L.name, "count": 0, "ms": 0.0,
                                    "roofline_us": round(conv_roofline_us(L, conv_batch, False, CONV_H, 2, peaks), 2)})
        e["count"] += 1
        e["ms"] += float(ms)
    res["per_shape_full_bit_nhwc_in"] = [
        {"first": e["first"], "count": e["count"], "us_each": round(1e3 * e["ms"] / e["count"], 1), "roofline_us": e["roofline_us"],
         "frac_roofline": round(e["roofline_us"] / (1e3 * e["ms"] / e["count"]), 3)} for e in shapes.values()]
    res.update({"layers": len(layers), "batch": conv_batch, "weights": sum(L.weights for L in layers),
                "tera_ops_per_pass": round(ops / 1e12, 3)})
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
        for name, part, fn in (("full_bit", False, lambda: nq.nq_gemm_full(x, w, sc, ACT_SCALE, y_out=y)),
                               ("part_bit", True, lambda: nq.nq_gemm_part(x, hi, n, N_BITS, 4, sc, ACT_SCALE, y_out=y))):
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
            roof_us = layer_roofline_us(M, n, k, M * k, n * k * (0.5 if part else 1.0), M * n * 2, peaks)
            row[name] = {"ms": round(ms, 4), "tops": round(2.0 * M * n * k / (ms * 1e-3) / 1e12, 1),
                         "roofline_us": round(roof_us, 1), "frac_roofline": round(roof_us / (ms * 1e3), 3)}
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
    ap.add_argument("--cpu-rows", type=int, default=4096)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--conv-batch", type=int, default=32)
    ap.add_argument("--no-conv", dest="conv", action="store_false")
    ap.add_argument("--no-graphs", dest="graphs", action="store_false",
                    help="run the convolution stacks of the timed steps layer by layer instead of as CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-ceiling", dest="ceiling", action="store_false",
                    help="skip the 2 s measurement of the INT8 tensor ceiling (fractions then use 2 x bf16 sustained)")
    ap.add_argument("--no-model-switch", dest="model_switch", action="store_false")
    ap.add_argument("--no-model-rows", dest="model_rows", action="store_false",
                    help="skip the ResNet-101-shaped stack and the ViT-B linears (timed after the steps)")
    ap.add_argument("--model-batch", type=int, default=128)
    ap.add_argument("--no-chains", dest="chains", action="store_false",
                    help="skip the dependent-chain rows (ResNet-18-shaped at --conv-batch, ResNet-101-shaped at --model-batch)")
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
            pk = measured_peaks()
            pk["int8_tops"], pk["int8_source"] = 2.0 * pk["bf16_tflops_sustained"], "2 x bf16 sustained"
            print(json.dumps({"rows": {"gemm_nested_8192": _nested_rows(nq, torch, torch.device("cuda", local_rank), pk)}}), flush=True)
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
