#!/usr/bin/env python
"""Benchmark of the dense-GEMM hot path on B200.

A step is one pass of the whole path (tile loop, operand staging, K loop with
the accumulator resident, epilogue, store) over one batch of synthetic input:
the BF16 GEMM M = N = K = 8192 with FP32 output.  With N GPUs every rank owns
its own 8192-row block of A (M-sharded, B replicated: no collective on the data
path), so per-GPU work is fixed ("weak" scaling) and `value` sums all ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line on rank 0.  After the timed region of the headline workload
the same line gets a `configs` list: the other benchmark configurations (the FP32
256^3 GEMM, the blocked 1024^3 GEMM, the MLP layers, corners of the shape sweep),
each timed on its own by CUDA-graph replay with an L2 flush before every launch,
with the roofline that binds it.

    python bench.py --table [--only NAME] [--library] [--f32-tensor]

prints the full per-workload table (every configuration, the whole sweep, the
paper's MLP grid and the extra operand types) as markdown instead.

Run bare with --gpus N > 1 (no WORLD_SIZE in the environment) it starts the N
ranks itself, one per GPU, through torch.distributed.run on 127.0.0.1.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GEMM TFLOP/s (device-timed, 1 B200) and fraction of dense BF16/FP32 peak"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "bench_c4_bf16_8192_dram_traffic.json")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def workload(size=None):
    """The benchmark workload: configuration 4 (BF16 8192^3, FP32 output).  `size`
    shrinks M = N = K for profiler captures, which must stay small."""
    import dataclasses
    import nk_inputs
    w = nk_inputs.config(4)
    if size:
        w = dataclasses.replace(w, name=f"c4_bf16_{size}_profiling_size", M=size, N=size, K=size)
    return w


def recorded_traffic(kernel_name: str, shape) -> tuple:
    """DRAM bytes per launch of the benchmark kernel from the committed profiler capture, or
    (None, why) when the capture is of another kernel, another shape, or of kernel sources that
    have changed since (the record carries the hash of the sources it was taken from)."""
    if not os.path.exists(TRAFFIC_JSON):
        return None, "no capture on record"
    with open(TRAFFIC_JSON) as f:
        rec = json.load(f)
    if rec.get("kernel") != kernel_name or list(rec.get("shape", [])) != list(shape):
        return None, "the capture on record is of another kernel or shape"
    from paper_2511_13764_b200 import _build
    if rec.get("source_hash") != _build.source_hash():
        return None, "kernel sources changed since the capture"
    return float(rec["dram_read_bytes"]) + float(rec["dram_write_bytes"]), f"ncu capture of {rec.get('captured')}"


# --------------------------------------------------------------------------- reference arm
def oracle_sample_rate(w, B, rows_per_step, steps, warmup, seed_shift=0):
    """Time the CPU oracle, as it stands, on `rows_per_step` stratified rows of
    the workload per step.  Returns (TFLOP/s, seconds per step, threads)."""
    import numpy as np
    import nk_inputs
    import oracle
    threads = os.cpu_count() or 1
    rows = nk_inputs.stratified_rows(w.seed + seed_shift, w.M, rows_per_step)
    # only the sampled rows of A are needed: build them into a sparse full-size buffer
    A = np.zeros(w.M * w.K, dtype=np.uint16 if w.in_dtype == "bf16" else np.float32)
    for r in rows:
        A[r * w.K:(r + 1) * w.K] = nk_inputs.fill(w.seed, nk_inputs.TENSOR_A, w.K, w.dist_a[0], w.dist_a[1],
                                                  w.in_dtype, start=int(r) * w.K)
    times = []
    for s in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.gemm_workload(w, A, B, None, rows=rows, nthreads=threads, want_scale=False)
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    flops = 2.0 * len(rows) * w.N * w.K
    return flops / sec / 1e12, sec, threads, len(rows)


def workload_config(w, world=1):
    """The `config` object of the JSON line: it names the workload, so both arms print the same one."""
    e_in = 4 if w.in_dtype == "f32" else 2
    a_mb, b_mb, c_mb = (w.M * w.K * e_in) >> 20, (w.K * w.N * e_in) >> 20, (w.M * w.N * 4) >> 20
    return {"workload": w.name, "M": w.M, "N": w.N, "K": w.K, "in_dtype": w.in_dtype,
            "out_dtype": w.out_dtype, "layout": w.layout, "epilogue": w.epilogue,
            "l2": f"inputs larger than L2 (A {a_mb} MB + B {b_mb} MB + C {c_mb} MB per step)",
            "parallelism": f"M-sharded x{world}, B replicated, no collective"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import nk_inputs
    w = workload(args.size)
    B = nk_inputs.fill(w.seed, nk_inputs.TENSOR_B, w.K * w.N, w.dist_b[0], w.dist_b[1], w.in_dtype)
    # probe the oracle's speed on 8 rows, then size the per-step sample so the whole
    # run stays near two minutes
    _, probe_sec, threads, _ = oracle_sample_rate(w, B, 8, 1, 0)
    total_steps = args.steps + args.warmup
    rows = int(max(1, min(256, 120.0 / max(total_steps, 1) / (probe_sec / 8))))
    tf, sec, threads, nrows = oracle_sample_rate(w, B, rows, args.steps, args.warmup)
    sample = f"{nrows} stratified rows of the {w.M}x{w.N}x{w.K} problem per step (all {w.N} columns, full K)"
    cfg = workload_config(w, int(os.environ.get("WORLD_SIZE", "1")))
    out = {
        "impl": "reference", "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": cfg,
        "cpu_baseline": {"value": tf, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)
    return 0


# --------------------------------------------------------------------------- multi-rank plumbing
def shard_seed(seed: int, rank: int) -> int:
    """Seed of rank `rank`'s block of A rows (B keeps the workload's seed on every rank)."""
    return seed + 7919 * rank


def init_distributed(world: int, device=None):
    """One process per GPU: NCCL when a CUDA device is given, gloo otherwise (CPU tests)."""
    import torch.distributed as dist
    if world <= 1 or dist.is_initialized():
        return
    if device is not None:
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group("gloo")


def max_over_ranks(x: float, world: int, device=None) -> float:
    """MAX all-reduce of one float (the step time every rank measured)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank: float, world: int, ms_per_step: float) -> float:
    """Aggregate over all ranks: every rank does `flops_per_rank` per step (weak scaling)."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv) -> int:
    """Started bare with --gpus n > 1: run n ranks of this script, one per GPU, through
    torch.distributed.run with a loopback rendezvous, and hand back its exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.ok = False
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            pass

    def sample(self):
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {
                0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown",
            }
            for bit, n in names.items():
                if r & bit:
                    self.reasons.add(n)
        except Exception:
            pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# --------------------------------------------------------------------------- per-workload timing
def time_launch(launch, st, iters, flush, graph_pairs):
    """Median (and best) time in ms of `launch(cuda_stream)`, each call timed on its own after an
    L2 flush.  With `graph_pairs` a CUDA graph of that many (flush, launch) pairs is replayed and a
    graph of the flushes alone subtracted: CUDA-event stamps are a microsecond or two coarse on
    some boxes, the graph difference resolves a fraction of a microsecond, and the launches come
    without host gaps, as they would inside a captured pipeline."""
    import torch
    # a quarter of a second of idling first: a heavy row just before leaves the part power-throttled for
    # a while, which a short FMA-bound row would otherwise inherit
    torch.cuda.synchronize()
    time.sleep(0.25)
    for _ in range(3):
        launch(st.cuda_stream)
    torch.cuda.synchronize()
    if graph_pairs and flush is not None:
        side = torch.cuda.Stream()
        side.wait_stream(st)
        graphs = []
        for with_launch in (True, False):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                cs = torch.cuda.current_stream().cuda_stream
                for _ in range(graph_pairs):
                    flush.fill_(1)
                    if with_launch:
                        launch(cs)
            graphs.append(g)

        def replay_ms(g):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            g.replay()
            b.record(st)
            b.synchronize()
            return a.elapsed_time(b)

        # The two graphs are timed in turn, so that a drift of the clocks (the previous row may have
        # left the part power-throttled) hits both alike; the median of the differences is reported.
        for g in graphs:
            replay_ms(g)
        diffs = sorted(replay_ms(graphs[0]) - replay_ms(graphs[1]) for _ in range(max(5, iters // 2)))
        per = diffs[len(diffs) // 2] / graph_pairs
        return per, diffs[0] / graph_pairs
    times = []
    for _ in range(iters):
        if flush is not None:
            flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(st)
        launch(st.cuda_stream)
        b.record(st)
        b.synchronize()
        times.append(a.elapsed_time(b))
    times.sort()
    return times[len(times) // 2], times[0]


def time_workload(w, iters, flags=0, flush=None, graph_pairs=0, library=False, device=0):
    """Returns (median ms, best ms, kernel name, launches per run, library ms or None).  Operands are
    random values of the workload's types made on the device (this only measures; parity is the
    tests' business).  `library` also times torch.matmul (cuBLAS) on the same shape and element
    type (row-major operands, no epilogue, FP32 without TF32): context for the table, never part
    of the product path."""
    import torch
    import paper_2511_13764_b200 as nk
    dev = torch.device("cuda", device)
    tt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16, "s8": torch.int8, "s32": torch.int32,
          "e4m3": torch.uint8, "e5m2": torch.uint8}
    ein, eout = tt[w.in_dtype], tt[w.out_dtype]
    g = torch.Generator(device=dev).manual_seed(w.seed)
    if w.in_dtype == "s8":
        A = torch.randint(-128, 128, (w.M * w.K,), device=dev, generator=g, dtype=torch.int8)
        B = torch.randint(-128, 128, (w.K * w.N,), device=dev, generator=g, dtype=torch.int8)
        library = False      # no library column for INT8
    elif w.in_dtype in ("e4m3", "e5m2"):
        f8 = torch.float8_e4m3fn if w.in_dtype == "e4m3" else torch.float8_e5m2
        A = (torch.rand(w.M * w.K, device=dev, generator=g) * 2 - 1).to(f8)
        B = (torch.rand(w.K * w.N, device=dev, generator=g) * 2 - 1).to(f8)
        library = False      # nor for 8-bit floating point
    else:
        A = (torch.rand(w.M * w.K, device=dev, generator=g) * 2 - 1).to(ein)
        B = (torch.rand(w.K * w.N, device=dev, generator=g) * 2 - 1).to(ein)
    bias = (torch.randn(w.N, device=dev, generator=g) * 0.02).to(tt[w.bias_dtype]) if w.epilogue != "none" else None
    C = torch.empty(w.M * w.N, dtype=eout, device=dev)
    plan = nk.plan_for(w, device=device, flags=flags)
    wsb = plan.workspace_bytes
    ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream()

    def run(cs):
        plan.run(A, B, C, bias=bias, workspace=ws if wsb else None, workspace_bytes=wsb, stream=cs)

    med, best = time_launch(run, st, iters, flush, graph_pairs)
    plan.check()
    lib_ms = None
    if library:
        torch.backends.cuda.matmul.allow_tf32 = False
        A2, B2 = A.view(w.M, w.K), B.view(w.K, w.N)
        C2 = torch.empty(w.M, w.N, dtype=ein, device=dev)
        lib_ms, _ = time_launch(lambda cs: torch.matmul(A2, B2, out=C2), st, iters, flush, graph_pairs)
    return med, best, plan.kernel_name, plan.launches_per_run, lib_ms


def fma_peak_tflops(device=0) -> float:
    """FP32 FMA-pipe peak: SMs x 128 lanes x 2 flop x the maximum SM clock."""
    import torch
    prop = torch.cuda.get_device_properties(device)
    return prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12


def roofline_row(w, ms, peaks, fma_peak, split=False):
    """The roofline that binds workload `w` at the box's peaks, and the fraction `ms` reaches:
    (TFLOP/s, algorithmic GB/s, bound, peak, unit, frac).  8-bit operands run at twice the BF16
    rate on the tensor cores (nominal ratio applied to the measured BF16 peak); `split` marks FP32
    operands multiplied as six BF16 products (a sixth of the BF16 peak)."""
    tensor_peak, hbm_peak = float(peaks["bf16_tflops"]), float(peaks["hbm_gbs"])
    tf = w.flops / (ms * 1e-3) / 1e12
    gbs = w.algorithmic_bytes / (ms * 1e-3) / 1e9
    compute_peak = (tensor_peak / 6 if split else 2 * tensor_peak if w.in_dtype in ("s8", "e4m3", "e5m2")
                    else tensor_peak if w.in_dtype != "f32" else fma_peak)
    t_compute = w.flops / (compute_peak * 1e12)
    t_hbm = w.algorithmic_bytes / (hbm_peak * 1e9)
    if t_hbm >= t_compute:
        return tf, gbs, "hbm", hbm_peak, "GB/s", gbs / hbm_peak
    bound = "tensor/6" if split else "tensor" if w.in_dtype != "f32" else "alu"
    return tf, gbs, bound, compute_peak, "TFLOP/s", tf / compute_peak


def config_rows():
    """The configurations reported beside the headline: C1, C2, C3, the paper's MLP layers (flat B,
    and the widest one with VNNI-blocked operands), and the corners of the shape sweep."""
    import nk_inputs
    rows = [nk_inputs.config(1), nk_inputs.config(2), nk_inputs.config(3)]
    mlp = {w.name: w for w in nk_inputs.paper_mlp()}
    rows += [mlp["mlp_bf16_flat_1024"], mlp["mlp_bf16_flat_2048"], mlp["mlp_bf16_flat_4096"], mlp["mlp_bf16_vnni_4096"]]
    sweep = {w.name: w for w in nk_inputs.sweep()}
    rows += [sweep["c5_f32_16x16384x16384"], sweep["c5_bf16_16x16384x16384"],
             sweep["c5_f32_4096x4096x4096"], sweep["c5_bf16_4096x4096x4096"]]
    return rows


def time_configs(peaks, device=0, iters=9, graph_pairs=20):
    import torch
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=torch.device("cuda", device))
    fma = fma_peak_tflops(device)
    out = []
    for w in config_rows():
        med, best, kname, launches, _ = time_workload(w, iters, flush=flush, device=device,
                                                      graph_pairs=graph_pairs if w.flops < 5e11 else 0)
        tf, gbs, bound, peak, unit, frac = roofline_row(w, med, peaks, fma)
        out.append({"workload": w.name, "kernel": kname, "launches": launches, "us": med * 1e3, "value": tf,
                    "unit": UNIT, "alg_gbs": gbs, "bound": bound, "peak": peak, "peak_unit": unit, "frac": frac,
                    "flop": w.flops, "alg_bytes": w.algorithmic_bytes})
    del flush
    return out


def run_table(args):
    """Every workload, one row each, as a markdown table (and optionally JSON)."""
    import torch
    import nk_inputs
    import paper_2511_13764_b200 as nk
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    peaks = load_peaks()
    fma = fma_peak_tflops(0)
    flush = None if args.no_flush else torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    works = ([nk_inputs.config(i) for i in (1, 2, 3, 4)] + nk_inputs.sweep() + nk_inputs.paper_mlp() + nk_inputs.f16_set()
             + nk_inputs.s8_set() + nk_inputs.fp8_set() + nk_inputs.bt_set())
    rows = []
    print(f"| workload | kernel | launches | median us | TFLOP/s | alg. GB/s | bound | frac ({peaks['_source']}) |"
          + (" cuBLAS us |" if args.library else ""))
    print("|---|---|---|---|---|---|---|---|" + ("---|" if args.library else ""))
    todo = []
    for w in works:
        if args.only and not any(o in w.name for o in args.only.split(",")):
            continue
        todo.append((w, w.name, args.flags, False))
        if args.f32_tensor and w.in_dtype == "f32" and w.N % 8 == 0 and w.K % 8 == 0:
            todo.append((w, w.name + " +tensor", args.flags | nk.FLAG_F32_TENSOR, True))
    for w, label, flags, split in todo:
        med, best, kname, launches, lib_ms = time_workload(w, args.iters, flags=flags, flush=flush,
                                                           graph_pairs=args.graph if w.flops < 5e11 else 0,
                                                           library=args.library and not split)
        tf, gbs, bound, peak, unit, frac = roofline_row(w, med, peaks, fma, split)
        rows.append(dict(workload=label, kernel=kname, launches=launches, median_us=med * 1e3,
                         best_us=best * 1e3, tflops=tf, gbs=gbs, bound=bound, frac=frac,
                         library_us=None if lib_ms is None else lib_ms * 1e3))
        print(f"| {label} | {kname} | {launches} | {med * 1e3:.1f} | {tf:.1f} | {gbs:.0f} | {bound} | {frac:.3f} |"
              + (f" {lib_ms * 1e3:.1f} |" if lib_ms is not None else " |" if args.library else ""), flush=True)
    if not args.only or any(o in "x_quantize_s8_8192x8192" for o in args.only.split(",")):
        # the quantisation kernel of the INT8 path: an HBM stream of 4 bytes in and 1 byte out per element
        n = 8192 * 8192
        x = torch.rand(n, device="cuda") * 2 - 1
        q = torch.empty(n, dtype=torch.int8, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        times = []
        for i in range(args.iters + 3):
            if flush is not None:
                flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            nk.quantize_s8(x, q, n, 127.0, stream=st)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                times.append(e0.elapsed_time(e1))
        med = sorted(times)[len(times) // 2]
        gbs = 5.0 * n / (med * 1e-3) / 1e9
        frac = gbs / float(peaks["hbm_gbs"])
        rows.append(dict(workload="x_quantize_s8_8192x8192", kernel="quantize_s8", launches=1, median_us=med * 1e3,
                         best_us=min(times) * 1e3, tflops=0.0, gbs=gbs, bound="hbm", frac=frac, library_us=None))
        print(f"| x_quantize_s8_8192x8192 | quantize_s8 | 1 | {med * 1e3:.1f} | 0.0 | {gbs:.0f} | hbm | {frac:.3f} |"
              + (" |" if args.library else ""), flush=True)
    if args.json:
        with open(args.json, "w") as f:
            json.dump(rows, f, indent=1)
    return 0


# --------------------------------------------------------------------------- our arm
def run_dry(args):
    """The multi-rank plumbing with the GEMM left out (no GPU needed): rendezvous, barrier, the MAX of
    the per-rank step times, the whole-job aggregate, one JSON line from rank 0.  The per-rank "step"
    is a sleep whose length grows with the rank, so the slowest rank must set the time."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    init_distributed(world, None)
    print(f"[bench] rank {rank} of {world} (dry run, no device)", file=sys.stderr, flush=True)
    w = workload(args.size)
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.002 * (rank + 1))
    ms = (time.perf_counter() - t0) * 1e3
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(ms, world, None)
    ms_per_step = ms / args.steps
    cfg = workload_config(w, world)
    out = {"metric": METRIC, "value": whole_job_tflops(w.flops, world, ms_per_step), "unit": UNIT, "n_gpus": world,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
           "dry_run": True, "gpu_launches": 0}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    import nk_inputs
    import paper_2511_13764_b200 as nk

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GEMM has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    init_distributed(world, dev)
    print(f"[bench] rank {rank} of {world} on cuda:{local} ({torch.cuda.get_device_name(local)})", file=sys.stderr,
          flush=True)

    peaks = load_peaks()
    w = workload(args.size)
    # rank r owns its own block of 8192 rows of A (seed shifted by the rank); B is replicated
    A = nk_inputs.fill(shard_seed(w.seed, rank), nk_inputs.TENSOR_A, w.M * w.K, w.dist_a[0], w.dist_a[1], w.in_dtype)
    B = nk_inputs.fill(w.seed, nk_inputs.TENSOR_B, w.K * w.N, w.dist_b[0], w.dist_b[1], w.in_dtype)
    hA = torch.from_numpy(A).pin_memory()
    hB = torch.from_numpy(B).pin_memory()
    dA = hA.to(dev, non_blocking=True)
    dB = hB.to(dev, non_blocking=True)
    dC = torch.empty(w.M * w.N, dtype=torch.float32, device=dev)
    plan = nk.plan_for(w, device=local)
    ws_bytes = plan.workspace_bytes
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def step():
        plan.run(dA, dB, dC, workspace=ws if ws_bytes else None, workspace_bytes=ws_bytes, stream=sp)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    plan.check()

    # best of 10 launches timed one by one after an L2 flush, on a chip that is not yet under sustained
    # load: the mode the pool's burst peak was taken in
    extras = rank == 0 and world == 1 and not args.no_modes and not args.no_cpu_baseline
    burst = None
    if extras:
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        singles = []
        for _ in range(10):
            flush.fill_(1)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            step()
            a1.record(stream)
            a1.synchronize()
            singles.append(a0.elapsed_time(a1))
        del flush
        burst = w.flops / (min(singles) * 1e-3) / 1e12
        torch.cuda.synchronize()
        time.sleep(0.5)

    sampler = ClockSampler(local)
    ev0 = torch.cuda.Event(enable_timing=True)
    ev1 = torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    while not ev1.query():
        sampler.sample()
        time.sleep(0.002)
    barrier()
    ms = ev0.elapsed_time(ev1)
    plan.check()
    ms = max_over_ranks(ms, world, dev)
    ms_per_step = ms / args.steps
    value = whole_job_tflops(w.flops, world, ms_per_step)

    # per-launch duration of the GEMM kernel: one launch per step, so the CUDA-event time of the
    # timed region divided by the steps is the kernel's average launch duration, measured live
    # on the launching stream (L2 cannot carry data across launches: A, B, C total 512 MB)
    traffic, traffic_note = recorded_traffic(plan.kernel_name, (w.M, w.N, w.K))
    k_avg = ms_per_step          # average launch duration inside the timed region
    achieved = w.flops / (k_avg * 1e-3) / 1e12
    peak = float(peaks["bf16_tflops"])
    roofline = {
        "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
        "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_note,
        "peak_source": f"MEASURED_PEAKS.json bf16_tflops (burst), of {peaks['_source']}",
        "frac_of_sustained_peak": achieved / float(peaks["bf16_tflops_sustained"]),
        "frac_of_nominal_2250": achieved / 2250.0,
        "kernel": plan.kernel_name,
        "hbm_algorithmic_gbs": w.algorithmic_bytes / (k_avg * 1e-3) / 1e9,
    }

    # The other mode the pool's peak figures were taken in: launches back to back for about four
    # seconds (compare with the sustained peak; the part is power-managed).
    if extras:
        per_round = max(10, int(0.25 / (ms_per_step * 1e-3)))
        sus_sampler = ClockSampler(local)
        t_begin = time.perf_counter()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launched = 0
        s0.record(stream)
        while time.perf_counter() - t_begin < 4.0:
            for _ in range(per_round):
                step()
            launched += per_round
            torch.cuda.synchronize()
            sus_sampler.sample()
        s1.record(stream)
        s1.synchronize()
        plan.check()
        sustained = launched * w.flops / (s0.elapsed_time(s1) * 1e-3) / 1e12
        roofline["burst_best_of_10"] = {"value": burst, "unit": UNIT, "frac_of_burst_peak": burst / peak}
        roofline["sustained_4s"] = {"value": sustained, "unit": UNIT, "launches": launched,
                                    "frac_of_sustained_peak": sustained / float(peaks["bf16_tflops_sustained"]),
                                    "clocks": sus_sampler.summary()}

    # end to end through the C ABI with HOST buffers: H2D of A and B, GEMM, D2H of C per step
    hC = torch.empty(w.M * w.N, dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(args.steps, 5))
    plan.run_host(hA, hB, hC, dA, dB, dC, workspace=ws if ws_bytes else None, workspace_bytes=ws_bytes, stream=sp)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        plan.run_host(hA, hB, hC, dA, dB, dC, workspace=ws if ws_bytes else None, workspace_bytes=ws_bytes,
                      stream=sp)
    barrier()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, world, dev)
    e2e = {"value": whole_job_tflops(w.flops, world, e2e_s * 1e3), "unit": UNIT,
           "h2d_bytes_per_step": int(A.nbytes + B.nbytes), "d2h_bytes_per_step": int(w.M * w.N * 4),
           "steps": e2e_steps}

    cfg = workload_config(w, world)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
        "roofline": roofline, "e2e": e2e,
        "gpu_launches": plan.launches_per_run * args.steps,
        "clocks": sampler.summary(),
    }

    # the other configurations, each timed on its own (outside the contract's timed region)
    if extras and not args.no_configs and args.size is None:
        del dA, dB, dC, hC
        torch.cuda.empty_cache()
        out["configs"] = time_configs(peaks, device=local)
        out["configs_timing"] = ("per launch, CUDA-graph replay of 20 (L2 flush, GEMM) pairs minus a graph of the "
                                 "flushes, median of 5; rows of 5e11 flop and more: CUDA events around single "
                                 "launches after a flush, median of 9")

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tf, sec, threads, nrows = oracle_sample_rate(w, B, min(1024, w.M), 1, 0)
        out["cpu_baseline"] = {
            "value": tf, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{nrows} stratified rows of the {w.M}x{w.N}x{w.K} problem (all columns, full K), "
                      f"{sec:.1f} s"}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="timed steps and the end-to-end leg only (profiler captures): no CPU oracle, no extra modes")
    ap.add_argument("--no-modes", action="store_true", help="skip the best-of-10 and four-second measurements")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration list")
    ap.add_argument("--size", type=int, default=None,
                    help="shrink M=N=K (profiler captures only; not a benchmark number)")
    ap.add_argument("--dry-run", action="store_true",
                    help="multi-rank plumbing only: no device, the step is a sleep (CPU tests)")
    ap.add_argument("--table", action="store_true", help="print the per-workload table instead of the JSON line")
    ap.add_argument("--iters", type=int, default=9, help="--table: timed launches per row")
    ap.add_argument("--only", default=None, help="--table: comma-separated substrings of workload names")
    ap.add_argument("--json", default=None, help="--table: also write the rows to this file")
    ap.add_argument("--no-flush", action="store_true", help="--table: leave L2 warm between launches")
    ap.add_argument("--flags", type=lambda x: int(x, 0), default=0, help="--table: NK_FLAG_* bits given to every plan")
    ap.add_argument("--graph", type=int, default=20,
                    help="--table: (flush, GEMM) pairs per CUDA-graph replay (0: CUDA events around single launches)")
    ap.add_argument("--library", action="store_true", help="--table: add a column with torch.matmul (cuBLAS)")
    ap.add_argument("--f32-tensor", action="store_true",
                    help="--table: after every FP32 row, the same workload with NK_FLAG_F32_TENSOR")
    args = ap.parse_args()
    if args.table:
        return run_table(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus, sys.argv[1:])
    if args.impl == "reference":
        return run_reference(args)
    if args.dry_run:
        return run_dry(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
