"""Times every benchmark configuration through the C ABI and prints a table.

    python -m paper_2511_13764_b200.perf_table [--iters 20] [--only c3] [--json out.json]

Each launch is timed on its own with CUDA events on the launching stream, after
warm-up, with L2 flushed in between (a 512 MB buffer is overwritten), so
operands come from HBM as they would in a real pipeline.  Per configuration the
table gives the median time, TFLOP/s, the algorithmic HBM GB/s, and the
fraction of the roofline that binds it: the measured BF16 tensor peak, the
measured HBM copy bandwidth, or the FP32 FMA-pipe peak (SMs x 128 x 2 x max SM
clock); with --f32-tensor every FP32 row is followed by the same workload
multiplied on the tensor cores (a sixth of the BF16 tensor peak: six BF16
products per FP32 product).  It only measures; parity is the tests' business.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["bf16_tflops"]), float(p["hbm_gbs"]), "measured"
    return 1590.0, 6650.0, "fallback"


def time_launch(launch, st, iters, flush, graph_pairs):
    """Median (and best) time in ms of `launch(cuda_stream)`, each call timed on its own after an
    L2 flush.  With `graph_pairs` a CUDA graph of that many (flush, launch) pairs is replayed and a
    graph of the flushes alone subtracted: CUDA-event stamps are a microsecond or two coarse on
    some boxes, the graph difference resolves a fraction of a microsecond, and the launches come
    without host gaps, as they would inside a captured pipeline."""
    import time
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


def time_workload(w, iters, flags=0, flush=None, graph_pairs=0, library=False):
    """Returns (median ms, best ms, kernel name, launches per run, library ms or None).  `library`
    also times torch.matmul (cuBLAS) on the same shape and element type (row-major operands, no
    epilogue, FP32 without TF32): context for the table, never part of the product path."""
    import torch
    import paper_2511_13764_b200 as nk
    dev = torch.device("cuda", 0)
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
    plan = nk.plan_for(w, flags=flags)
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


def main():
    import torch
    import nk_inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--only", default=None, help="substring of the workload name")
    ap.add_argument("--json", default=None)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--flags", type=lambda x: int(x, 0), default=0, help="NK_FLAG_* bits given to every plan")
    ap.add_argument("--graph", type=int, default=0,
                    help="time N (flush, GEMM) pairs per CUDA-graph replay against N flushes (finer than event stamps)")
    ap.add_argument("--library", action="store_true", help="add a column with torch.matmul (cuBLAS) on the same shape")
    ap.add_argument("--f32-tensor", action="store_true",
                    help="after every FP32 row, the same workload with NK_FLAG_F32_TENSOR (three BF16 planes, six "
                         "cross terms on the tensor cores); its roofline is a sixth of the BF16 tensor peak")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    tensor_peak, hbm_peak, src = peaks()
    prop = torch.cuda.get_device_properties(0)
    fma_peak = prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12
    flush = None if args.no_flush else torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    works = ([nk_inputs.config(i) for i in (1, 2, 3, 4)] + nk_inputs.sweep() + nk_inputs.paper_mlp() + nk_inputs.f16_set()
             + nk_inputs.s8_set() + nk_inputs.fp8_set() + nk_inputs.bt_set())
    rows = []
    print(f"| workload | kernel | launches | median us | TFLOP/s | alg. GB/s | bound | frac ({src}) |"
          + (" cuBLAS us |" if args.library else ""))
    print("|---|---|---|---|---|---|---|---|" + ("---|" if args.library else ""))
    import paper_2511_13764_b200 as nk
    todo = []
    for w in works:
        if args.only and args.only not in w.name:
            continue
        todo.append((w, w.name, args.flags, False))
        if args.f32_tensor and w.in_dtype == "f32" and w.N % 8 == 0 and w.K % 8 == 0:
            todo.append((w, w.name + " +tensor", args.flags | nk.FLAG_F32_TENSOR, True))
    for w, label, flags, split in todo:
        med, best, kname, launches, lib_ms = time_workload(w, args.iters, flags=flags, flush=flush,
                                                           graph_pairs=args.graph if w.flops < 5e11 else 0,
                                                           library=args.library and not split)
        tf = w.flops / (med * 1e-3) / 1e12
        gbs = w.algorithmic_bytes / (med * 1e-3) / 1e9
        # 8-bit operands run at twice the BF16 rate on the tensor cores (nominal ratio applied to the measured BF16 peak)
        compute_peak = (tensor_peak / 6 if split else 2 * tensor_peak if w.in_dtype in ("s8", "e4m3", "e5m2")
                        else tensor_peak if w.in_dtype != "f32" else fma_peak)
        t_compute = w.flops / (compute_peak * 1e12)
        t_hbm = w.algorithmic_bytes / (hbm_peak * 1e9)
        if t_hbm >= t_compute:
            bound, frac = "hbm", gbs / hbm_peak
        else:
            bound, frac = ("tensor/6" if split else "tensor" if w.in_dtype != "f32" else "alu"), tf / compute_peak
        rows.append(dict(workload=label, kernel=kname, launches=launches, median_us=med * 1e3,
                         best_us=best * 1e3, tflops=tf, gbs=gbs, bound=bound, frac=frac,
                         library_us=None if lib_ms is None else lib_ms * 1e3))
        print(f"| {label} | {kname} | {launches} | {med * 1e3:.1f} | {tf:.1f} | {gbs:.0f} | {bound} | {frac:.3f} |"
              + (f" {lib_ms * 1e3:.1f} |" if lib_ms is not None else " |" if args.library else ""), flush=True)
    if args.json:
        with open(args.json, "w") as f:
            json.dump(rows, f, indent=1)


if __name__ == "__main__":
    main()
