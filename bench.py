#!/usr/bin/env python
"""Benchmark of libfact on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-shapes]

One "step" is one pass over the square-GEMM configuration (C = A.B at 4096^3
and 8192^3, BF16 in, FP32 accumulate, BF16 out, operands N(0,1)/sqrt(K),
seed 1).  The headline value is whole-job TFLOP/s (2 M N K per product,
epilogue work not counted) with inputs resident in HBM; `e2e` repeats it with
pinned-host inputs copied in and the result copied out inside the timed region.
`shapes` adds, for every shape of the five configurations, its own time,
TFLOP/s, GB/s and roofline fraction, next to a cuBLAS (torch.matmul) side
reference that is never on the product path.

With N > 1 (torchrun) every rank runs the same workload on its own GPU (the
path shards by rows / batch entries with no exchange step): weak scaling, value
= all ranks' FLOPs / max-over-ranks time.

`--impl reference` times the FP64 CPU oracle on the host cores on a bounded row
slab of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "TFLOP/s & % of dense BF16 tensor peak per fused-epilogue GEMM shape"
WORKLOAD = "config 2: square BF16 GEMM 4096^3 + 8192^3, N(0,1)/sqrt(K), seed 1"
L2_FLUSH_BYTES = 512 << 20

# DRAM traffic per launch of the dominant kernel (8192^3): dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture of that launch (954.7 MB + 125.9 MB, mean of five launches; another box: 845.0 + 128.3).
DOMINANT_TRAFFIC_BYTES = 1.0806e9


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        # "under load" = the samples drawing at least half of the largest power seen
        busy = [c for c, w in zip(sm, pw) if w >= 0.5 * max(pw)] if pw else sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_under_load": len(busy),
                "power_w_max": max(pw) if pw else None}


# ------------------------------------------------------------------------------------------ reference arm
def oracle_time_case(case, ins, target_seconds: float):
    """Time the oracle (as it stands) on a leading row slab of `case` sized for about `target_seconds`.
    Returns (tflops, rows, seconds, threads)."""
    import numpy as np

    import oracle
    from paper_2604_26666_b200 import workloads as wl

    xb, wb = wl.bits(ins.X), wl.bits(ins.W)
    bias = None if ins.bias is None else wl.bits(ins.bias)
    res = None if ins.residual is None else wl.bits(ins.residual)
    if case.batch > 1:
        xb, wb = xb[:1], wb[:1]
        res = None if res is None else res[:1]
    flops_per_row = 2.0 * case.n_weight_cols * case.K

    def run(rows):
        idx = np.arange(rows, dtype=np.int64)
        t0 = time.perf_counter()
        oracle.linear(xb, wb, layout=case.layout, epilogue=case.epilogue, bias=bias, residual=res, rows=idx)
        return time.perf_counter() - t0

    # two probes: the first call pays for thread start-up and cold caches and underestimates the rate
    probe_rows = min(case.M, 64)
    t_probe = run(probe_rows)
    rate = probe_rows * flops_per_row / max(t_probe, 1e-9)
    probe_rows = int(max(probe_rows, min(case.M, 1.5 * rate / flops_per_row)))
    t_probe = run(probe_rows)
    rate = probe_rows * flops_per_row / max(t_probe, 1e-9)
    rows = int(max(probe_rows, min(case.M, target_seconds * rate / flops_per_row)))
    rows = max(8, rows // 8 * 8) if case.M >= 8 else case.M
    t = run(rows)
    return rows * flops_per_row / t / 1e12, rows, t, oracle.max_threads()


def run_reference(args):
    """`--impl reference`: the CPU oracle on the host cores, bounded row slabs of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2604_26666_b200 import workloads as wl

    cases = [c for c in wl.benchmark_cases() if c.config == 2]
    per_step_budget = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    inputs = [wl.make_inputs(c) for c in cases]
    times, flops, samples, threads = [], [], [], 1
    for it in range(args.warmup + args.steps):
        t_step, f_step, desc = 0.0, 0.0, []
        for c, ins in zip(cases, inputs):
            tf, rows, secs, threads = oracle_time_case(c, ins, per_step_budget / len(cases))
            t_step += secs
            f_step += tf * 1e12 * secs
            desc.append(f"{c.name}: first {rows} of {c.M} rows")
        if it >= args.warmup:
            times.append(t_step)
            flops.append(f_step)
            samples = desc
    value = sum(flops) / sum(times) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "each step is a bounded leading-row slab of every GEMM"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": "; ".join(samples)},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ product arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="fact", choices=["fact", "reference"])
    ap.add_argument("--no-shapes", action="store_true", help="skip the per-shape table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tune", action="store_true", help="run the on-device tuner for every shape first")
    ap.add_argument("--shape", default=None,
                    help="time only this benchmark shape (a name from the `shapes` table, `all`, `attention`, `fp8`, `grouped`, `normfold`, `blocks` or `untuned`): "
                         "--warmup/--steps launches, no side reference; the small command used for profiling")
    ap.add_argument("--layout", default="NK", choices=["NK", "KN"], help="weight layout of the config 4/5 linears")
    ap.add_argument("--no-trains", action="store_true",
                    help="with --shape: skip the back-to-back launch trains of the short shapes (the profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    import torch

    from paper_2604_26666_b200 import workloads as wl
    from paper_2604_26666_b200.binding import Handle

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    from paper_2604_26666_b200 import dist_util

    rank, world, local_rank = dist_util.env_ranks()
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    dist = dist_util.init("nccl", dev)
    h = Handle(local_rank)
    if h.debug_flags() & ~(256 | 2048 | 4096 | 8192):  # only a -DFACT_EXPERIMENTS build honours the work-skipping switches
        raise SystemExit("bench.py refuses to run with work-skipping FACT_DEBUG_FLAGS bits set")
    peaks = load_peaks()
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def flush_l2():
        # Overwrite the L2 with a 512 MB fill, then read the buffer back: the read pass evicts the fill's dirty
        # lines, so the timed kernel starts on an L2 full of unrelated *clean* lines and is not charged the
        # write-back of 126 MB that are not its own (that write-back cost HBM-bound shapes 10-20 %).
        flush_buf.fill_(1)
        flush_buf.view(torch.int64).sum()

    # (the handle has already loaded the package's tuned table for the benchmark shapes)
    if args.shape is not None:
        names = None if args.shape == "all" else args.shape.split(",")
        if args.shape == "untuned" or args.shape.startswith("untuned:"):
            # `untuned:1024x1024x8192[,MxNxK...]` times only those shapes (the small command used for profiling)
            only = None
            if ":" in args.shape:
                only = [tuple(int(v) for v in t.split("x")) for t in args.shape.split(":", 1)[1].split(",")]
            print(json.dumps({"untuned": untuned_table(h, dev, stream, flush_l2, warm=args.warmup, iters=max(args.steps, 3),
                                                       shapes=only, tune=args.tune),
                              "gpu_launches": h.launch_count()}))
            h.close()
            return 0
        rows = [] if args.shape in ("attention", "blocks", "fp8", "grouped", "normfold") else per_shape_table(
            h, dev, stream, flush_l2, peaks, args.tune, names=names, warm=args.warmup, iters=args.steps,
            side_ref=False, layout=args.layout, trains=not args.no_trains)
        if args.shape in ("all", "attention"):
            att = attention_table(h, dev, stream, flush_l2, peaks, warm=args.warmup)
        elif args.shape in ("blocks", "fp8", "grouped", "normfold"):
            att = []
        else:  # attention shapes can be named like the GEMM shapes
            att = attention_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps, side_ref=False,
                                  names=names)
        blk = []
        if args.shape == "all":
            blk = block_table(h, dev, stream, flush_l2, peaks)
        elif args.shape == "blocks":  # --warmup / --steps apply, no eager side reference: the form the ncu runs use
            blk = block_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps, side_ref=False)
        f8 = []
        if args.shape in ("all", "fp8"):
            f8 = fp8_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps,
                           side_ref=args.shape == "all")
        elif names is not None and args.shape not in ("grouped", "normfold"):  # FP8 shapes can be named like the GEMM shapes
            f8 = fp8_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps, side_ref=False,
                           names=names)
        grp = []
        if args.shape in ("all", "grouped"):
            grp = grouped_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps,
                                side_ref=args.shape == "all")
        nfold = []
        if args.shape in ("all", "normfold"):
            nfold = norm_fold_table(h, dev, stream, flush_l2, peaks, warm=args.warmup, iters=args.steps)
        print(json.dumps({"shapes": rows, "attention": att, "blocks": blk, "fp8": f8, "grouped": grp,
                          "norm_fold": nfold, "gpu_launches": h.launch_count()}))
        h.close()
        return 0

    # ---------------------------------------------------------------- headline: config 2
    cases = [c for c in wl.benchmark_cases() if c.config == 2]
    host_inputs = [wl.make_inputs(c, pin=True) for c in cases]
    dev_inputs = [(i.X.to(dev), i.W.to(dev)) for i in host_inputs]
    outs = [torch.empty((c.M, c.N), dtype=torch.bfloat16, device=dev) for c in cases]
    step_flops = sum(c.flops for c in cases)
    dom = max(range(len(cases)), key=lambda i: cases[i].flops)

    if args.tune:
        for c, (X, W), o in zip(cases, dev_inputs, outs):
            h.tune("gemm", X, W, layout=c.layout, out=o)

    def step(events=None):
        for i, (c, (X, W), o) in enumerate(zip(cases, dev_inputs, outs)):
            if events is not None and i == dom:
                events[0].record(stream)
            h.gemm(X, W, layout=c.layout, out=o)
            if events is not None and i == dom:
                events[1].record(stream)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    launches0 = h.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for s in range(args.steps):
        flush_l2()  # untimed: between timed iterations the L2 is overwritten by a 512 MB fill and read-back
        ev[s][0].record(stream)
        step(events=(ev[s][2], ev[s][3]))
        ev[s][1].record(stream)
    barrier()
    launches = h.launch_count() - launches0
    step_ms = [e[0].elapsed_time(e[1]) for e in ev]
    dom_ms = [e[2].elapsed_time(e[3]) for e in ev]
    total_ms = dist_util.max_over_ranks(sum(step_ms), dist, dev)
    assert h.device_status() == 0, "a device-side wait timed out during the timed region"
    k_cycles, k_ns = h.last_kernel_clock()  # the dominant launch is the last one of a step
    value = world * step_flops * args.steps / (total_ms * 1e-3) / 1e12
    dom_case = cases[dom]
    dom_avg_ms = sum(dom_ms) / len(dom_ms)
    achieved = dom_case.flops / (dom_avg_ms * 1e-3) / 1e12

    # ---------------------------------------------------------------- end to end: host buffers in, host result out
    # Through the library's host-buffer entry point (fact_gemm_host over the C ABI): every step hands it pinned host
    # operands and a pinned host result; the call copies in, multiplies and copies out on the handle's three streams,
    # and the copies of neighbouring problems overlap the kernels (two device scratch buffers per shape, in turn).
    from paper_2604_26666_b200.pipeline import HostGemmPipeline

    host_outs = [torch.empty((c.M, c.N), dtype=torch.bfloat16).pin_memory() for c in cases]
    e2e_steps = max(3, min(args.steps, 10))
    pipe = HostGemmPipeline(h, [(c.M, c.N, c.K) for c in cases], layout=cases[0].layout)

    def e2e_step():
        for c, hi, ho in zip(cases, host_inputs, host_outs):
            pipe.submit(hi.X, hi.W, ho, stream=stream)

    e2e_step()
    pipe.finish(stream)
    barrier()
    t_wall0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    pipe.h2d_bytes = pipe.d2h_bytes = 0
    for _ in range(e2e_steps):
        e2e_step()
    h.gemm_host_wait(stream)  # the stream waits for every call's copy-out
    e1.record(stream)
    pipe.finish(stream)
    barrier()
    e2e_ms = dist_util.max_over_ranks(e0.elapsed_time(e1), dist, dev)
    e2e_wall_ms = (time.perf_counter() - t_wall0) * 1e3
    e2e_value = world * step_flops * e2e_steps / (e2e_ms * 1e-3) / 1e12
    h2d = pipe.h2d_bytes // e2e_steps
    d2h = pipe.d2h_bytes // e2e_steps
    # the results that came back over PCIe are the ones the device-resident run produced
    for o, ho in zip(outs, host_outs):
        assert torch.equal(o.cpu(), ho), "end-to-end result differs from the device-resident result"
    del host_outs

    # ---------------------------------------------------------------- every shape of the five configurations
    shapes = []
    # (single-GPU information: in a multi-rank run every rank but 0 would sit in the process group for minutes)
    tables = not args.no_shapes and rank == 0 and world == 1
    if tables:
        shapes = per_shape_table(h, dev, stream, flush_l2, peaks, args.tune)
    attention, blocks, fp8, grouped, norm_fold = [], [], [], [], []
    if tables:
        norm_fold = norm_fold_table(h, dev, stream, flush_l2, peaks)
        attention = attention_table(h, dev, stream, flush_l2, peaks)
        fp8 = fp8_table(h, dev, stream, flush_l2, peaks)
        grouped = grouped_table(h, dev, stream, flush_l2, peaks)
        blocks = block_table(h, dev, stream, flush_l2, peaks)
    clocks = sampler.stop()  # sampled from the first warm-up step to the end of the per-shape table

    # ---------------------------------------------------------------- CPU baseline (oracle) on rank 0
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tf, rows, secs, threads = oracle_time_case(dom_case, host_inputs[dom], 15.0)
        cpu = {"value": tf, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
               "sample": f"first {rows} of {dom_case.M} rows of the {dom_case.M}^3 GEMM, {secs:.1f} s "
                         f"(cost is linear in M)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "b_layout": "KN (row-major B)", "timing": "CUDA events per step",
                       "l2": "512 MB fill + read-back between timed steps (untimed: L2 left full of unrelated clean lines); step footprint 480 MB > L2",
                       "parallelism": f"dp{world} (independent replicas of the workload, no collective)"},
            "pct_of_peak": {"burst_measured": 100 * value / world / peaks["bf16_tflops"],
                            "sustained_measured": 100 * value / world / peaks["bf16_tflops_sustained"],
                            "nominal_2250": 100 * value / world / 2250.0, "peaks": peaks["source"]},
            "roofline": {"bound": "tensor", "kernel": f"fact_gemm_kernel on {dom_case.name}", "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                         "peak_source": peaks["source"] + " (burst)", "launch_ms": dom_avg_ms,
                         "traffic": DOMINANT_TRAFFIC_BYTES, "algorithmic_bytes": dom_case.algorithmic_bytes},
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps, "wall_ms_per_step": e2e_wall_ms / e2e_steps,
                    "api": "fact_gemm_host over the C ABI (pinned host in, pinned host out; copy-in, product and "
                           "copy-out on the handle's three streams, two device scratch buffers per shape)"},
            "gpu_launches": launches, "debug_flags": h.debug_flags(),
            "clocks": dict(clocks, sm_mhz_in_dominant_kernel=(1e3 * k_cycles / k_ns if k_ns else None)),
            "cpu_baseline": cpu,
            "shapes": shapes,
            "attention": attention,
            "fp8": fp8,
            "grouped": grouped,
            "norm_fold": norm_fold,
            "blocks": blocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    h.close()
    return 0


SHORT_SHAPE_US = 120.0  # shapes whose single cold launch is shorter than this are (also) timed back to back


def back_to_back_us(call_set, case, X, W, bias, res, out, h, dev, stream, reps=5, min_launches=20):
    """Microseconds per launch of `case`, from N >= 20 launches back to back between one event pair, rotating through
    R copies of the operands and outputs with R x footprint > 2 x L2 (so no launch finds its data in L2).  Median of
    `reps` such trains.  call_set "side": the cuBLAS matmul-only side reference on the same buffers."""
    import torch

    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    foot = max(1.0, case.algorithmic_bytes)
    R = int(min(512, max(2, -(-2 * l2 // int(foot)) + 1)))
    sets = []
    for _ in range(R):
        sets.append((X.clone(), W.clone(), None if bias is None else bias.clone(),
                     None if res is None else res.clone(), torch.empty_like(out)))
    n = R * max(1, -(-min_launches // R))

    def one(s):
        Xs, Ws, bs, rs, os_ = s
        if call_set == "side":
            if case.batch > 1:
                torch.bmm(Xs, Ws if case.layout == "KN" else Ws.transpose(1, 2))
            else:
                torch.matmul(Xs, Ws if case.layout == "KN" else Ws.t())
        elif case.op == "gemm":
            h.gemm(Xs, Ws, layout=case.layout, out=os_)
        elif case.op == "gemm_batched":
            h.gemm_batched(Xs, Ws, layout=case.layout, out=os_)
        elif case.op == "gemm_splitk":
            h.gemm_splitk(Xs, Ws, layout=case.layout, out=os_)
        else:
            h.linear(Xs, Ws, bias=bs, residual=rs, epilogue=case.epilogue, layout=case.layout, out=os_)

    for s in sets:  # warm-up: every set once (also sizes the workspace)
        one(s)
    torch.cuda.synchronize(dev)
    # The train is replayed from a CUDA graph: issued from Python, a launch costs the host more than these kernels
    # take, and the figure would be the interpreter's launch rate.
    graph = torch.cuda.CUDAGraph()
    side_stream = torch.cuda.Stream(dev)
    with torch.cuda.graph(graph, stream=side_stream):
        for i in range(n):
            one(sets[i % R])  # (inside the capture torch's current stream is the capturing stream)
    graph.replay()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        a.record(stream)
        graph.replay()
        b.record(stream)
        torch.cuda.synchronize(dev)
        ts.append(a.elapsed_time(b) / n)
    del graph
    del sets
    return sorted(ts)[len(ts) // 2] * 1e3


def per_shape_table(h, dev, stream, flush_l2, peaks, tune, names=None, warm=5, iters=20, side_ref=True, layout="NK",
                    trains=True):
    """Time every benchmark shape alone (5 warm-up + 20 timed launches, L2 overwritten between launches)."""
    import torch

    from paper_2604_26666_b200 import workloads as wl

    rows = []
    for case in wl.benchmark_cases(layout) + wl.paper_cases():
        if names is not None and case.name not in names:
            continue
        ins = wl.make_inputs(case)
        X, W = ins.X.to(dev), ins.W.to(dev)
        bias = None if ins.bias is None else ins.bias.to(dev)
        res = None if ins.residual is None else ins.residual.to(dev)
        odt = torch.float32 if case.out == "f32" else torch.bfloat16
        oshape = (case.batch, case.M, case.N) if case.batch > 1 else (case.M, case.N)
        out = torch.empty(oshape, dtype=odt, device=dev)

        def call():
            if case.op == "gemm":
                h.gemm(X, W, layout=case.layout, out=out)
            elif case.op == "gemm_batched":
                h.gemm_batched(X, W, layout=case.layout, out=out)
            elif case.op == "gemm_splitk":
                h.gemm_splitk(X, W, layout=case.layout, out=out)
            else:
                h.linear(X, W, bias=bias, residual=res, epilogue=case.epilogue, layout=case.layout, out=out)

        def side():
            # cuBLAS through torch: the bare product only, as a side reference
            if case.batch > 1:
                torch.bmm(X, W if case.layout == "KN" else W.transpose(1, 2))
            else:
                torch.matmul(X, W if case.layout == "KN" else W.t())

        def side_same_op():
            # the same fused operation composed from PyTorch's own operators (eager; cuBLASLt's bias epilogue where
            # F.linear uses it): what the fusion is worth, next to the bare product above
            import torch.nn.functional as F
            wt = W.t() if case.layout == "KN" else W  # [N, K]
            if case.epilogue == "SILU_GATE":
                y = F.linear(X, wt)
                n = y.shape[-1] // 2
                return F.silu(y[:, :n]) * y[:, n:]
            y = F.linear(X, wt, bias)
            if case.epilogue == "BIAS_RELU":
                return torch.relu(y)
            if case.epilogue == "BIAS_GELU_TANH":
                return F.gelu(y, approximate="tanh")
            if case.epilogue == "BIAS_RESIDUAL":
                return y + res
            return y

        if tune:
            h.tune(case.op, X, W, layout=case.layout, bias=bias, residual=res, epilogue=case.epilogue, out=out)

        def time_it(fn, warm=warm, iters=iters, cold=True):
            for _ in range(warm):
                fn()
            ts = []
            for _ in range(iters):
                if cold:
                    flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                ts.append((a, b))
            torch.cuda.synchronize(dev)
            return sorted(x.elapsed_time(y) for x, y in ts)

        def kernel_span_us(n=7):
            """The kernel's own clock: microseconds and SM MHz of the first CTA's span in a cold launch, median of n
            (fact_last_kernel_clock; no launch or completion latency in it)."""
            spans = []
            for _ in range(n):
                flush_l2()
                call()
                cyc, ns = h.last_kernel_clock()
                spans.append((ns * 1e-3, 1e3 * cyc / ns if ns else 0.0))
            spans.sort()
            return spans[len(spans) // 2]

        t = time_it(call)
        t_hot = time_it(call, cold=False) if side_ref else t
        t_side = time_it(side, iters=10) if side_ref else [0.0]
        med = t[len(t) // 2]
        t_tensor = case.flops / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm = case.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        bound = "tensor" if t_tensor >= t_hbm else "hbm"
        cfg = h.get_config(case.op, case.batch, case.M, case.N, case.K, case.epilogue, case.layout, odt).as_dict()
        row = {
            "name": case.name, "config": case.config, "op": case.op, "epilogue": case.epilogue,
            "layout": case.layout, "batch": case.batch, "M": case.M, "N": case.N, "K": case.K, "out": case.out,
            "us_median": med * 1e3, "us_min": t[0] * 1e3, "us_hot_l2_median": t_hot[len(t_hot) // 2] * 1e3,
            "bound": bound, "roofline_us": max(t_tensor, t_hbm) * 1e3,
            "cublas_matmul_only_us": t_side[len(t_side) // 2] * 1e3, "tile": cfg,
        }
        if side_ref and case.op == "linear" and case.epilogue != "NONE":
            t_same = time_it(side_same_op, iters=10)
            row["torch_eager_same_op_us"] = t_same[len(t_same) // 2] * 1e3
        # Shapes of the order of 100 us and below: an event pair around ONE launch that follows the L2-flush kernels
        # also times the launch itself (10-12 us on this part), so the figure that counts for them is N launches back
        # to back between one event pair, rotating through R sets of operands and outputs whose total exceeds twice
        # the L2 -- every launch still finds its data in DRAM, and the cost per launch is the stream time it adds.
        # Which time the roofline fraction uses: an HBM-bound shape (and the latency-bound 512^3) the train -- every
        # launch cold, write-back of the previous output included, no launch latency -- against the measured copy
        # bandwidth; a tensor-bound shape the single cold launch against the burst peak (a kernel timed alone), with
        # the train against the sustained peak (a kernel timed inside a long run) reported beside it.
        t_use, used_train = med, False
        if med * 1e3 < SHORT_SHAPE_US:
            # (short launches only: there the event pair's fixed 7-10 us are a large part of the figure)
            span_us, span_mhz = kernel_span_us()
            row.update({"us_kernel_span_first_cta": span_us, "sm_mhz_in_kernel": span_mhz,
                        "roofline_frac_of_kernel_span": max(t_tensor, t_hbm) * 1e3 / span_us if span_us else None})
        if med * 1e3 < SHORT_SHAPE_US and trains:
            t_b2b = back_to_back_us(call_set=None, case=case, X=X, W=W, bias=bias, res=res, out=out, h=h, dev=dev,
                                    stream=stream) * 1e-3
            row["us_back_to_back_cold"] = t_b2b * 1e3
            if side_ref:
                row["cublas_matmul_only_back_to_back_us"] = back_to_back_us(
                    call_set="side", case=case, X=X, W=W, bias=bias, res=res, out=out, h=h, dev=dev, stream=stream)
            t_tensor_sustained = case.flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
            row["roofline_frac_train"] = (t_hbm if bound == "hbm" else t_tensor_sustained) / t_b2b
            row["roofline_train_peak"] = "measured copy bandwidth" if bound == "hbm" else "measured sustained BF16 peak"
            if bound == "hbm":
                t_use, used_train = t_b2b, True
        row["timing"] = ("back-to-back launches over rotating buffer sets (total > 2 x L2), per launch"
                         if used_train else "one launch per event pair after an L2 flush, median")
        row.update({
            "us": t_use * 1e3, "tflops": case.flops / (t_use * 1e-3) / 1e12,
            "gbs": case.algorithmic_bytes / (t_use * 1e-3) / 1e9,
            "pct_of_bf16_peak_burst": 100 * case.flops / (t_use * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "roofline_frac": max(t_tensor, t_hbm) / t_use,
            "roofline_frac_single_launch": max(t_tensor, t_hbm) / med,
        })
        rows.append(row)
        del X, W, out
    return rows


UNTUNED_SHAPES = [(1024, 1024, 1024), (2048, 2048, 2048), (2048, 8192, 1024), (8192, 1024, 4096), (16, 4096, 4096),
                  (64, 8192, 8192), (128, 14336, 4096), (256, 4096, 14336), (1000, 1000, 1000), (4096, 128, 4096),
                  (8192, 64, 8192), (1536, 1536, 6144), (512, 512, 8192), (512, 2048, 16384), (1024, 1024, 8192),
                  (256, 256, 32768), (128, 4096, 8192), (2048, 512, 4096), (768, 768, 3072), (32, 14336, 4096),
                  (4096, 4096, 512), (8192, 8192, 128)]


def untuned_table(h, dev, stream, flush_l2, warm=3, iters=9, shapes=None, tune=False):
    """Shapes the tuner's table does not know (`--shape untuned`): the library's own choice of configuration (its cost
    model: data-parallel tiles, K slices through a workspace, or K slices as a cluster), the same call held to one
    slice, and `torch.matmul`; single launches after an L2 flush, mean of the middle of `iters` runs."""
    import torch

    def time_it(fn):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(iters):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize(dev)
            ts.append(a.elapsed_time(b) * 1e3)
        ts.sort()
        mid = ts[len(ts) // 4: len(ts) - len(ts) // 4]
        return sum(mid) / len(mid)

    rows = []
    g = torch.Generator(device="cpu").manual_seed(77)
    for (M, N, K) in (shapes or UNTUNED_SHAPES):
        X = torch.randn(M, K, generator=g).to(torch.bfloat16).to(dev)
        W = (torch.randn(N, K, generator=g) * K ** -0.5).to(torch.bfloat16).to(dev)
        out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        cfg = h.get_config("gemm", 1, M, N, K, "NONE", "NK", torch.bfloat16).as_dict()
        rows.append({
            "M": M, "N": N, "K": K, "config": cfg,
            "us": time_it(lambda: h.gemm(X, W, layout="NK", out=out)),
            "us_one_slice": time_it(lambda: h.gemm(X, W, layout="NK", out=out, cfg={"split_k": 1})),
            "torch_matmul_us": time_it(lambda: torch.matmul(X, W.t(), out=out)),
        })
        if tune:  # (--tune: what the on-device tuner finds for the shape, timed the same way)
            best, _, n_tried = h.tune("gemm", X, W, layout="NK", out=out, cold_l2=True)
            rows[-1].update({"tuned_config": best.as_dict(), "tuned_candidates": n_tried,
                             "us_tuned": time_it(lambda: h.gemm(X, W, layout="NK", out=out))})
        del X, W, out
    return rows


def attention_table(h, dev, stream, flush_l2, peaks, warm=5, iters=20, side_ref=True, names=None):
    """Time the fused attention kernel on the transformer blocks' attention shapes (L2 overwritten between
    launches); torch's scaled_dot_product_attention on the same tensors is a side reference."""
    import torch

    from paper_2604_26666_b200 import workloads as wl

    rows = []
    for case in wl.attention_cases():
        if names is not None and case.name not in names:
            continue
        q, k, v = wl.make_attention_inputs(case, dev)
        out = torch.empty_like(q)

        def call():
            h.attention(q, k, v, causal=case.causal, out=out)

        qt, kt, vt = (x.permute(0, 2, 1, 3) for x in (q, k, v))

        def side():
            torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=case.causal,
                                                             enable_gqa=case.Hq != case.Hkv)

        def time_it(fn, n):
            for _ in range(warm):
                fn()
            ts = []
            for _ in range(n):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                ts.append((a, b))
            torch.cuda.synchronize(dev)
            return sorted(x.elapsed_time(y) for x, y in ts)

        t = time_it(call, iters)
        med = t[len(t) // 2]
        try:
            ts = time_it(side, 10) if side_ref else [0.0]
        except Exception:  # the side reference is optional
            ts = [float("nan")]
        t_tensor = case.flops / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm = case.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        rows.append({
            "name": case.name, "B": case.B, "T": case.T, "heads_q": case.Hq, "heads_kv": case.Hkv,
            "head_dim": case.D, "causal": case.causal, "us_median": med * 1e3, "us_min": t[0] * 1e3,
            "tflops": case.flops / (med * 1e-3) / 1e12, "bound": "tensor" if t_tensor >= t_hbm else "hbm",
            "roofline_us": max(t_tensor, t_hbm) * 1e3, "roofline_frac": max(t_tensor, t_hbm) / med,
            "torch_sdpa_us": ts[len(ts) // 2] * 1e3,
        })
        assert h.device_status() == 0
        del q, k, v, out
    return rows


def fp8_table(h, dev, stream, flush_l2, peaks, warm=5, iters=20, side_ref=True, names=None):
    """Time fact_linear_fp8 (FP8 E4M3 operands, BF16 output) on the FP8 shapes, L2 overwritten between launches;
    torch._scaled_mm (cuBLASLt, matmul only) on the same operands is a side reference.  The peak is the measured
    BF16 burst peak times the nominal FP8 : BF16 ratio of 2 (there is no measured FP8 figure)."""
    import torch

    from paper_2604_26666_b200 import workloads as wl

    rows = []
    peak = 2.0 * peaks["bf16_tflops"]
    for case in wl.fp8_cases():
        if names is not None and case.name not in names:
            continue
        ins = wl.make_fp8_inputs(case)
        X, W = ins.X.to(dev), ins.W.to(dev)
        bias = None if ins.bias is None else ins.bias.to(dev)
        out = torch.empty((case.M, case.N), dtype=torch.bfloat16, device=dev)

        def call():
            h.linear_fp8(X, W, ins.scale, bias, epilogue=case.epilogue, out=out)

        def time_it(fn, n):
            for _ in range(warm):
                fn()
            ts = []
            for _ in range(n):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                ts.append((a, b))
            torch.cuda.synchronize(dev)
            return sorted(x.elapsed_time(y) for x, y in ts)

        t = time_it(call, iters)
        med = t[len(t) // 2]
        ts = [0.0]
        if side_ref:
            try:
                xs, wt = X.view(torch.float8_e4m3fn), W.view(torch.float8_e4m3fn).t()
                one = torch.tensor(1.0, device=dev)
                ts = time_it(lambda: torch._scaled_mm(xs, wt, scale_a=one, scale_b=one, out_dtype=torch.bfloat16), 10)
            except Exception:  # the side reference is optional
                ts = [float("nan")]
        t_tensor = case.flops / (peak * 1e12) * 1e3
        t_hbm = case.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        c = h.get_config("linear_fp8", 1, case.M, case.N, case.K, case.epilogue, "NK", torch.bfloat16).as_dict()
        rows.append({
            "name": case.name, "M": case.M, "N": case.N, "K": case.K, "epilogue": case.epilogue, "dtype": "f8e4m3",
            "us_median": med * 1e3, "us_min": t[0] * 1e3, "tflops": case.flops / (med * 1e-3) / 1e12,
            "gbs": case.algorithmic_bytes / (med * 1e-3) / 1e9,
            "bound": "tensor" if t_tensor >= t_hbm else "hbm", "peak_tflops": peak,
            "peak_source": "2 x measured BF16 burst (nominal FP8 : BF16 ratio)",
            "roofline_us": max(t_tensor, t_hbm) * 1e3, "roofline_frac": max(t_tensor, t_hbm) / med,
            "cublaslt_scaled_mm_only_us": ts[len(ts) // 2] * 1e3, "tile": c,
        })
        assert h.device_status() == 0
        del X, W, out
    return rows


def grouped_table(h, dev, stream, flush_l2, peaks, warm=3, iters=10, side_ref=True, names=None):
    """Time fact_linear_grouped on mixture-of-experts-shaped problems (uneven, seeded group sizes), L2 overwritten
    between launches; a loop of torch.matmul calls, one per group (cuBLAS, matmul only), is a side reference."""
    import torch

    from paper_2604_26666_b200 import workloads as wl

    rows_out = []
    for case in wl.grouped_cases():
        if names is not None and case.name not in names:
            continue
        rows = wl.grouped_rows(case)
        X, W = wl.make_grouped_inputs(case, dev)
        out = torch.empty((case.tokens, case.N), dtype=torch.bfloat16, device=dev)
        offs = [0]
        for r in rows:
            offs.append(offs[-1] + r)

        bias = None
        if case.epilogue.startswith("BIAS"):
            gb = torch.Generator(device=dev).manual_seed(case.seed + 2)
            bias = (torch.randn((case.N,), generator=gb, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)

        def call():
            h.linear_grouped(X, W, rows, bias=bias, epilogue=case.epilogue, out=out)

        def side():
            for g in range(case.groups):
                torch.matmul(X[offs[g]:offs[g + 1]], W[g].t())

        def time_it(fn, n):
            for _ in range(warm):
                fn()
            ts = []
            for _ in range(n):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                ts.append((a, b))
            torch.cuda.synchronize(dev)
            return sorted(x.elapsed_time(y) for x, y in ts)

        t = time_it(call, iters)
        med = t[len(t) // 2]
        try:
            ts = time_it(side, 5) if side_ref else [0.0]
        except Exception:  # the side reference is optional
            ts = [float("nan")]
        t_tensor = case.flops / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm = case.algorithmic_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        rows_out.append({
            "name": case.name, "tokens": case.tokens, "groups": case.groups, "N": case.N, "K": case.K,
            "epilogue": case.epilogue, "rows_min": min(rows), "rows_max": max(rows),
            "us_median": med * 1e3, "us_min": t[0] * 1e3, "tflops": case.flops / (med * 1e-3) / 1e12,
            "gbs": case.algorithmic_bytes / (med * 1e-3) / 1e9, "bound": "tensor" if t_tensor >= t_hbm else "hbm",
            "roofline_us": max(t_tensor, t_hbm) * 1e3, "roofline_frac": max(t_tensor, t_hbm) / med,
            "torch_matmul_loop_only_us": ts[len(ts) // 2] * 1e3,
        })
        assert h.device_status() == 0
        del X, W, out
    return rows_out


def norm_fold_table(h, dev, stream, flush_l2, peaks, warm=3, iters=10):
    """Output projection (+ residual) -> row normalisation -> first MLP layer, two ways: three launches (linear,
    fact_norm, linear) and two (the producer leaves row sums, the consumer corrects its accumulator; the weights are
    folded once, outside the timed region).  Chain times with L2 overwritten before each chain, and the SM cycles of
    each product with and without the extras."""
    import torch

    from paper_2604_26666_b200 import workloads as wl

    rows = []
    for case in wl.norm_chain_cases():
        t = wl.make_norm_chain_inputs(case, dev)
        T, H, F = case.tokens, case.hidden, case.ffn
        x1 = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
        n = torch.empty_like(x1)
        y = torch.empty((T, F), dtype=torch.bfloat16, device=dev)
        stats = torch.empty((H // 64, T, 2), dtype=torch.float32, device=dev)
        wf, cs, bf = h.fold_norm(t["w1"], t["gamma"], t.get("beta"), t.get("b1"))
        colsum = None if case.gated else cs

        def producer(with_sums):
            h.linear(t["a"], t["wo"], bias=t.get("bo"), residual=t["x0"], epilogue="BIAS_RESIDUAL", out=x1,
                     stats_out=stats if with_sums else None)

        def consumer(folded):
            if folded:
                h.linear(x1, wf, bias=bf, epilogue=case.epilogue, out=y, x_norm=case.kind, x_stats=stats,
                         w_colsum=colsum)
            else:
                h.linear(n, t["w1"], bias=t.get("b1"), epilogue=case.epilogue, out=y)

        def unfused():
            producer(False)
            h.norm(x1, t["gamma"], t.get("beta"), kind=case.kind, out=n)
            consumer(False)

        def fused():
            producer(True)
            consumer(True)

        def time_both(f0, f1):  # alternating, so that both see the same clocks
            for _ in range(warm):
                f0()
                f1()
            ts = ([], [])
            for _ in range(iters):
                for k, fn in enumerate((f0, f1)):
                    flush_l2()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    fn()
                    b.record(stream)
                    ts[k].append((a, b))
            torch.cuda.synchronize(dev)
            return tuple(sorted(x.elapsed_time(z) for x, z in t) for t in ts)

        def cycles(fn):
            out = []
            for _ in range(5):
                flush_l2()
                fn()
                torch.cuda.synchronize(dev)
                out.append(h.last_kernel_clock()[0])
            return sorted(out)[2]

        tu, tf = time_both(unfused, fused)
        unfused()  # leaves n and stats-free x1 for the per-product cycle counts
        rows.append({
            "name": case.name, "tokens": T, "hidden": H, "ffn": F, "norm": case.kind, "epilogue": case.epilogue,
            "us_three_launches": tu[len(tu) // 2] * 1e3, "us_two_launches": tf[len(tf) // 2] * 1e3,
            "tflops_two_launches": case.flops / (tf[len(tf) // 2] * 1e-3) / 1e12,
            "producer_cycles": cycles(lambda: producer(False)), "producer_cycles_with_sums": cycles(lambda: producer(True)),
            "consumer_cycles": cycles(lambda: consumer(False)), "consumer_cycles_folded": cycles(lambda: consumer(True)),
        })
        assert h.device_status() == 0
        del t, x1, n, y, wf
    return rows


def block_table(h, dev, stream, flush_l2, peaks, warm=3, iters=10, side_ref=True):
    """Time one forward pass of the paper's two transformer blocks through fact_block_forward (seven launches on one
    stream; also replayed from a CUDA graph) next to the same block in PyTorch eager BF16 on this GPU."""
    import torch
    import torch.nn.functional as F

    from paper_2604_26666_b200 import workloads as wl

    def time_it(fn, n):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(n):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            ts.append((a, b))
        torch.cuda.synchronize(dev)
        t = sorted(x.elapsed_time(y) for x, y in ts)
        return t[len(t) // 2]

    rows = []
    for case in wl.block_cases():
        x, w = wl.make_block_inputs(case, dev)
        desc = h.block_desc(case.kind, case.B, case.T, case.Hq, case.Hkv, case.D, case.ffn, w)
        y = torch.empty_like(x)
        h.block_forward(desc, x, out=y)  # allocates the workspace, configures the kernels
        launches0 = h.launch_count()
        h.block_forward(desc, x, out=y)
        launches = h.launch_count() - launches0
        ms = time_it(lambda: h.block_forward(desc, x, out=y), iters)
        ms_graph = None
        try:
            graph = torch.cuda.CUDAGraph()
            torch.cuda.synchronize(dev)
            with torch.cuda.graph(graph, stream=torch.cuda.Stream(dev)):  # capture needs a side stream
                h.block_forward(desc, x, out=y)
            ms_graph = time_it(graph.replay, iters)
        except Exception as e:  # the graph replay is an extra, the stream launch is the number
            print(f"# graph capture of {case.name} failed: {e}", file=sys.stderr)
        C, Hq, Hkv, D = case.hidden, case.Hq, case.Hkv, case.D

        def eager():
            norm = (lambda v, g, b: F.layer_norm(v, (C,), g, b, 1e-5)) if case.kind == "gpt" else \
                   (lambda v, g, b: F.rms_norm(v, (C,), g, 1e-5))
            n1 = norm(x, w["norm1_gamma"], w.get("norm1_beta"))
            qkv = F.linear(n1, w["wqkv"], w.get("bqkv")).view(case.B, case.T, Hq + 2 * Hkv, D)
            q, k, v = (t.transpose(1, 2) for t in (qkv[:, :, :Hq], qkv[:, :, Hq:Hq + Hkv], qkv[:, :, Hq + Hkv:]))
            a = F.scaled_dot_product_attention(q, k, v, is_causal=True, enable_gqa=Hq != Hkv)
            x1 = F.linear(a.transpose(1, 2).reshape(case.B * case.T, C), w["wo"], w.get("bo")) + x
            n2 = norm(x1, w["norm2_gamma"], w.get("norm2_beta"))
            if case.kind == "gpt":
                hh = F.gelu(F.linear(n2, w["w1"], w["b1"]), approximate="tanh")
            else:
                gu = F.linear(n2, w["w1"])
                hh = F.silu(gu[:, :case.ffn]) * gu[:, case.ffn:]
            return F.linear(hh, w["w2"], w.get("b2")) + x1

        ms_eager = None
        if side_ref:
            try:
                ms_eager = time_it(eager, iters)
            except Exception as e:
                print(f"# eager reference of {case.name} failed: {e}", file=sys.stderr)
        assert h.device_status() == 0
        # the block's normalisation kernel alone: HBM-bound, one read and one write of the activation
        nout = torch.empty_like(x)
        kind = "layer" if case.kind == "gpt" else "rms"
        ms_norm = time_it(lambda: h.norm(x, w["norm1_gamma"], w.get("norm1_beta"), kind=kind, out=nout), iters)
        norm_bytes = 2 * x.numel() * 2
        del nout
        rows.append({
            "norm_us": ms_norm * 1e3, "norm_gbs": norm_bytes / (ms_norm * 1e-3) / 1e9,
            "norm_frac_of_hbm_peak": norm_bytes / (ms_norm * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "name": case.name, "kind": case.kind, "batch": case.B, "seq": case.T, "hidden": C, "heads_q": Hq,
            "heads_kv": Hkv, "head_dim": D, "ffn": case.ffn, "ms": ms, "ms_cuda_graph": ms_graph,
            "tflops": case.flops / (ms * 1e-3) / 1e12, "launches": launches, "torch_eager_bf16_ms": ms_eager,
            "speedup_vs_torch_eager": (ms_eager / ms) if ms_eager else None,
        })
        del x, w, y, desc
        torch.cuda.empty_cache()
    return rows


if __name__ == "__main__":
    sys.exit(main())
