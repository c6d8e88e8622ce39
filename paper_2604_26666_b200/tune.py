"""Run the on-device tile-configuration tuner over the benchmark shapes and
write the table that `Handle` loads by default.

    python -m paper_2604_26666_b200.tune --set all               (writes the whole table the package ships)
    python -m paper_2604_26666_b200.tune [--out PATH] [--layout NK|KN|both] [--shapes a,b,...] [--warm] [--log PATH]
    python -m paper_2604_26666_b200.tune --set paper --merge     (the paper's own shapes, added to the table)
    python -m paper_2604_26666_b200.tune --set fp8 --merge       (the FP8 shapes)

The counterpart of the paper's verify and auto-tuning actions (Section 4.2, Actions 4 and 5): every
feasible candidate is first checked on the device against the default configuration's output, then
timed (5 warm-up + 20 timed launches, the protocol of Section 5.1) with the L2 overwritten before
each launch (the numbers the benchmark reports are cold-L2 numbers; --warm times back to back
instead), and the fastest verified candidate is kept per problem key.  --log writes one JSON line per
candidate: its configuration, what happened to it (timed / infeasible / no_workspace / launch_failed /
verify_failed), its time and its distance from the reference output.
"""
from __future__ import annotations

import argparse
import json
import sys
from pathlib import Path

import torch

from . import workloads as wl
from .binding import Handle

DEFAULT_TABLE = Path(__file__).resolve().parent / "tuned_b200.txt"


def tune_case(h: Handle, case: wl.Case, dev: str = "cuda:0", cold: bool = True):
    ins = wl.make_inputs(case)
    X, W = ins.X.to(dev), ins.W.to(dev)
    bias = None if ins.bias is None else ins.bias.to(dev)
    res = None if ins.residual is None else ins.residual.to(dev)
    odt = torch.float32 if case.out == "f32" else torch.bfloat16
    return h.tune(case.op, X, W, layout=case.layout, bias=bias, residual=res, epilogue=case.epilogue, out_dtype=odt,
                  cold_l2=cold, records=True)


def tune_fp8_case(h: Handle, case: wl.Fp8Case, dev: str = "cuda:0", cold: bool = True):
    ins = wl.make_fp8_inputs(case)
    bias = None if ins.bias is None else ins.bias.to(dev)
    return h.tune("linear_fp8", ins.X.to(dev), ins.W.to(dev), layout="NK", bias=bias, epilogue=case.epilogue,
                  cold_l2=cold, records=True)


def report(name, layout, flops, cfg, ms, n, recs, log):
    counts = {}
    for r in recs:
        counts[r["outcome"]] = counts.get(r["outcome"], 0) + 1
    rest = ", ".join(f"{v} {k}" for k, v in sorted(counts.items()) if k != "timed")
    print(f"{name:32s} {layout} best {ms * 1e3:9.1f} us  {flops / ms / 1e9:8.1f} TFLOP/s  of {n:3d} timed"
          f"{' (' + rest + ')' if rest else ''}: {cfg}", flush=True)
    if log is not None:
        for r in recs:
            log.write(json.dumps(dict(r, shape=name, layout=layout)) + "\n")


def paper_set():
    """The paper's own Level-1 shapes and the four linears of each of its two blocks at the paper's token counts."""
    cases = list(wl.paper_cases())
    for b in wl.block_cases():
        tok, C, qc = b.B * b.T, b.hidden, (b.Hq + 2 * b.Hkv) * b.D
        bias = b.kind == "gpt"
        cases += [
            wl.Case(f"{b.name}_qkv", "linear", tok, qc, C, epilogue="BIAS" if bias else "NONE", layout="NK",
                    has_bias=bias, seed=b.seed, w_scale=0.02),
            wl.Case(f"{b.name}_out", "linear", tok, C, C, epilogue="BIAS_RESIDUAL", layout="NK", has_bias=bias,
                    has_residual=True, seed=b.seed, w_scale=0.02),
            wl.Case(f"{b.name}_up", "linear", tok, b.ffn, C, epilogue="BIAS_GELU_TANH" if bias else "SILU_GATE",
                    layout="NK", has_bias=bias, seed=b.seed, w_scale=0.02),
            wl.Case(f"{b.name}_down", "linear", tok, C, b.ffn, epilogue="BIAS_RESIDUAL", layout="NK", has_bias=bias,
                    has_residual=True, seed=b.seed, w_scale=0.02),
        ]
    return cases


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=str(DEFAULT_TABLE))
    ap.add_argument("--layout", default="both", choices=["NK", "KN", "both"])
    ap.add_argument("--shapes", default=None)
    ap.add_argument("--set", default="benchmark", choices=["benchmark", "paper", "fp8", "all"])
    ap.add_argument("--merge", action="store_true", help="start from the table already in --out")
    ap.add_argument("--warm", action="store_true", help="time launches back to back (warm L2) instead of cold")
    ap.add_argument("--log", default=None, help="write one JSON line per candidate to this file")
    args = ap.parse_args(argv)
    h = Handle(0, load_table=False)
    if args.merge and Path(args.out).exists():
        h.tune_cache_load(args.out)
    names = None if args.shapes is None else set(args.shapes.split(","))
    cold = not args.warm
    log = open(args.log, "w") if args.log else None
    sets = ["benchmark", "paper", "fp8"] if args.set == "all" else [args.set]
    seen = set()
    for which in sets:
        if which == "fp8":
            for case in wl.fp8_cases():
                if names is not None and case.name not in names:
                    continue
                cfg, ms, n, recs = tune_fp8_case(h, case, cold=cold)
                report(case.name, "NK", case.flops, cfg, ms, n, recs, log)
            continue
        layouts = ["NK", "KN"] if (args.layout == "both" and which == "benchmark") else \
                  [args.layout if args.layout != "both" else "NK"]
        for layout in layouts:
            for case in (wl.benchmark_cases(layout) if which == "benchmark" else paper_set()):
                key = (case.name, case.layout)
                if key in seen or (names is not None and case.name not in names):
                    continue
                seen.add(key)
                cfg, ms, n, recs = tune_case(h, case, cold=cold)
                report(case.name, case.layout, case.flops, cfg, ms, n, recs, log)
    if log is not None:
        log.close()
    h.tune_cache_save(args.out)
    print("wrote", args.out)
    h.close()


if __name__ == "__main__":
    sys.exit(main())
