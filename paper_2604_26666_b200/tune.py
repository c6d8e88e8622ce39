"""Run the on-device tile-configuration tuner over the benchmark shapes and
write the table that `Handle` loads by default.

    python -m paper_2604_26666_b200.tune [--out PATH] [--layout NK|KN|both] [--shapes a,b,...]
    python -m paper_2604_26666_b200.tune --set paper --merge     (the paper's own shapes, added to the table)
    python -m paper_2604_26666_b200.tune --set fp8 --merge       (the FP8 shapes)

The counterpart of the paper's auto-tuning action (Section 4.2, Action 5): every
feasible candidate is timed on the device (5 warm-up + 20 timed launches, the
protocol of Section 5.1) and the fastest is kept per problem key.
"""
from __future__ import annotations

import argparse
import sys
from pathlib import Path

import torch

from . import workloads as wl
from .binding import Handle

DEFAULT_TABLE = Path(__file__).resolve().parent / "tuned_b200.txt"


def tune_case(h: Handle, case: wl.Case, dev: str = "cuda:0"):
    ins = wl.make_inputs(case)
    X, W = ins.X.to(dev), ins.W.to(dev)
    bias = None if ins.bias is None else ins.bias.to(dev)
    res = None if ins.residual is None else ins.residual.to(dev)
    odt = torch.float32 if case.out == "f32" else torch.bfloat16
    return h.tune(case.op, X, W, layout=case.layout, bias=bias, residual=res, epilogue=case.epilogue, out_dtype=odt)


def tune_fp8_case(h: Handle, case: wl.Fp8Case, dev: str = "cuda:0"):
    ins = wl.make_fp8_inputs(case)
    bias = None if ins.bias is None else ins.bias.to(dev)
    return h.tune("linear_fp8", ins.X.to(dev), ins.W.to(dev), layout="NK", bias=bias, epilogue=case.epilogue)


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
    ap.add_argument("--set", default="benchmark", choices=["benchmark", "paper", "fp8"])
    ap.add_argument("--merge", action="store_true", help="start from the table already in --out")
    args = ap.parse_args(argv)
    h = Handle(0, load_table=False)
    if args.merge and Path(args.out).exists():
        h.tune_cache_load(args.out)
    names = None if args.shapes is None else set(args.shapes.split(","))
    seen = set()
    layouts = ["NK", "KN"] if (args.layout == "both" and args.set == "benchmark") else [args.layout if args.layout != "both" else "NK"]
    if args.set == "fp8":
        for case in wl.fp8_cases():
            if names is not None and case.name not in names:
                continue
            cfg, ms, n = tune_fp8_case(h, case)
            print(f"{case.name:32s} NK best {ms * 1e3:9.1f} us  {case.flops / ms / 1e9:8.1f} TFLOP/s  "
                  f"of {n:3d} candidates: {cfg}", flush=True)
        layouts = []
    for layout in layouts:
        for case in (wl.benchmark_cases(layout) if args.set == "benchmark" else paper_set()):
            key = (case.name, case.layout)
            if key in seen or (names is not None and case.name not in names):
                continue
            seen.add(key)
            cfg, ms, n = tune_case(h, case)
            print(f"{case.name:32s} {case.layout} best {ms * 1e3:9.1f} us  {case.flops / ms / 1e9:8.1f} TFLOP/s  "
                  f"of {n:3d} candidates: {cfg}", flush=True)
    h.tune_cache_save(args.out)
    print("wrote", args.out)
    h.close()


if __name__ == "__main__":
    sys.exit(main())
