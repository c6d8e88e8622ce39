"""Shared helpers for the GPU parity tests: run a problem through the C-ABI
binding and through the FP64 oracle on the same BF16 bits, and gate the
difference."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl

ACTIVATIONS = ("BIAS_GELU_TANH", "SILU_GATE")


def gates(ref: np.ndarray, got: np.ndarray, out: str, epilogue: str):
    """Returns (worst err/contract-gate, worst err/tight-gate).
    Contract gate: BF16 outputs |err| <= 1e-2 + 1e-2 |ref|; FP32 outputs
    |err| <= 2e-3 max(|ref|, rms(ref)) (a pure relative bound is undefined at
    outputs that happen to fall next to zero).
    Tight gate (BF16): |err| <= 1.5 * 2^-8 |ref| + c rms(ref), c = 2^-9, or 2^-8
    behind an approximated activation: BF16 rounding plus FP32 accumulation noise.
    Tight gate (FP32): |err| <= 1e-5 * sum-scale, approximated by 2e-5 max(|ref|, rms)."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if ref.size == 0:
        return 0.0, 0.0
    rms = float(np.sqrt(np.mean(ref * ref)))
    act = epilogue in ACTIVATIONS
    r2 = ref.reshape(-1, ref.shape[-1])
    g2 = got.reshape(-1, got.shape[-1])
    worst_c = worst_t = 0.0
    step = max(1, (1 << 22) // max(1, r2.shape[1]))  # a few million elements at a time: whole 8192 x 14336 outputs
    for i in range(0, r2.shape[0], step):
        r, g = r2[i:i + step], g2[i:i + step]
        err = np.abs(g - r)
        if out == "bf16":
            contract = err / (1e-2 + 1e-2 * np.abs(r))
            c = 2.0 ** -8 if act else 2.0 ** -9
            tight = err / (1.5 * 2.0 ** -8 * np.abs(r) + c * rms + 1e-30)
        else:
            contract = err / (2e-3 * np.maximum(np.abs(r), rms) + 1e-30)
            tight = err / (2e-5 * np.maximum(np.abs(r), rms) + 1e-30)
        # (a NaN anywhere must fail the gate, not vanish in max())
        worst_c = max(worst_c, float(np.nan_to_num(contract, nan=np.inf).max()))
        worst_t = max(worst_t, float(np.nan_to_num(tight, nan=np.inf).max()))
    return worst_c, worst_t


def to_f64(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return oracle.bf16_to_f64(wl.bits(t.contiguous()))
    return t.double().numpy()


def oracle_for(ins: wl.Inputs, case: wl.Case, rows=None, variant="blocked"):
    return oracle.linear(
        wl.bits(ins.X), wl.bits(ins.W), layout=case.layout, epilogue=case.epilogue,
        bias=None if ins.bias is None else wl.bits(ins.bias),
        residual=None if ins.residual is None else wl.bits(ins.residual),
        rows=rows, variant=variant)


def run_gpu(h, ins: wl.Inputs, case: wl.Case, cfg=None, splits=0, out=None, dev="cuda:0"):
    X = ins.X.to(dev)
    W = ins.W.to(dev)
    bias = None if ins.bias is None else ins.bias.to(dev)
    res = None if ins.residual is None else ins.residual.to(dev)
    odt = torch.float32 if case.out == "f32" else torch.bfloat16
    if case.op == "gemm":
        return h.gemm(X, W, layout=case.layout, out=out, out_dtype=odt, cfg=cfg)
    if case.op == "gemm_batched":
        return h.gemm_batched(X, W, layout=case.layout, out=out, out_dtype=odt, cfg=cfg)
    if case.op == "gemm_splitk":
        return h.gemm_splitk(X, W, layout=case.layout, out=out, out_dtype=odt, splits=splits, cfg=cfg)
    return h.linear(X, W, bias=bias, residual=res, epilogue=case.epilogue, layout=case.layout, out=out,
                    out_dtype=odt, cfg=cfg)


def check_case(h, case: wl.Case, cfg=None, splits=0, rows=None, contract_max=1.0, tight_max=1.0, ins=None):
    """Run on the GPU and in the oracle; assert both gates; return the two ratios."""
    if ins is None:
        ins = wl.make_inputs(case)
    got = run_gpu(h, ins, case, cfg=cfg, splits=splits)
    torch.cuda.synchronize()
    assert h.device_status() == 0, "a device-side wait timed out"
    g = to_f64(got)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        g = g[..., rows, :]
    ref = oracle_for(ins, case, rows=rows)
    assert g.shape == ref.shape, (g.shape, ref.shape)
    assert np.isfinite(g).all(), "non-finite output"
    c, t = gates(ref, g, case.out, case.epilogue)
    assert c <= contract_max, f"{case.name}: contract gate ratio {c:.3f}"
    assert t <= tight_max, f"{case.name}: tight gate ratio {t:.3f}"
    return c, t


def small_int_inputs(case: wl.Case, seed: int, lo=-3, hi=3) -> wl.Inputs:
    """Integer-valued BF16 inputs: every product and partial sum is exact in FP32."""
    g = torch.Generator().manual_seed(seed)
    b = (case.batch,) if case.batch > 1 else ()

    def draw(shape):
        return torch.randint(lo, hi + 1, shape, generator=g).to(torch.float32).to(torch.bfloat16)

    X = draw(b + (case.M, case.K))
    W = draw(b + ((case.K, case.n_weight_cols) if case.layout == "KN" else (case.n_weight_cols, case.K)))
    bias = draw((case.N,)) if case.has_bias else None
    res = draw(b + (case.M, case.N)) if case.has_residual else None
    return wl.Inputs(X, W, bias, res)


def stratified_rows(M: int, n: int, seed: int = 0, tile: int = 128) -> np.ndarray:
    """Row sample that touches the first/last rows, every position class inside a tile
    and a spread of tiles."""
    rng = np.random.default_rng(seed)
    rows = {0, M - 1, min(M - 1, tile - 1), min(M - 1, tile), max(0, M - tile), M // 2}
    while len(rows) < min(n, M):
        rows.add(int(rng.integers(0, M)))
    return np.array(sorted(rows), dtype=np.int64)
