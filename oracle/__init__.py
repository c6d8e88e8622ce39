"""FP64 CPU oracle for the fused-epilogue GEMM family -- TEST INFRASTRUCTURE.

Only the tests, ``__graft_entry__.smoke()`` and the CPU-baseline / reference
legs of ``bench.py`` may import this package.  It does not import the CUDA
package and the CUDA package does not import it.

The arithmetic lives in ``fact_oracle.c`` (plain C, FP64, OpenMP over
independent output blocks).  This module only compiles that file with gcc,
loads it with ctypes and marshals numpy arrays.

What it computes (Section 5.1 "Benchmark problems" and the pattern-p2 GEMMs of
Section 5.2): ``Y = epilogue(X @ W)`` on BF16 bit patterns, with every product
and sum in double and one ascending-k sum per output element.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "fact_oracle.c"

EPILOGUES = {
    "NONE": 0,
    "BIAS": 1,
    "BIAS_RELU": 2,
    "BIAS_GELU_TANH": 3,
    "SILU_GATE": 4,
    "BIAS_RESIDUAL": 5,
}
LAYOUTS = {"KN": 0, "NK": 1}

_lib = None


def _cpu_tag() -> str:
    """A short tag of this host's instruction-set flags: a library built with
    ``-march=native`` on one host must not be loaded on a different CPU."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1((flags + _SRC.read_text()).encode()).hexdigest()[:12]


def lib_path() -> Path:
    return _HERE / f"libfact_oracle_{_cpu_tag()}.so"


def build(force: bool = False) -> Path:
    """Compile the C oracle for this host (gcc, OpenMP).  Building the checker
    is not using it."""
    out = lib_path()
    if out.exists() and not force:
        return out
    tmp = out.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
           "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, out)
    return out


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    i64, p, i32 = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
    lib.fact_oracle_linear.restype = i32
    lib.fact_oracle_linear.argtypes = [
        i64, i64, i64, i64,  # batch M N_out K
        p, i64, i64,  # X ldx strideX
        p, i64, i64, i32,  # W ldw strideW layout
        p,  # bias
        p, i64, i64,  # R ldr strideR
        i32,  # epi
        p, i64,  # rows n_rows
        p, i64, i64,  # Y ldy strideY
        i32, i32,  # variant nthreads
    ]
    lib.fact_oracle_round_bf16.restype = ctypes.c_uint16
    lib.fact_oracle_round_bf16.argtypes = [ctypes.c_double]
    lib.fact_oracle_bf16_to_f64.restype = ctypes.c_double
    lib.fact_oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
    lib.fact_oracle_gelu_tanh.restype = ctypes.c_double
    lib.fact_oracle_gelu_tanh.argtypes = [ctypes.c_double]
    lib.fact_oracle_silu.restype = ctypes.c_double
    lib.fact_oracle_silu.argtypes = [ctypes.c_double]
    lib.fact_oracle_max_threads.restype = i32
    _lib = lib
    return lib


def max_threads() -> int:
    return int(_load().fact_oracle_max_threads())


def _bits(a, name):
    a = np.asarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"{name}: expected BF16 bit patterns as uint16, got {a.dtype}")
    if a.shape[-1] > 1 and a.strides[-1] != 2:
        raise ValueError(f"{name}: innermost dimension must be contiguous")
    if min(a.shape) <= 1:
        a = np.ascontiguousarray(a)  # size-0/1 dimensions carry arbitrary strides
    return a


def linear(X, W, *, layout="KN", epilogue="NONE", bias=None, residual=None, rows=None,
           variant="blocked", nthreads=0):
    """``Y = epilogue(X @ W)`` in FP64.

    X : uint16 BF16 bits, [M, K] or [batch, M, K] (row stride may exceed K).
    W : uint16 BF16 bits; layout "KN": [K, Nw] (or [batch, K, Nw]);
        layout "NK": [Nw, K] (nn.Linear weight).  Nw = 2*N_out for SILU_GATE
        (gate columns first, then up columns), else N_out.
    bias : uint16 [N_out] or None;  residual : uint16 [M, N_out] (or batched) or None.
    rows : optional 1-D int64 row indices; only those output rows are computed.
    variant : "naive" (triple loop) or "blocked" (interchanged loops, same sums).
    Returns float64 [rows or M, N_out] (with a leading batch dim if X has one).
    """
    lib = _load()
    X = _bits(X, "X")
    W = _bits(W, "W")
    batched = X.ndim == 3
    if batched != (W.ndim == 3):
        raise ValueError("X and W must both be batched or both not")
    if not batched:
        X3, W3 = X[None], W[None]
    else:
        X3, W3 = X, W
    batch, M, K = X3.shape
    lay = LAYOUTS[layout]
    if lay == 0:
        if W3.shape[1] != K:
            raise ValueError("W (KN) first dim must equal K")
        Nw = W3.shape[2]
    else:
        if W3.shape[2] != K:
            raise ValueError("W (NK) second dim must equal K")
        Nw = W3.shape[1]
    epi = EPILOGUES[epilogue]
    if epi == EPILOGUES["SILU_GATE"]:
        if Nw % 2:
            raise ValueError("SILU_GATE needs an even number of weight columns")
        N_out = Nw // 2
    else:
        N_out = Nw
    if W3.shape[0] != batch:
        raise ValueError("batch mismatch")
    ldx = X3.strides[1] // 2
    sX = X3.strides[0] // 2 if batch > 1 else 0
    ldw = W3.strides[1] // 2
    sW = W3.strides[0] // 2 if batch > 1 else 0
    bias_p = None
    if bias is not None:
        bias = np.ascontiguousarray(_bits(bias, "bias"))
        if bias.shape != (N_out,):
            raise ValueError("bias must have N_out entries")
        bias_p = bias.ctypes.data
    R_p, ldr, sR = None, 0, 0
    if residual is not None:
        residual = _bits(residual, "residual")
        R3 = residual if batched else residual[None]
        if R3.shape != (batch, M, N_out):
            raise ValueError("residual must be [M, N_out]")
        ldr = R3.strides[1] // 2
        sR = R3.strides[0] // 2 if batch > 1 else 0
        R_p = R3.ctypes.data
    rows_p, n_rows = None, 0
    if rows is not None:
        rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
        rows_p, n_rows = rows.ctypes.data, rows.shape[0]
    n_out_rows = n_rows if rows is not None else M
    Y = np.empty((batch, n_out_rows, N_out), dtype=np.float64)
    rc = lib.fact_oracle_linear(
        batch, M, N_out, K,
        X3.ctypes.data, ldx, sX,
        W3.ctypes.data, ldw, sW, lay,
        bias_p,
        R_p, ldr, sR,
        epi,
        rows_p, n_rows,
        Y.ctypes.data, N_out, n_out_rows * N_out,
        {"naive": 0, "blocked": 1}[variant], int(nthreads),
    )
    if rc != 0:
        raise ValueError(f"fact_oracle_linear rejected its arguments (code {rc})")
    return Y if batched else Y[0]


def linear_softmax(X, W, *, layout="NK", bias=None, rows=None):
    """The "GEMM-Softmax" fusion of the paper's Table 1, written out as its definition: ``Z = X @ W (+ bias)`` in
    FP64 by ``linear``, then the softmax of every row, ``Y[m, n] = exp(Z[m, n] - max_j Z[m, j]) / sum_j exp(Z[m, j] -
    max_j Z[m, j])`` (subtracting the row maximum changes nothing mathematically and keeps the exponentials finite)."""
    Z = linear(X, W, layout=layout, epilogue="NONE" if bias is None else "BIAS", bias=bias, rows=rows)
    Z = Z - Z.max(axis=-1, keepdims=True)
    E = np.exp(Z)
    return E / E.sum(axis=-1, keepdims=True)


def linear_grouped(X, W, group_rows, *, layout="NK", epilogue="NONE", bias=None, residual=None):
    """Grouped linear layer (the "Grouped GEMM" of the paper's Table 1), written out as its definition: the rows of X
    are cut into consecutive groups of ``group_rows[g]`` rows and group g is multiplied by ``W[g]``:
    ``Y[rows of g] = epilogue(X[rows of g] @ W[g])``, one call of ``linear`` per group.
    X : uint16 [M, K];  W : uint16 [G, Nw, K] ("NK") or [G, K, Nw] ("KN");  bias [N_out] shared by the groups;
    residual [M, N_out].  Returns float64 [M, N_out]."""
    X = _bits(X, "X")
    W = _bits(W, "W")
    rows = [int(r) for r in group_rows]
    if W.ndim != 3 or W.shape[0] != len(rows) or sum(rows) != X.shape[0] or min(rows, default=0) < 0:
        raise ValueError("group_rows must give one non-negative row count per weight matrix and sum to the rows of X")
    Nw = W.shape[2] if layout == "KN" else W.shape[1]
    N_out = Nw // 2 if epilogue == "SILU_GATE" else Nw
    Y = np.empty((X.shape[0], N_out), dtype=np.float64)
    r0 = 0
    for g, n in enumerate(rows):
        if n:
            res = None if residual is None else np.ascontiguousarray(residual[r0:r0 + n])
            Y[r0:r0 + n] = linear(np.ascontiguousarray(X[r0:r0 + n]), np.ascontiguousarray(W[g]), layout=layout,
                                  epilogue=epilogue, bias=bias, residual=res)
        r0 += n
    return Y


def round_bf16(x: float) -> int:
    """Nearest-even BF16 bit pattern of a double (one rounding)."""
    return int(_load().fact_oracle_round_bf16(float(x)))


def bf16_to_f64(bits) -> np.ndarray:
    """Exact widening of BF16 bit patterns to float64 (numpy, no C call)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def gelu_tanh(z: float) -> float:
    return float(_load().fact_oracle_gelu_tanh(float(z)))


def silu(g: float) -> float:
    return float(_load().fact_oracle_silu(float(g)))
