"""Build libfact.so in-tree with nvcc for sm_100a (no JIT cache, no pip install).

    python -m paper_2604_26666_b200.build [--force] [--verbose]

FACT_EXPERIMENTS=1 in the environment adds -DFACT_EXPERIMENTS: a library for timing experiments whose kernels
honour the work-skipping FACT_DEBUG_FLAGS bits (loads, products or stores left out; results are garbage).
The default build has no such code.
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libfact.so"
STAMP = PKG / "libfact.so.srchash"

SOURCES = ["fact_api.cu"]
HEADERS = ["gemm_kernel.cuh", "kcluster_kernel.cuh", "attention_kernel.cuh", "norm_kernel.cuh", "tune_kernels.cuh", "ptx.cuh"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "--shared", "-Xcompiler", "-fPIC",
    "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if os.path.exists(cand) else "nvcc"


def _flags() -> list:
    return NVCC_FLAGS + (["-DFACT_EXPERIMENTS"] if os.environ.get("FACT_EXPERIMENTS") == "1" else [])


def source_hash() -> str:
    h = hashlib.sha1()
    for f in [CSRC / s for s in SOURCES + HEADERS] + [ROOT / "include" / "fact.h"]:
        h.update(f.read_bytes())
    h.update(" ".join(_flags()).encode())
    return h.hexdigest()


def is_current() -> bool:
    return LIB.exists() and STAMP.exists() and STAMP.read_text().strip() == source_hash()


def build(force: bool = False, verbose: bool = False) -> Path:
    if is_current() and not force:
        return LIB
    cmd = [_nvcc(), *_flags(), "-I", str(ROOT / "include"), "-I", str(CSRC)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(CSRC / s) for s in SOURCES]
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd += ["-o", str(tmp)]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
    os.replace(tmp, LIB)
    STAMP.write_text(source_hash() + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
