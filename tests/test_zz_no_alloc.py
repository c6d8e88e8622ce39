"""fact_gemm_splitk_static: the split-K GEMM for callers that cannot allocate device memory.

Some integrations run where cudaMalloc is not allowed (memory owned by an arena, allocator locks
forbidden on the hot path).  They get one entry point that takes no handle and no workspace: its
scratch is a fixed array inside the library image.  This test drives it through the C ABI, several
times in a row with different problems (a later call must not be disturbed by what an earlier one
left in the shared scratch), and checks each result twice: against the FP64 oracle under the FP32
tolerance of the other split-K tests, and bit for bit against the ordinary fact_gemm_splitk path,
which runs the same kernels with the same slices in the same order.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, oracle_for, to_f64

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed, layout):
    return wl.Case(f"static_{M}x{N}x{K}", "gemm_splitk", M, N, K, layout=layout, out="f32", seed=seed,
                   x_dist="uniform", w_dist="uniform")


# (M, N, K, splits, layout, seed): two calls in a row with different sizes, layouts and slice counts, then the
# library's own choice of slices (0) and a K that is not a whole number of 64-element blocks
SEQUENCE = [(256, 384, 16384, 12, "KN", 31), (136, 200, 4096 + 64, 5, "NK", 32), (256, 256, 8192, 0, "KN", 33),
            (200, 136, 4096 + 72, 3, "NK", 34)]


def test_static_scratch_splitk_matches_the_oracle_and_the_workspace_path():
    from paper_2604_26666_b200.binding import Handle, gemm_splitk_static_status, lib

    L = lib()
    h = Handle(0)
    dev = "cuda:0"
    stream = torch.cuda.current_stream(0)
    for (M, N, K, splits, layout, seed) in SEQUENCE:
        case = _case(M, N, K, seed, layout)
        ins = wl.make_inputs(case)
        A, B = ins.X.to(dev), ins.W.to(dev)
        want = h.gemm_splitk(A, B, layout=layout, splits=splits)
        got = torch.full((M, N), float("nan"), dtype=torch.float32, device=dev)  # caller-owned output
        rc = L.fact_gemm_splitk_static(
            0, M, N, K, ctypes.c_void_p(A.data_ptr()), A.stride(0), ctypes.c_void_p(B.data_ptr()), B.stride(0),
            0 if layout == "KN" else 1, ctypes.c_void_p(got.data_ptr()), got.stride(0), 1, splits,
            ctypes.c_void_p(stream.cuda_stream))
        assert rc == 0, rc
        assert gemm_splitk_static_status(0) == 0, "a device-side wait of the static call gave up"
        assert h.device_status() == 0
        assert torch.isfinite(got).all()
        # the oracle, under the FP32 tolerance
        ref = oracle_for(ins, case)
        c, t = gates(ref, to_f64(got), "f32", "NONE")
        assert c <= 1.0 and t <= 1.0, (case.name, c, t)
        # same kernels, same slices, same order of additions: the two paths agree bit for bit
        assert torch.equal(got, want), f"{case.name}: static and workspace paths differ"
    h.close()


def test_static_scratch_refuses_what_does_not_fit():
    from paper_2604_26666_b200.binding import lib

    L = lib()
    dev = "cuda:0"
    # 64 slices of a 1024 x 1024 FP32 plane = 256 MiB of partials: far beyond the 16 MiB scratch
    M = N = 1024
    K = 64 * 64
    A = torch.zeros(M, K, dtype=torch.bfloat16, device=dev)
    B = torch.zeros(K, N, dtype=torch.bfloat16, device=dev)
    C = torch.full((M, N), 7.0, dtype=torch.float32, device=dev)
    rc = L.fact_gemm_splitk_static(0, M, N, K, ctypes.c_void_p(A.data_ptr()), K, ctypes.c_void_p(B.data_ptr()), N, 0,
                                   ctypes.c_void_p(C.data_ptr()), N, 1, 64, None)
    assert rc == 5  # FACT_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert (C == 7.0).all(), "a refused call must not touch the output"
    assert L.fact_gemm_splitk_static(99, M, N, K, None, K, None, N, 0, None, N, 1, 1, None) != 0


def test_static_binding_rejects_mismatched_tensors_before_any_launch():
    from paper_2604_26666_b200.binding import gemm_splitk_static

    dev = "cuda:0"
    A = torch.zeros(64, 128, dtype=torch.bfloat16, device=dev)
    B = torch.zeros(128, 96, dtype=torch.bfloat16, device=dev)
    with pytest.raises(ValueError):  # inner dimensions differ
        gemm_splitk_static(A, torch.zeros(120, 96, dtype=torch.bfloat16, device=dev),
                           torch.zeros(64, 96, dtype=torch.float32, device=dev))
    with pytest.raises(ValueError):  # an output that is too small would be written past its end
        gemm_splitk_static(A, B, torch.zeros(32, 96, dtype=torch.float32, device=dev))
    out = gemm_splitk_static(A, B, torch.full((64, 96), 3.0, dtype=torch.float32, device=dev))
    torch.cuda.synchronize()
    assert (out == 0).all()
