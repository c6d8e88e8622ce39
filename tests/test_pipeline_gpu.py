"""The host-buffer front end: pinned host operands in, pinned host results out, copies overlapped."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, to_f64

pytestmark = pytest.mark.gpu


def test_host_pipeline_matches_the_oracle_and_reuses_buffers_safely():
    from paper_2604_26666_b200.binding import Handle
    from paper_2604_26666_b200.pipeline import HostGemmPipeline

    h = Handle(0)
    shapes = [(300, 264, 520), (128, 512, 256)]
    pipe = HostGemmPipeline(h, shapes, layout="KN")
    problems = []
    # more problems than buffer sets, alternating shapes, distinct data each time
    for i in range(7):
        M, N, K = shapes[i % 2]
        case = wl.Case(f"p{i}", "gemm", M, N, K, layout="KN", seed=100 + i, w_scale=0.1)
        ins = wl.make_inputs(case, pin=True)
        out = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        problems.append((case, ins, out))
        pipe.submit(ins.X, ins.W, out)
    pipe.finish()
    assert h.device_status() == 0
    for case, ins, out in problems:
        ref = oracle.linear(wl.bits(ins.X), wl.bits(ins.W), layout="KN")
        c, t = gates(ref, to_f64(out), "bf16", "NONE")
        assert c <= 1.0 and t <= 1.0, (case.name, c, t)
    assert pipe.h2d_bytes == sum((c.M * c.K + c.K * c.N) * 2 for c, _, _ in problems)
    assert pipe.d2h_bytes == sum(c.M * c.N * 2 for c, _, _ in problems)
    h.close()


def test_gemm_host_entry_point_layouts_strides_and_errors():
    """fact_gemm_host through the binding: host operands with row strides, the [N x K] weight layout, an FP32 result,
    a K that is not a whole number of 16-byte pieces (the device copy is padded), pageable memory, argument errors."""
    import ctypes

    from paper_2604_26666_b200.binding import FactError, Handle, lib

    h = Handle(0)
    g = torch.Generator().manual_seed(9)
    M, N, K = 200, 136, 100  # K * 2 bytes is not a multiple of 16
    Abig = torch.randn(M, K + 12, generator=g).to(torch.bfloat16).pin_memory()
    Wbig = (torch.randn(N, K + 4, generator=g) * 0.1).to(torch.bfloat16)  # pageable on purpose
    A, W = Abig[:, :K], Wbig[:, :K]
    Cbig = torch.zeros(M, N + 8, dtype=torch.float32).pin_memory()
    C = Cbig[:, :N]
    scratch = torch.empty(h.gemm_host_scratch_bytes(M, N, K, torch.float32, "NK"), dtype=torch.uint8, device="cuda:0")
    for _ in range(3):  # the same scratch again and again: each call waits for the copy-out of the one before
        h.gemm_host(A, W, C, scratch, layout="NK")
    h.gemm_host_wait()
    torch.cuda.current_stream(0).synchronize()
    assert h.device_status() == 0
    ref = oracle.linear(wl.bits(Abig)[:, :K], wl.bits(Wbig)[:, :K], layout="NK")
    c, t = gates(ref, C.double().numpy(), "f32", "NONE")
    assert c <= 1.0 and t <= 1.0, (c, t)
    assert (Cbig[:, N:] == 0).all(), "wrote outside the N columns of the host result"
    # argument errors come back as status codes before anything is enqueued
    with pytest.raises(ValueError):
        h.gemm_host(A, W, C, scratch[:128], layout="NK")
    vp = ctypes.c_void_p
    rc = lib().fact_gemm_host(h._h, M, N, K, vp(A.data_ptr()), K + 12, vp(W.data_ptr()), K + 4, 1, vp(C.data_ptr()),
                              N + 8, 1, None, vp(scratch.data_ptr()), 64, None)
    assert rc == 5  # FACT_ERR_WORKSPACE_TOO_SMALL
    rc = lib().fact_gemm_host(h._h, M, N, K, None, K, vp(W.data_ptr()), K + 4, 1, vp(C.data_ptr()), N + 8, 1, None,
                              vp(scratch.data_ptr()), scratch.numel(), None)
    assert rc == 1  # FACT_ERR_INVALID_ARG
    assert lib().fact_gemm_host(h._h, 0, N, K, None, K, None, K, 1, None, N, 1, None, None, 0, None) == 0  # empty
    h.close()
