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
