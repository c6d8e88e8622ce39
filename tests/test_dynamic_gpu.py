"""Dynamic tile scheduling (cfg.schedule = 2): the grid has one cluster per tile and the clusters that run obtain
further tiles by cancelling the launch of clusters that have not started (Section 4.2, Action 2: the grid-level
scheduling policy is a design choice of its own).  Which CTA group computes a tile must never change a value."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl
from paper_2604_26666_b200.binding import FactError
from tests.helpers import check_case, gates, oracle_for, run_gpu, small_int_inputs, to_f64

pytestmark = pytest.mark.gpu

ALL_EPI = ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"]


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0, load_table=False)
    yield hd
    hd.close()


def mk(name, M, N, K, op="linear", epilogue="NONE", layout="NK", out="bf16", seed=11, **kw):
    has_bias = epilogue in ("BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "BIAS_RESIDUAL")
    return wl.Case(name, op, M, N, K, epilogue=epilogue, layout=layout, out=out, has_bias=has_bias,
                   has_residual=epilogue == "BIAS_RESIDUAL", seed=seed, **kw)


# several waves of small tiles on 148 SMs: 12 x 18 tiles of 128 x 64, or 6 x 18 pairs of 256 x 64
M, N, K = 1500, 1100 + 52, 264


@pytest.mark.parametrize("cg", [1, 2])
@pytest.mark.parametrize("epi", ALL_EPI)
def test_every_epilogue_through_the_dynamic_scheduler(h, epi, cg):
    case = mk(f"dyn_{epi}_{cg}", M, N, K, epilogue=epi, layout="NK" if cg == 1 else "KN")
    tile_n = 128 if epi == "SILU_GATE" else 64
    cfg = {"tile_m": 128 * cg, "tile_n": tile_n * (2 if (cg == 2 and case.layout == "KN") else 1), "cta_group": cg,
           "schedule": 2}
    check_case(h, case, cfg=cfg)


@pytest.mark.parametrize("out", ["bf16", "f32"])
def test_dynamic_schedule_is_exact_on_integers_and_repeatable(h, out):
    case = mk(f"dyn_int_{out}", 2100, 640, 520, epilogue="BIAS_RESIDUAL", out=out)
    ins = small_int_inputs(case, seed=5)
    cfg = {"tile_m": 256, "tile_n": 64, "cta_group": 2, "schedule": 2}
    got = run_gpu(h, ins, case, cfg=cfg)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    ref = oracle_for(ins, case)
    if out == "f32":
        assert np.array_equal(got.cpu().double().numpy(), ref)
    else:
        want = np.vectorize(oracle.round_bf16, otypes=[np.uint16])(ref)
        assert np.array_equal(wl.bits(got.cpu().contiguous()), want)
    # which group gets which tile differs from launch to launch; no value may
    real = wl.make_inputs(case)
    first = run_gpu(h, real, case, cfg=cfg)
    for _ in range(4):
        assert torch.equal(first, run_gpu(h, real, case, cfg=cfg))
    # and the static schedule of the same tiles, walking K upwards in every tile like the dynamic one, gives the same
    # bits: a tile's sum does not depend on who computes it
    static = run_gpu(h, real, case, cfg=dict(cfg, schedule=1))
    torch.cuda.synchronize()
    c, t = gates(to_f64(static), to_f64(first), out, "NONE")
    assert c <= 1 and t <= 1


def test_dynamic_schedule_large_and_direct_store_paths(h):
    # 256-wide pair tiles, long enough K for the ring to wrap; then an output the staged path cannot store
    check_case(h, mk("dyn_wide", 2560 + 40, 2048, 1024 + 64, epilogue="BIAS_GELU_TANH"),
               cfg={"tile_m": 256, "tile_n": 256, "cta_group": 2, "schedule": 2})
    check_case(h, mk("dyn_direct", 1500, 1101, 136, epilogue="BIAS_RELU"),
               cfg={"tile_m": 128, "tile_n": 64, "cta_group": 1, "schedule": 2})


def test_dynamic_schedule_grouped(h):
    g = torch.Generator().manual_seed(3)
    rows = [700, 0, 1333, 129, 2200, 64]
    Mtot, Kg, Ng, G = sum(rows), 256 + 8, 512, len(rows)
    X = torch.randn(Mtot, Kg, generator=g).to(torch.bfloat16)
    W = (torch.randn(G, Ng, Kg, generator=g) * 0.05).to(torch.bfloat16)
    b = torch.randn(Ng, generator=g).to(torch.bfloat16)
    ref = oracle.linear_grouped(wl.bits(X), wl.bits(W), rows, layout="NK", epilogue="BIAS_RELU", bias=wl.bits(b))
    outs = []
    for sched in (1, 2):
        y = h.linear_grouped(X.cuda(), W.cuda(), rows, bias=b.cuda(), epilogue="BIAS_RELU",
                             cfg={"tile_m": 128, "tile_n": 64, "cta_group": 1, "schedule": sched})
        torch.cuda.synchronize()
        assert h.device_status() == 0
        c, t = gates(ref, to_f64(y), "bf16", "BIAS_RELU")
        assert c <= 1 and t <= 1, (sched, c, t)
        outs.append(y)


def test_dynamic_schedule_refusals_and_fallbacks(h):
    case = mk("dyn_refuse", 1500, 1152, 512)
    ins = wl.make_inputs(case)
    with pytest.raises(FactError):  # K slices are not whole tiles
        run_gpu(h, ins, case, cfg={"tile_m": 128, "tile_n": 64, "cta_group": 1, "schedule": 2, "split_k": 2})
    with pytest.raises(FactError):
        run_gpu(h, ins, case, cfg={"schedule": 3})
    # a single wave: nothing to hand out, the static grid runs
    small = mk("dyn_one_wave", 300, 200, 128)
    check_case(h, small, cfg={"tile_m": 128, "tile_n": 64, "cta_group": 1, "schedule": 2})


def test_dynamic_schedule_in_a_cuda_graph_and_back_to_back(h):
    """A dynamically scheduled launch can be captured and replayed, and launches that follow one another on a stream
    (each is allowed to move onto the SMs while its predecessor's last CTAs leave) give the same bits every time."""
    case = mk("dyn_graph", 2048, 1024, 520, epilogue="BIAS_RELU")
    ins = wl.make_inputs(case)
    dev = "cuda:0"
    X, W, b = ins.X.to(dev), ins.W.to(dev), ins.bias.to(dev)
    cfg = {"tile_m": 256, "tile_n": 64, "cta_group": 2, "schedule": 2}
    first = h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", cfg=cfg)
    torch.cuda.synchronize()
    out = torch.empty_like(first)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream(dev)):
        for _ in range(4):  # four launches back to back inside the graph
            h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", out=out, cfg=cfg)
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, first)
    assert h.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", case.epilogue)
    assert c <= 1 and t <= 1, (c, t)
