"""GPU parity of fact_linear_grouped (row groups with a weight matrix each, one launch) against the oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def draw(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


def run_and_check(h, rows, N, K, epilogue="NONE", layout="NK", out_dtype=torch.bfloat16, cfg=None, seed=0):
    G, M = len(rows), sum(rows)
    Nw = 2 * N if epilogue == "SILU_GATE" else N
    X = draw((M, K), seed)
    W = draw((G, Nw, K) if layout == "NK" else (G, K, Nw), seed + 1, K ** -0.5)
    bias = draw((N,), seed + 2) if epilogue.startswith("BIAS") else None
    res = draw((M, N), seed + 3) if epilogue == "BIAS_RESIDUAL" else None
    dev = "cuda:0"
    out = h.linear_grouped(X.to(dev), W.to(dev), rows, bias=None if bias is None else bias.to(dev),
                           residual=None if res is None else res.to(dev), epilogue=epilogue, layout=layout,
                           out_dtype=out_dtype, cfg=cfg)
    torch.cuda.synchronize()
    assert h.device_status() == 0, "a device-side wait timed out"
    ref = oracle.linear_grouped(wl.bits(X), wl.bits(W), rows, layout=layout, epilogue=epilogue,
                                bias=None if bias is None else wl.bits(bias),
                                residual=None if res is None else wl.bits(res))
    g = to_f64(out)
    assert g.shape == ref.shape and np.isfinite(g).all()
    c, t = gates(ref, g, "f32" if out_dtype == torch.float32 else "bf16", epilogue)
    assert c <= 1.0 and t <= 1.0, (c, t)
    return out


CASES = [
    # name, group rows, N, K, epilogue, layout, config
    ("ragged_groups", [200, 1, 130, 128, 515], 384, 264, "NONE", "NK", None),
    ("empty_groups", [0, 300, 0, 0, 77, 0], 256, 128, "BIAS", "NK", None),
    ("one_group", [700], 320, 512, "BIAS_RELU", "NK", None),
    ("many_small_groups", [((7 * i) % 41) for i in range(96)], 192, 320, "BIAS_GELU_TANH", "NK", None),
    ("pairs_of_ctas", [300, 256, 1, 255, 257], 512, 256, "NONE", "NK", dict(tile_n=128, cta_group=2)),
    ("wide_pair_tiles", [1000, 24, 1500], 1024, 384, "BIAS", "NK", dict(tile_n=256, cta_group=2)),
    ("narrow_tiles", [90, 400, 33], 200, 96, "BIAS", "NK", dict(tile_n=32, cta_group=1)),
    ("silu_gate", [260, 120, 400], 256, 192, "SILU_GATE", "NK", None),
    ("residual", [129, 511, 64], 384, 256, "BIAS_RESIDUAL", "NK", None),
    ("kn_layout", [200, 333, 90], 320, 256, "BIAS", "KN", None),
    ("direct_stores", [200, 1, 130, 128, 515], 384, 264, "BIAS_RESIDUAL", "NK", dict(store_mode=1)),
    ("direct_odd_width", [90, 400, 33], 203, 96, "BIAS", "NK", None),     # rows of 406 bytes: registers only
    ("staged_residual_pairs", [300, 256, 1, 255, 257], 512, 256, "BIAS_RESIDUAL", "NK", dict(tile_n=256, cta_group=2)),
]


@pytest.mark.parametrize("name,rows,N,K,epi,layout,cfg", CASES, ids=[c[0] for c in CASES])
def test_grouped_matches_oracle(h, name, rows, N, K, epi, layout, cfg):
    run_and_check(h, rows, N, K, epilogue=epi, layout=layout, cfg=cfg, seed=31)


def test_grouped_f32_output_and_exact_integers(h):
    run_and_check(h, [150, 300, 70], 256, 320, out_dtype=torch.float32, seed=32)
    g = torch.Generator().manual_seed(33)
    rows = [130, 0, 259, 1, 400]
    M, N, K = sum(rows), 320, 448
    X = torch.randint(-3, 4, (M, K), generator=g).float().to(torch.bfloat16)
    W = torch.randint(-3, 4, (len(rows), N, K), generator=g).float().to(torch.bfloat16)
    for cfg in (None, dict(tile_n=64, cta_group=2), dict(tile_n=256, cta_group=1)):
        out = h.linear_grouped(X.cuda(), W.cuda(), rows, out_dtype=torch.float32, cfg=cfg)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        ref = oracle.linear_grouped(wl.bits(X), wl.bits(W), rows, layout="NK")
        assert np.array_equal(out.double().cpu().numpy(), ref), cfg


def test_grouped_rows_outside_the_groups_are_untouched(h):
    """The output buffer has more rows than the groups cover, and a leading dimension larger than N: nothing outside
    the [M x N] result may be written (tiles are ragged at every group's end)."""
    rows = [100, 37, 200]
    M, N, K = sum(rows), 192, 128
    X, W = draw((M, K), 34), draw((3, N, K), 35, K ** -0.5)
    buf = torch.full((M + 300, N + 64), 7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[:M, :N]
    h.linear_grouped(X.cuda(), W.cuda(), rows, out=out)
    torch.cuda.synchronize()
    assert torch.all(buf[M:] == 7.0) and torch.all(buf[:M, N:] == 7.0)
    ref = oracle.linear_grouped(wl.bits(X), wl.bits(W), rows, layout="NK")
    c, t = gates(ref, to_f64(out.contiguous()), "bf16", "NONE")
    assert c <= 1.0 and t <= 1.0


def test_grouped_argument_errors(h):
    from paper_2604_26666_b200.binding import Config, lib, _ptr

    M, N, K = 256, 128, 128
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((2, N, K), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    i64 = ctypes.c_int64

    def call(groups, rows, stride_w=N * K, cfg=None):
        arr = (i64 * max(len(rows), 1))(*rows)
        return lib().fact_linear_grouped(h._h, groups, arr, N, K, _ptr(X), K, _ptr(W), K, stride_w, 1, None, None, 0, _ptr(Y), N,
                                         0, 0, cfg, s)

    assert call(2, [128, 128]) == 0
    assert call(0, []) == 0                       # no groups: nothing to do
    assert call(2, [0, 0]) == 0
    assert call(2, [128, -1]) == 1                # negative row count
    assert call(5000, [0] * 5000) == 1            # more groups than the handle's table holds
    assert call(2, [128, 128], stride_w=N * K - 8) == 1   # the groups' weights overlap
    assert call(2, [128, 128], stride_w=N * K + 4) == 2   # stride not a multiple of 8 elements
    assert call(2, [128, 128], cfg=ctypes.byref(Config(split_k=2))) == 3
    assert call(2, [128, 128], cfg=ctypes.byref(Config(split_k=-1))) == 3
    assert call(2, [128, 128], cfg=ctypes.byref(Config(store_mode=2))) == 0   # staged: rows of whole 16-byte pieces
    assert call(2, [128, 128], cfg=ctypes.byref(Config(store_mode=1))) == 0   # straight from registers
    torch.cuda.synchronize()
    assert h.device_status() == 0


@pytest.mark.parametrize("epi,cfg", [("NONE", None), ("BIAS_GELU_TANH", dict(tile_n=128, cta_group=2)),
                                     ("SILU_GATE", dict(tile_n=256, cta_group=1))])
def test_grouped_fp8_matches_oracle(h, epi, cfg):
    """FP8 E4M3 operands through the grouped path: the oracle is the FP8 linear oracle, group by group."""
    from oracle import fp8 as ofp8

    rows = [140, 0, 300, 1, 259]
    M, N, K = sum(rows), 256, 400
    Nw = 2 * N if epi == "SILU_GATE" else N
    g = torch.Generator().manual_seed(41)
    X = (torch.randn((M, K), generator=g) * 2).to(torch.float8_e4m3fn)
    W = (torch.randn((len(rows), Nw, K), generator=g) * 0.5).to(torch.float8_e4m3fn)
    bias = torch.randn((N,), generator=g).to(torch.bfloat16) if epi.startswith("BIAS") else None
    scale = 0.05
    out = h.linear_grouped_fp8(X.cuda(), W.cuda(), rows, scale, None if bias is None else bias.cuda(), epilogue=epi, cfg=cfg)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    xc, wc = X.view(torch.uint8).numpy(), W.view(torch.uint8).numpy()
    ref = np.empty((M, N))
    r0 = 0
    for gi, n in enumerate(rows):
        if n:
            if epi == "SILU_GATE":
                acc = ofp8.linear_fp8(xc[r0:r0 + n], wc[gi], scale)
                gate, up = acc[:, :N], acc[:, N:]
                ref[r0:r0 + n] = gate / (1.0 + np.exp(-gate)) * up
            else:
                ref[r0:r0 + n] = ofp8.linear_fp8(xc[r0:r0 + n], wc[gi], scale,
                                                 None if bias is None else bias.double().numpy(), epi)
        r0 += n
    c, t = gates(ref, to_f64(out), "bf16", epi)
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_grouped_benchmark_shape_sampled_rows(h):
    """The short-K grouped shape of the benchmark's table at full size, in the configuration the benchmark times
    (staged stores): rows sampled at every group boundary and in between, each against the oracle."""
    case = [c for c in wl.grouped_cases() if c.name == "g8_short_k_gelu"][0]
    rows = wl.grouped_rows(case)
    X, W = wl.make_grouped_inputs(case, "cuda:0")
    gb = torch.Generator(device="cuda:0").manual_seed(case.seed + 2)
    bias = (torch.randn((case.N,), generator=gb, device="cuda:0", dtype=torch.float32) * 0.02).to(torch.bfloat16)
    out = h.linear_grouped(X, W, rows, bias=bias, epilogue=case.epilogue)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    starts = np.concatenate([[0], np.cumsum(rows)])
    rng = np.random.default_rng(5)
    worst_c = worst_t = 0.0
    Xc, bc = X.cpu(), bias.cpu()
    for g, n in enumerate(rows):
        if n == 0:
            continue
        local = sorted({0, n - 1, n // 2, *rng.integers(0, n, size=4).tolist()})
        idx = [int(starts[g]) + r for r in local]
        ref = oracle.linear(wl.bits(Xc[idx].contiguous()), wl.bits(W[g].cpu()), layout="NK", epilogue=case.epilogue,
                            bias=wl.bits(bc))
        c, t = gates(ref, to_f64(out[idx]), "bf16", case.epilogue)
        worst_c, worst_t = max(worst_c, c), max(worst_t, t)
    assert worst_c <= 1.0 and worst_t <= 1.0, (worst_c, worst_t)
