"""GPU parity of fact_linear_fp8 (FP8 E4M3 operands, tcgen05.mma.kind::f8f6f4) against the FP64 FP8 oracle."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import fp8 as ofp8
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, stratified_rows, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def bias_f64(ins):
    return None if ins.bias is None else ins.bias.double().numpy()


def check(h, case, cfg=None, out_dtype=torch.bfloat16, rows=None, ins=None, tight_max=1.0):
    ins = ins or wl.make_fp8_inputs(case)
    dev = "cuda:0"
    got = h.linear_fp8(ins.X.to(dev), ins.W.to(dev), ins.scale, None if ins.bias is None else ins.bias.to(dev),
                       epilogue=case.epilogue, out_dtype=out_dtype, cfg=cfg)
    torch.cuda.synchronize()
    assert h.device_status() == 0, "a device-side wait timed out"
    g = to_f64(got)
    if rows is not None:
        g = g[rows]
    ref = ofp8.linear_fp8(ins.X.numpy(), ins.W.numpy(), ins.scale, bias_f64(ins), case.epilogue, rows=rows)
    assert g.shape == ref.shape and np.isfinite(g).all()
    c, t = gates(ref, g, "f32" if out_dtype == torch.float32 else "bf16", case.epilogue)
    assert c <= 1.0, f"{case.name}: contract gate ratio {c:.3f}"
    assert t <= tight_max, f"{case.name}: tight gate ratio {t:.3f}"
    return got


SMALL = [
    # name, M, N, K, epilogue, config
    ("one_tile", 128, 128, 128, "NONE", None),
    ("ragged_all", 300, 200, 272, "BIAS", None),                 # K = 2 k-blocks + 16
    ("relu_1cta_narrow", 513, 96, 1040, "BIAS_RELU", dict(tile_n=32, cta_group=1)),
    ("gelu_2cta", 1000, 640, 2048, "BIAS_GELU_TANH", dict(tile_n=256, cta_group=2)),
    ("short_k", 257, 384, 16, "NONE", None),                     # one partial k-block
    ("wide_1cta", 640, 1024, 512, "BIAS", dict(tile_n=256, cta_group=1, stages=4)),
    ("stream_k", 1280, 1280, 1024, "BIAS_GELU_TANH", dict(tile_n=64, cta_group=1, split_k=-1)),
    ("split_k", 256, 256, 8192, "BIAS", dict(tile_n=128, cta_group=1, split_k=8)),
]


@pytest.mark.parametrize("name,M,N,K,epi,cfg", SMALL, ids=[c[0] for c in SMALL])
def test_fp8_linear_matches_oracle(h, name, M, N, K, epi, cfg):
    case = wl.Fp8Case(name, M, N, K, epilogue=epi, has_bias=epi != "NONE", seed=21)
    check(h, case, cfg=cfg)


def test_fp8_f32_output(h):
    case = wl.Fp8Case("f32_out", 384, 320, 640, seed=22)
    check(h, case, out_dtype=torch.float32)


def test_fp8_is_exact_on_small_integers(h):
    """Operands that are small integers (all exactly representable in E4M3): every product and partial sum is an
    integer below 2^24, so FP32 accumulation is exact in any order and the FP32 output must EQUAL the oracle's."""
    g = torch.Generator().manual_seed(23)
    M, N, K = 515, 384, 1168
    X = torch.randint(-4, 5, (M, K), generator=g).float().to(torch.float8_e4m3fn).view(torch.uint8)
    W = torch.randint(-4, 5, (N, K), generator=g).float().to(torch.float8_e4m3fn).view(torch.uint8)
    for cfg in (None, dict(tile_n=64, cta_group=2), dict(tile_n=256, cta_group=2, split_k=-1), dict(tile_n=128, cta_group=1, split_k=3)):
        out = h.linear_fp8(X.cuda(), W.cuda(), 0.25, out_dtype=torch.float32, cfg=cfg)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        ref = ofp8.linear_fp8(X.numpy(), W.numpy(), 0.25)
        assert np.array_equal(out.double().cpu().numpy(), ref), cfg


def test_fp8_every_code_and_extremes(h):
    """All 254 finite codes as operands (subnormals included), the largest magnitudes against each other, and zeros."""
    codes = torch.tensor([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=torch.uint8)
    K = 256
    X = codes.repeat(2)[:K].unsqueeze(0).repeat(128, 1).contiguous()
    X = torch.roll(X, shifts=3, dims=1) if False else X
    W = torch.stack([torch.roll(codes.repeat(2)[:K], s) for s in range(64)]).contiguous()
    out = h.linear_fp8(X.cuda(), W.cuda(), 2.0 ** -10, out_dtype=torch.float32)
    torch.cuda.synchronize()
    ref = ofp8.linear_fp8(X.numpy(), W.numpy(), 2.0 ** -10)
    err = np.abs(out.double().cpu().numpy() - ref)
    # sums of up to 256 products of magnitude up to 448^2: FP32 accumulation error is bounded by K * 2^-24 * sum |x w|
    bound = K * 2.0 ** -24 * (np.abs(ofp8.e4m3_to_f64(X.numpy())) @ np.abs(ofp8.e4m3_to_f64(W.numpy())).T) * 2.0 ** -10
    assert (err <= bound + 1e-30).all()
    big = torch.full((128, 128), 0x7E, dtype=torch.uint8)
    out = h.linear_fp8(big.cuda(), big.cuda(), 1.0, out_dtype=torch.float32)
    assert torch.all(out == 448.0 * 448.0 * 128)
    zero = torch.zeros((128, 128), dtype=torch.uint8)
    out = h.linear_fp8(zero.cuda(), big.cuda(), 1.0, out_dtype=torch.float32)
    assert torch.all(out == 0)


def test_fp8_accepts_float8_tensors_and_residual_and_gate(h):
    g = torch.Generator().manual_seed(24)
    M, N, K = 256, 256, 512
    x = torch.randn((M, K), generator=g)
    wg = torch.randn((2 * N, K), generator=g) * 0.05
    r = torch.randn((M, N), generator=g).to(torch.bfloat16)
    xq, wq = x.to(torch.float8_e4m3fn), wg.to(torch.float8_e4m3fn)
    xv = ofp8.e4m3_to_f64(xq.view(torch.uint8).numpy())
    wv = ofp8.e4m3_to_f64(wq.view(torch.uint8).numpy())
    # SiLU(gate) * up
    out = h.linear_fp8(xq.cuda(), wq.cuda(), 0.5, epilogue="SILU_GATE")
    acc = 0.5 * (xv @ wv.T)
    gate, up = acc[:, :N], acc[:, N:]
    ref = gate / (1.0 + np.exp(-gate)) * up
    c, t = gates(ref, to_f64(out), "bf16", "SILU_GATE")
    assert c <= 1.0 and t <= 1.0, (c, t)
    # + residual
    out = h.linear_fp8(xq.cuda(), wq[:N].contiguous().cuda(), 0.5, residual=r.cuda(), epilogue="BIAS_RESIDUAL")
    ref = 0.5 * (xv @ wv[:N].T) + r.double().numpy()
    c, t = gates(ref, to_f64(out), "bf16", "BIAS_RESIDUAL")
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_fp8_argument_errors(h):
    from paper_2604_26666_b200.binding import lib, _ptr

    M, N, K = 128, 128, 128
    X = torch.zeros((M, K + 16), dtype=torch.uint8, device="cuda")
    W = torch.zeros((N, K), dtype=torch.uint8, device="cuda")
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    call = lambda x, ldx, scale=1.0: lib().fact_linear_fp8(h._h, M, N, K, x, ldx, _ptr(W), K, ctypes.c_float(scale), None, None, 0,
                                                          _ptr(Y), N, 0, 0, None, None, 0, s)
    assert call(_ptr(X), K + 16) == 0
    assert call(_ptr(X), K + 8) == 2                                   # rows must be 16-byte multiples
    assert call(ctypes.c_void_p(X.data_ptr() + 8), K + 16) == 2        # 16-byte aligned base
    assert call(_ptr(X), K - 16) == 1                                  # leading dimension below K
    assert call(_ptr(X), K + 16, float("nan")) == 1
    assert call(None, K + 16) == 1
    torch.cuda.synchronize()
    assert h.device_status() == 0


@pytest.mark.parametrize("name", [c.name for c in wl.fp8_cases()])
def test_fp8_full_size_sampled_rows(h, name):
    """The benchmark's FP8 shapes in the configuration bench.py times: a stratified sample of output rows against
    the oracle (every column of each)."""
    case = {c.name: c for c in wl.fp8_cases()}[name]
    rows = stratified_rows(case.M, 48, seed=3)
    check(h, case, rows=rows)
