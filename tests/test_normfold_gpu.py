"""GPU parity of the row normalisation folded between two linear layers (Table 1's "GEMM-LayerNorm-GEMM fusion"):
the partial row sums a producing call leaves (fact_linear_ex / fact_row_stats), the folded weights
(fact_fold_norm), and the consuming call that corrects its accumulator per row, each against the FP64 oracle of
the plain definition (oracle/normfold.py)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import normfold as nf
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def draw(shape, seed, scale=1.0, shift=0.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale + shift).to(torch.bfloat16)


def as_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(a, dtype=np.float64)).to(torch.bfloat16)


def fold_gate(ref, got, mean_over_std=0.0, pre=None, gated=False):
    """Worst |err| over its bound.  Besides the rounding of the output (1.5 * 2^-8 |ref|), every term x_k Wf[n,k] of
    the folded product carries the 2^-9 rounding of Wf, and the terms include the row mean that the correction takes
    out again: independent errors of 2^-9 / sqrt(3) on terms whose squares sum to (1 + (mean/std)^2) rms(z)^2,
    z the value before the activation (`pre`; the activations' slopes are at most 1.13), at 4.5 sigma over ~1e5
    outputs, is dz = 2.6 * 2^-9 * sqrt(1 + (mean/std)^2) rms(z); 2^-7 leaves a margin.  A gated output silu(g) * u
    (`pre` = [g | u]) moves by at most dz * (1.1 |u| + |silu(g)|)."""
    ref, got = np.asarray(ref, dtype=np.float64), np.asarray(got, dtype=np.float64)
    z = ref if pre is None else np.asarray(pre, dtype=np.float64)
    dz = 2.0 ** -7 * np.sqrt(1.0 + mean_over_std ** 2) * float(np.sqrt(np.mean(z * z)))
    if gated:
        g, u = z[:, :z.shape[1] // 2], z[:, z.shape[1] // 2:]
        dz = dz * (1.1 * np.abs(u) + np.abs(g / (1.0 + np.exp(-g))))
    bound = 1.5 * 2.0 ** -8 * np.abs(ref) + dz
    return float((np.abs(got - ref) / bound).max())


def pre_activation(epi):
    """The epilogue whose oracle output is the value the activation of `epi` is applied to (None: `epi` has none)."""
    return {"BIAS_RELU": "BIAS", "BIAS_GELU_TANH": "BIAS", "SILU_GATE": "NONE"}.get(epi)


# ---------------------------------------------------------------------------------------------- row sums of a tensor
@pytest.mark.parametrize("M,C", [(77, 768), (1000, 200), (129, 4096), (5, 8), (2051, 1032)])
def test_row_stats_kernel(h, M, C):
    x = draw((M, C), 100 + M, 1.3, 0.4)
    got = h.row_stats(x.to(DEV)).cpu().double().numpy()
    ref = nf.row_stats(wl.bits(x))
    assert got.shape == ref.shape
    mag = np.abs(to_f64(x)).max()
    assert np.abs(got[:, :, 0] - ref[:, :, 0]).max() <= 64 * 2.0 ** -22 * mag
    assert np.abs(got[:, :, 1] - ref[:, :, 1]).max() <= 64 * 2.0 ** -22 * mag * mag


# ------------------------------------------------------------------------------------ row sums left by a linear layer
PRODUCERS = [
    # M, N, K, epilogue, cfg
    (300, 768, 256, "BIAS_RESIDUAL", None),
    (1061, 320, 512, "BIAS", None),                       # the second n-tile holds one 64-column chunk only
    (515, 192, 128, "NONE", dict(cta_group=1, tile_n=64)),
    (640, 512, 320, "BIAS_GELU_TANH", dict(cta_group=2, tile_n=128)),
    (1024, 384, 256, "SILU_GATE", dict(tile_n=256)),        # (the default tile, 96 output columns, is not stageable)
    (2048, 2304, 768, "BIAS_RESIDUAL", dict(split_k=-1)),   # a stream-K request is dropped: the tiles run whole
    (4224, 768, 768, "BIAS_RESIDUAL", None),
    (300, 200, 128, "BIAS_RESIDUAL", None),               # the last chunk holds 8 columns: the others add zeros
    (5, 64, 72, "BIAS_RELU", None),                       # fewer rows than a warp owns
]


@pytest.mark.parametrize("M,N,K,epi,cfg", PRODUCERS)
def test_linear_leaves_row_sums(h, M, N, K, epi, cfg):
    Nw = 2 * N if epi == "SILU_GATE" else N
    x, w = draw((M, K), 1, 1.0), draw((Nw, K), 2, 1.0 / np.sqrt(K))
    bias = draw((N,), 3, 0.5) if epi.startswith("BIAS") else None
    res = draw((M, N), 4, 1.0, 0.3) if epi == "BIAS_RESIDUAL" else None
    stats = torch.full(((N + 63) // 64, M, 2), float("nan"), dtype=torch.float32, device=DEV)
    y = h.linear(x.to(DEV), w.to(DEV), bias=None if bias is None else bias.to(DEV),
                 residual=None if res is None else res.to(DEV), epilogue=epi, cfg=cfg, stats_out=stats)
    torch.cuda.synchronize()
    ref = oracle.linear(wl.bits(x), wl.bits(w), layout="NK", epilogue=epi, bias=None if bias is None else wl.bits(bias),
                        residual=None if res is None else wl.bits(res))
    assert np.abs(to_f64(y) - ref).max() <= 1e-2 + 1e-2 * np.abs(ref).max()
    # expected sums: over the oracle's values rounded to BF16.  The device rounds an FP32 value, the oracle an FP64
    # one: a few elements per chunk may land on the neighbouring BF16 value (2^-8 relative each), nothing more.
    want = nf.row_stats(wl.bits(as_bf16(ref)))
    got = stats.cpu().double().numpy()
    assert not np.isnan(got).any()  # every (chunk, row) was written
    mag = np.abs(ref).max()
    assert np.abs(got[:, :, 0] - want[:, :, 0]).max() <= 2.0 ** -6 * mag
    assert np.abs(got[:, :, 1] - want[:, :, 1]).max() <= 2.0 ** -5 * mag * mag
    # and they are the sums of exactly what was stored (a property: the stand-alone kernel over the device's own output)
    again = h.row_stats(y).cpu().double().numpy()
    assert np.abs(got - again).max() <= 64 * 2.0 ** -21 * max(mag, mag * mag)


# ------------------------------------------------------------------------------------------------ the folded weights
@pytest.mark.parametrize("N,K,with_beta,with_bias", [(100, 768, True, True), (257, 4096, False, False),
                                                      (64, 64, True, False), (3, 8, True, True)])
def test_fold_norm_kernel(h, N, K, with_beta, with_bias):
    w, gamma = draw((N, K), 11, 0.05), draw((K,), 12, 0.2, 1.0)
    beta = draw((K,), 13, 0.1) if with_beta else None
    bias = draw((N,), 14, 0.5) if with_bias else None
    wf, cs, bf = h.fold_norm(w.to(DEV), gamma.to(DEV), None if beta is None else beta.to(DEV),
                             None if bias is None else bias.to(DEV))
    prod, shift = nf.fold_norm(wl.bits(w), wl.bits(gamma), None if beta is None else wl.bits(beta),
                               None if bias is None else wl.bits(bias))
    want_wf = as_bf16(prod)  # the product is exact in FP32 and in FP64: one rounding either way, so bit-identical
    assert torch.equal(wf.cpu().view(torch.int16), want_wf.view(torch.int16))
    want_cs = to_f64(want_wf).sum(axis=1)
    assert np.abs(cs.cpu().double().numpy() - want_cs).max() <= K * 2.0 ** -23 * np.abs(to_f64(want_wf)).sum(axis=1).max()
    if with_beta:
        assert np.abs(to_f64(bf) - shift).max() <= 2.0 ** -8 * np.abs(shift).max() + 1e-6
    else:
        assert bf is None


# ------------------------------------------------------------------------------------------------ the consuming layer
CONSUMERS = [
    # M, N, K, kind, epilogue, mean/std of the rows, cfg
    (300, 256, 768, "layer", "BIAS", 0.3, None),
    (1061, 320, 512, "layer", "BIAS_GELU_TANH", 0.5, None),
    (515, 128, 200, "layer", "BIAS_RELU", 0.0, dict(cta_group=1, tile_n=64)),       # K not a multiple of 64
    (2048, 3072, 768, "layer", "BIAS_GELU_TANH", 0.25, None),
    (640, 192, 320, "layer", "BIAS_RESIDUAL", 0.3, dict(cta_group=2, tile_n=128)),
    (1024, 384, 512, "rms", "NONE", 0.3, None),
    (777, 256, 1024, "rms", "SILU_GATE", 0.1, dict(tile_n=128)),   # (64 stored columns per tile: the narrowest staged gate)
    (2048, 2304, 768, "rms", "NONE", 0.2, dict(split_k=-1)),
]


def consumer_inputs(M, N, K, kind, epi, mos, seed=0):
    Nw = 2 * N if epi == "SILU_GATE" else N
    x = draw((M, K), seed + 21, 1.0, mos)
    w = draw((Nw, K), seed + 22, 1.0 / np.sqrt(K))
    gamma = draw((K,), seed + 23, 0.2, 1.0)
    beta = draw((K,), seed + 24, 0.1) if kind == "layer" else None
    bias = draw((N,), seed + 25, 0.5) if epi.startswith("BIAS") else None
    res = draw((M, N), seed + 26, 1.0) if epi == "BIAS_RESIDUAL" else None
    return x, w, gamma, beta, bias, res


@pytest.mark.parametrize("M,N,K,kind,epi,mos,cfg", CONSUMERS)
def test_consumer_against_definition(h, M, N, K, kind, epi, mos, cfg):
    """The consuming call alone: its row sums and folded weights are prepared on the host from the oracle's
    definitions, so only the corrected product is under test."""
    x, w, gamma, beta, bias, res = consumer_inputs(M, N, K, kind, epi, mos)
    eps = 1e-5
    prod, shift = nf.fold_norm(wl.bits(w), wl.bits(gamma), None if beta is None else wl.bits(beta),
                               None if bias is None or beta is None else wl.bits(bias))
    wf = as_bf16(prod)
    colsum = torch.from_numpy(to_f64(wf).sum(axis=1)).float() if kind == "layer" else None
    bias_f = as_bf16(shift) if shift is not None else bias
    stats = torch.from_numpy(nf.row_stats(wl.bits(x))).float().contiguous()
    y = h.linear(x.to(DEV), wf.to(DEV), bias=None if bias_f is None else bias_f.to(DEV),
                 residual=None if res is None else res.to(DEV), epilogue=epi, cfg=cfg, x_norm=kind,
                 x_stats=stats.to(DEV), w_colsum=None if colsum is None else colsum.to(DEV), eps=eps)
    torch.cuda.synchronize()
    ref = nf.norm_linear(wl.bits(x), wl.bits(w), wl.bits(gamma), kind=kind, eps=eps,
                         beta_bits=None if beta is None else wl.bits(beta),
                         bias_bits=None if bias is None else wl.bits(bias),
                         residual_bits=None if res is None else wl.bits(res), epilogue=epi)
    pre = None
    if pre_activation(epi):
        pre = nf.norm_linear(wl.bits(x), wl.bits(w), wl.bits(gamma), kind=kind, eps=eps,
                             beta_bits=None if beta is None else wl.bits(beta),
                             bias_bits=None if bias is None else wl.bits(bias), epilogue=pre_activation(epi))
    assert fold_gate(ref, to_f64(y), mos, pre, gated=epi == "SILU_GATE") <= 1.0


@pytest.mark.parametrize("kind", ["layer", "rms"])
def test_chain_through_the_library(h, kind):
    """Producer -> (folded normalisation) -> consumer, everything by this library's kernels: out-projection with
    residual leaves the row sums, fact_fold_norm prepares the weights, the MLP's first layer consumes both.  The
    oracle rounds the intermediate activation to BF16 where the device stores it."""
    M, H, F = 1500, 768, 1024
    a, wo, bo = draw((M, H), 31), draw((H, H), 32, 1.0 / np.sqrt(H)), draw((H,), 33, 0.2)
    x0 = draw((M, H), 34, 1.0, 0.3)
    gamma = draw((H,), 35, 0.2, 1.0)
    beta = draw((H,), 36, 0.1) if kind == "layer" else None
    gate = kind == "rms"
    w1 = draw(((2 * F) if gate else F, H), 37, 1.0 / np.sqrt(H))
    b1 = None if gate else draw((F,), 38, 0.3)
    epi2 = "SILU_GATE" if gate else "BIAS_GELU_TANH"
    stats = torch.empty((H // 64, M, 2), dtype=torch.float32, device=DEV)
    x1 = h.linear(a.to(DEV), wo.to(DEV), bias=bo.to(DEV), residual=x0.to(DEV), epilogue="BIAS_RESIDUAL",
                  stats_out=stats)
    wf, cs, bf = h.fold_norm(w1.to(DEV), gamma.to(DEV), None if beta is None else beta.to(DEV),
                             None if b1 is None else b1.to(DEV))
    y = h.linear(x1, wf, bias=bf, epilogue=epi2, x_norm=kind, x_stats=stats,
                 w_colsum=cs if kind == "layer" else None, eps=1e-5, cfg=dict(tile_n=256) if gate else None)
    torch.cuda.synchronize()
    x1_ref = oracle.linear(wl.bits(a), wl.bits(wo), layout="NK", epilogue="BIAS_RESIDUAL", bias=wl.bits(bo),
                           residual=wl.bits(x0))
    x1_bits = wl.bits(as_bf16(x1_ref))
    ref = nf.norm_linear(x1_bits, wl.bits(w1), wl.bits(gamma), kind=kind, eps=1e-5,
                         beta_bits=None if beta is None else wl.bits(beta),
                         bias_bits=None if b1 is None else wl.bits(b1), epilogue=epi2)
    x1f = to_f64(as_bf16(x1_ref))
    mos = float(np.abs(x1f.mean(axis=1) / x1f.std(axis=1)).max())
    pre = nf.norm_linear(x1_bits, wl.bits(w1), wl.bits(gamma), kind=kind, eps=1e-5,
                         beta_bits=None if beta is None else wl.bits(beta),
                         bias_bits=None if b1 is None else wl.bits(b1), epilogue="NONE" if gate else "BIAS")
    assert fold_gate(ref, to_f64(y), mos, pre, gated=gate) <= 1.0
    # and the unfused route through fact_norm + fact_linear agrees with the same oracle under the plain gate
    n = h.norm(x1, gamma.to(DEV), None if beta is None else beta.to(DEV), kind=kind, eps=1e-5)
    y2 = h.linear(n, w1.to(DEV), bias=None if b1 is None else b1.to(DEV), epilogue=epi2)
    assert fold_gate(ref, to_f64(y2), 0.0, pre, gated=gate) <= 1.0


def test_refusals(h):
    from paper_2604_26666_b200.binding import FactError
    M, N, K = 256, 128, 128
    x, w = draw((M, K), 41).to(DEV), draw((N, K), 42).to(DEV)
    stats_n = torch.zeros((N // 64, M, 2), dtype=torch.float32, device=DEV)
    stats_k = torch.zeros((K // 64, M, 2), dtype=torch.float32, device=DEV)
    cs = torch.zeros(N, dtype=torch.float32, device=DEV)

    def code(**kw):
        with pytest.raises(FactError) as e:
            h.linear(x, kw.pop("w", w), **kw)
        return e.value.code

    assert code(stats_out=stats_n, out_dtype=torch.float32) == 3            # sums are over BF16 stores
    assert code(stats_out=stats_n, cfg=dict(store_mode=1)) == 3             # the direct-store path has no sums
    assert code(stats_out=stats_n, cfg=dict(split_k=2)) == 3                # K slices end in another kernel
    assert code(x_norm="layer", x_stats=stats_k) == 1                       # LayerNorm needs the column sums
    assert code(x_norm="rms") == 1                                          # and both need the row sums
    assert code(x_stats=stats_k) == 1                                       # row sums without a normalisation
    assert code(x_norm="layer", x_stats=stats_k, w_colsum=torch.zeros(2 * N, dtype=torch.float32, device=DEV)[:N],
                w=draw((2 * N, K), 43).to(DEV), epilogue="SILU_GATE") == 3  # gated: RMS only
    w96 = draw((96, K), 44).to(DEV)
    assert code(w=w96, x_norm="layer", x_stats=stats_k, w_colsum=cs[:96]) == 3   # N_out not a multiple of 64
    # nothing above may have left an error behind
    assert h.device_status() == 0
