"""GPU parity of the row-softmax epilogue (FACT_EPI_BIAS_SOFTMAX, Table 1's "GEMM-Softmax") against the oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import to_f64

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


CASES = [
    # M, N, K, bias, layout, out, config
    (300, 256, 512, True, "NK", "bf16", None),
    (1000, 200, 264, True, "NK", "bf16", None),          # ragged row width: 200 of a 224-wide tile
    (515, 10, 128, False, "NK", "f32", None),            # a classifier head: 10 classes
    (129, 1, 64, True, "NK", "f32", None),               # one column: every output is 1
    (640, 96, 1040, True, "KN", "bf16", dict(cta_group=1)),
    (2048, 256, 768, True, "NK", "bf16", dict(cta_group=2, tile_n=256)),
    (4096, 128, 256, False, "NK", "bf16", dict(cta_group=2)),
    (260, 33, 96, True, "NK", "f32", dict(tile_n=64, cta_group=1)),
]


@pytest.mark.parametrize("M,N,K,has_bias,layout,out,cfg", CASES)
def test_softmax_epilogue_matches_oracle(h, M, N, K, has_bias, layout, out, cfg):
    X = draw((M, K), 51)
    W = draw((N, K) if layout == "NK" else (K, N), 52, 2.0 * K ** -0.5)  # logits of a few units: a peaked softmax
    bias = draw((N,), 53) if has_bias else None
    odt = torch.float32 if out == "f32" else torch.bfloat16
    y = h.linear(X.cuda(), W.cuda(), bias=None if bias is None else bias.cuda(), epilogue="BIAS_SOFTMAX", layout=layout,
                 out_dtype=odt, cfg=cfg)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    ref = oracle.linear_softmax(wl.bits(X), wl.bits(W), layout=layout, bias=None if bias is None else wl.bits(bias))
    got = to_f64(y)
    assert got.shape == ref.shape and np.isfinite(got).all()
    err = np.abs(got - ref)
    # probabilities: exp of logits known to FP32 accumulation accuracy (relative error of p about |dz| <= 1e-4 at
    # these sizes) with __expf (2e-7), normalised; BF16 outputs add one rounding (2^-9 relative)
    tol = (2.0 ** -8 * ref + 1e-6) if out == "bf16" else (5e-4 * ref + 1e-7)
    assert (err <= tol).all(), float((err / tol).max())
    if out == "f32":
        assert np.allclose(got.sum(axis=1), 1.0, atol=1e-5)


def test_softmax_extreme_logits_do_not_overflow(h):
    M, N, K = 256, 64, 128
    X = draw((M, K), 54, 8.0)
    W = draw((N, K), 55, 8.0)  # logits of several hundred
    y = h.linear(X.cuda(), W.cuda(), epilogue="BIAS_SOFTMAX", layout="NK", out_dtype=torch.float32)
    torch.cuda.synchronize()
    ref = oracle.linear_softmax(wl.bits(X), wl.bits(W), layout="NK")
    got = y.double().cpu().numpy()
    assert np.isfinite(got).all() and np.allclose(got.sum(axis=1), 1.0, atol=1e-5)
    assert np.array_equal(got.argmax(axis=1), ref.argmax(axis=1))
    assert np.abs(got - ref).max() <= 2e-2  # logits of magnitude 500 carry FP32 accumulation errors of 1e-3 or so


def test_softmax_unsupported_forms(h):
    from paper_2604_26666_b200.binding import FactError

    X, W = draw((128, 64), 56).cuda(), draw((300, 64), 57).cuda()
    with pytest.raises(FactError) as e:
        h.linear(X, W, epilogue="BIAS_SOFTMAX", layout="NK")       # a row wider than a tile
    assert e.value.code == 3
    W = draw((128, 64), 58).cuda()
    for bad in (dict(split_k=2), dict(split_k=-1), dict(store_mode=2), dict(tile_n=64)):
        with pytest.raises(FactError) as e:
            h.linear(X, W, epilogue="BIAS_SOFTMAX", layout="NK", cfg=bad)
        assert e.value.code == 3, bad
    R = draw((128, 128), 59).cuda()
    with pytest.raises(FactError) as e:
        h.linear(X, W, residual=R, epilogue="BIAS_SOFTMAX", layout="NK")
    assert e.value.code == 1
