"""Seeded random sweep over shapes, layouts, epilogues and kernel configurations (pair size, tile width,
ring depth, raster group, K slices, store mode), each compared with the FP64 oracle element by element.
Small problems, many of them: ragged tails in M, N and K, tiles wider than the problem, 2-CTA pairs on an
odd number of 128-row blocks, gated epilogues across tile borders."""
import numpy as np
import pytest
import torch

from paper_2604_26666_b200 import workloads as wl
from paper_2604_26666_b200.binding import FactError
from tests.helpers import check_case

pytestmark = pytest.mark.gpu

EPIS = ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"]


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def random_case(rng, i):
    epi = EPIS[int(rng.integers(0, len(EPIS)))]
    layout = "KN" if rng.random() < 0.5 else "NK"
    out = "f32" if rng.random() < 0.3 else "bf16"
    M = int(rng.choice([1, 7, 64, 128, 129, 200, 256, 300, 384, 513]))
    N = int(rng.choice([8, 24, 64, 72, 128, 136, 200, 256, 264, 392, 520]))
    K = int(rng.choice([8, 64, 72, 128, 264, 520, 1032]))
    batch = int(rng.choice([1, 1, 1, 3]))
    op = "linear" if epi != "NONE" or rng.random() < 0.3 else ("gemm_batched" if batch > 1 else "gemm")
    if op != "gemm_batched":
        batch = 1
    has_bias = epi in ("BIAS", "BIAS_RELU", "BIAS_GELU_TANH") or (epi == "BIAS_RESIDUAL" and rng.random() < 0.6)
    case = wl.Case(f"rnd{i}", op, M, N, K, batch=batch, epilogue=epi, layout=layout, out=out, has_bias=has_bias,
                   has_residual=epi == "BIAS_RESIDUAL", seed=1000 + i, w_scale=0.08)
    cfg = {}
    if rng.random() < 0.8:
        cfg["cta_group"] = int(rng.choice([1, 2]))
    if rng.random() < 0.7:
        cfg["tile_n"] = int(rng.choice([32, 64, 96, 128, 160, 192, 256]))
    if rng.random() < 0.5:
        cfg["stages"] = int(rng.choice([2, 3, 4]))
    if rng.random() < 0.5:
        cfg["raster_group"] = int(rng.choice([1, 2, 3, 16]))
    if rng.random() < 0.35:
        cfg["split_k"] = int(rng.choice([2, 3, 5]))
    if rng.random() < 0.3:
        cfg["store_mode"] = 1
    return case, cfg


@pytest.mark.parametrize("seed", range(6))
def test_random_sweep(h, seed):
    rng = np.random.default_rng(seed)
    ran = 0
    for i in range(40):
        case, cfg = random_case(rng, seed * 100 + i)
        try:
            check_case(h, case, cfg=cfg or None)
            ran += 1
        except FactError as e:
            # configurations the library documents as unsupported (tile width vs layout / gate / pair size, stage
            # budget, staged stores on an unaligned output) are rejected before anything is launched
            assert e.code == 3, (case, cfg, e)
        except AssertionError as e:
            raise AssertionError(f"{case} cfg={cfg}: {e}") from e
    assert ran >= 15, f"only {ran} of 40 random cases were runnable"


@pytest.mark.parametrize("seed", [100, 101])
def test_random_sweep_register_row_stores(h, seed):
    """The same sweep with the rows stored from registers in 32-byte pieces (store_mode 3): no K slices, and only
    shapes it accepts have to run (output rows of whole 32-byte pieces, a stageable tile)."""
    rng = np.random.default_rng(seed)
    ran = 0
    for i in range(40):
        case, cfg = random_case(rng, seed * 100 + i)
        cfg.pop("split_k", None)
        cfg["store_mode"] = 3
        try:
            check_case(h, case, cfg=cfg)
            ran += 1
        except FactError as e:
            assert e.code == 3, (case, cfg, e)
        except AssertionError as e:
            raise AssertionError(f"{case} cfg={cfg}: {e}") from e
    assert ran >= 8, f"only {ran} of 40 random cases were runnable"
