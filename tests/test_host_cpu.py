"""CPU-only checks of the host side: the library loads and exports every symbol the header declares,
the header and the binding agree, the workload table matches the benchmark configurations."""
import re
from pathlib import Path

import pytest

from paper_2604_26666_b200 import workloads as wl

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def libfact():
    from paper_2604_26666_b200 import build
    from paper_2604_26666_b200.binding import lib

    build.build()  # nvcc cross-compiles for sm_100a without a GPU
    return lib()


def declared_symbols():
    text = (ROOT / "include" / "fact.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fact_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(libfact):
    from paper_2604_26666_b200.binding import EXPORTED

    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(libfact, n), f"{n} is declared in fact.h but not exported"
    assert sorted(EXPORTED) == names, "binding.EXPORTED and fact.h disagree"


def test_status_strings(libfact):
    assert libfact.fact_status_string(0) == b"FACT_OK"
    assert libfact.fact_status_string(7) == b"FACT_ERR_DEVICE_TIMEOUT"
    assert libfact.fact_status_string(99) == b"FACT_ERR_UNKNOWN"


def test_calls_without_a_handle_fail_cleanly(libfact):
    from ctypes import byref, c_int, c_size_t

    n = c_size_t(0)
    assert libfact.fact_workspace_bytes(None, 0, 1, 8, 8, 8, 0, 0, 0, None, byref(n)) == 1
    assert libfact.fact_gemm(None, 8, 8, 8, None, 8, None, 8, 0, None, 8, 0, None, None, 0, None) == 1
    assert libfact.fact_launch_count(None) == 0
    assert libfact.fact_destroy(None) == 0
    v = c_int(0)
    assert libfact.fact_device_status(None, None, byref(v)) == 1


def test_no_product_module_imports_the_oracle():
    for f in (ROOT / "paper_2604_26666_b200").glob("*.py"):
        assert not re.search(r"^\s*(import|from)\s+oracle\b", f.read_text(), flags=re.M), f
    for f in (ROOT / "paper_2604_26666_b200" / "csrc").iterdir():
        assert "oracle" not in f.read_text().lower(), f
    assert "paper_2604_26666_b200" not in (ROOT / "oracle" / "__init__.py").read_text().replace(
        "CUDA package", "")


def test_workload_table_matches_the_configurations():
    cases = {c.name: c for c in wl.benchmark_cases()}
    assert len(cases) == 13
    c = cases["c1_512_bias_relu"]
    assert (c.M, c.N, c.K, c.epilogue, c.layout, c.seed) == (512, 512, 512, "BIAS_RELU", "KN", 0)
    assert [cases[f"c2_square_{n}"].flops for n in (4096, 8192)] == [2.0 * 4096 ** 3, 2.0 * 8192 ** 3]
    c = cases["c3_batched_128x512x512x1024"]
    assert (c.batch, c.M, c.N, c.K) == (128, 512, 512, 1024)
    c = cases["c3_splitk_256x256x131072"]
    assert (c.M, c.N, c.K, c.out) == (256, 256, 131072, "f32")
    c = cases["c5_gate_up_silu"]
    assert c.n_weight_cols == 28672 and c.N == 14336 and c.flops == 2.0 * 8192 * 28672 * 4096
    c = cases["c4_mlp_up_gelu"]
    # X + W + bias read once, Y written once
    assert c.algorithmic_bytes == 2 * (16384 * 768 + 768 * 3072 + 3072 + 16384 * 3072)


def test_inputs_are_reproducible_and_scaled():
    import torch

    c = wl.case_by_name("c2_square_4096")
    small = wl.Case("s", "gemm", 64, 48, 4096, seed=c.seed, x_scale=c.x_scale, w_scale=c.w_scale)
    a = wl.make_inputs(small)
    b = wl.make_inputs(small)
    assert torch.equal(a.X, b.X) and torch.equal(a.W, b.W)
    assert a.X.dtype == torch.bfloat16 and a.W.shape == (4096, 48)
    assert abs(float(a.X.float().std()) * 64.0 - 1.0) < 0.05  # N(0,1)/sqrt(4096)
