"""Pins of the FP8 (E4M3) oracle against things other than itself: the values the 8-bit floating-point
format's definition fixes, a library conversion (torch.float8_e4m3fn), the BF16 oracle on the same values
(every E4M3 value is a BF16 value), and scalar brute force."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import fp8


def test_e4m3_values_the_format_fixes():
    v = fp8.e4m3_to_f64(np.arange(256, dtype=np.uint8))
    assert v[0x00] == 0.0 and v[0x80] == 0.0 and math.copysign(1.0, v[0x80]) == -1.0
    assert v[0x01] == 2.0 ** -9            # smallest subnormal
    assert v[0x07] == 7 * 2.0 ** -9        # largest subnormal
    assert v[0x08] == 2.0 ** -6            # smallest normal
    assert v[0x38] == 1.0 and v[0x39] == 1.125 and v[0x40] == 2.0 and v[0xC0] == -2.0
    assert v[0x7E] == 448.0 and v[0xFE] == -448.0   # largest magnitudes: there is no infinity
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF])
    pos = v[:0x7F]
    assert np.all(np.diff(pos) > 0), "positive codes are ordered like their values"
    assert np.array_equal(v[0x80:0xFF], -pos)


def test_e4m3_matches_the_library_conversion():
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float32).double().numpy()
    mine = fp8.e4m3_to_f64(codes.numpy())
    assert np.array_equal(np.isnan(lib), np.isnan(mine))
    ok = ~np.isnan(lib)
    assert np.array_equal(lib[ok], mine[ok])


def test_every_e4m3_value_is_a_bf16_value_and_the_bf16_oracle_agrees():
    rng = np.random.default_rng(5)
    codes = np.arange(256, dtype=np.uint8)
    codes = codes[(codes & 0x7F) != 0x7F]
    X = rng.choice(codes, size=(37, 96)).astype(np.uint8)
    W = rng.choice(codes, size=(23, 96)).astype(np.uint8)
    xb = np.array([[oracle.round_bf16(v) for v in row] for row in fp8.e4m3_to_f64(X)], dtype=np.uint16)
    wb = np.array([[oracle.round_bf16(v) for v in row] for row in fp8.e4m3_to_f64(W)], dtype=np.uint16)
    assert np.array_equal(oracle.bf16_to_f64(xb), fp8.e4m3_to_f64(X)), "E4M3 -> BF16 is exact"
    ref = oracle.linear(xb, wb, layout="NK", epilogue="NONE")
    got = fp8.linear_fp8(X, W)
    # both sum exact products in double, in possibly different orders
    assert np.allclose(got, ref, rtol=1e-13, atol=1e-9)
    bias = rng.standard_normal(23)
    bias_b = np.array([oracle.round_bf16(b) for b in bias], dtype=np.uint16)
    ref = oracle.linear(xb, wb, layout="NK", epilogue="BIAS_GELU_TANH", bias=bias_b)
    got = fp8.linear_fp8(X, W, 1.0, oracle.bf16_to_f64(bias_b), "BIAS_GELU_TANH")
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-9)


@pytest.mark.parametrize("epilogue", ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH"])
def test_linear_fp8_against_scalar_loops(epilogue):
    rng = np.random.default_rng(6)
    M, N, K = 5, 4, 19
    X = rng.integers(0, 0x7F, size=(M, K)).astype(np.uint8) | (rng.integers(0, 2, size=(M, K)).astype(np.uint8) << 7)
    W = rng.integers(0, 0x7F, size=(N, K)).astype(np.uint8) | (rng.integers(0, 2, size=(N, K)).astype(np.uint8) << 7)
    scale = 0.03125 * 1.7
    bias = None if epilogue == "NONE" else rng.standard_normal(N)
    got = fp8.linear_fp8(X, W, scale, bias, epilogue)
    table = fp8.e4m3_to_f64(np.arange(256, dtype=np.uint8))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(table[X[m, k]]) * float(table[W[n, k]])
            z = scale * acc + (0.0 if bias is None else float(bias[n]))
            if epilogue == "BIAS_RELU":
                z = max(z, 0.0)
            if epilogue == "BIAS_GELU_TANH":
                z = 0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))
            assert got[m, n] == pytest.approx(z, rel=1e-12, abs=1e-12)


def test_linear_fp8_special_cases():
    one = np.full((3, 8), 0x38, dtype=np.uint8)   # all ones: every output is K
    assert np.array_equal(fp8.linear_fp8(one, one[:2]), np.full((3, 2), 8.0))
    assert np.array_equal(fp8.linear_fp8(one, one[:2], scale=0.5), np.full((3, 2), 4.0))
    big = np.full((1, 4), 0x7E, dtype=np.uint8)   # 448 * 448 * 4
    assert fp8.linear_fp8(big, big)[0, 0] == 448.0 * 448.0 * 4
    rows = fp8.linear_fp8(np.arange(40, dtype=np.uint8).reshape(5, 8), one[:2], rows=[4, 0])
    full = fp8.linear_fp8(np.arange(40, dtype=np.uint8).reshape(5, 8), one[:2])
    assert np.array_equal(rows, full[[4, 0]])
    with pytest.raises(ValueError):
        fp8.linear_fp8(one, one, bias=np.zeros(3))
    with pytest.raises(ValueError):
        fp8.linear_fp8(one, one, epilogue="BIAS")
