"""CPU pins for the FP64 oracle: each check fixes the oracle to something other
than its own formula -- a library routine, a closed form, exact integer or
rational arithmetic, a mathematical identity -- so that a dropped term, a
transposed operand or a wrong index fails at least one of them."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl

ALL_EPI = ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"]


def rand_bits(gen, shape, scale=1.0):
    t = (torch.randn(shape, generator=gen, dtype=torch.float32) * scale).to(torch.bfloat16)
    return wl.bits(t), t


def bits_of(a):
    """float array of exactly representable values -> BF16 bits."""
    t = torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    assert (t.float().numpy() == np.asarray(a, dtype=np.float32)).all()
    return wl.bits(t).copy()


def as_w(layout, w_kn_bits):
    return w_kn_bits if layout == "KN" else np.ascontiguousarray(np.swapaxes(w_kn_bits, -1, -2))


# ----------------------------------------------------------------- loop orders
@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("epi", ALL_EPI)
def test_blocked_is_bit_identical_to_triple_loop(layout, epi):
    g = torch.Generator().manual_seed(11)
    M, N, K = 21, 300, 523  # > one row block, > one column block, > two k chunks, all ragged
    Nw = 2 * N if epi == "SILU_GATE" else N
    xb, _ = rand_bits(g, (M, K))
    wb, _ = rand_bits(g, (K, Nw), 0.1)
    bias = rand_bits(g, (N,))[0] if epi in ("BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "BIAS_RESIDUAL") else None
    res = rand_bits(g, (M, N))[0] if epi == "BIAS_RESIDUAL" else None
    kw = dict(layout=layout, epilogue=epi, bias=bias, residual=res)
    a = oracle.linear(xb, as_w(layout, wb), variant="naive", **kw)
    b = oracle.linear(xb, as_w(layout, wb), variant="blocked", **kw)
    assert a.shape == (M, N)
    assert np.array_equal(a, b)
    # thread count must not matter
    c = oracle.linear(xb, as_w(layout, wb), variant="blocked", nthreads=1, **kw)
    assert np.array_equal(a, c)
    # row subsets pick the same values
    rows = np.array([20, 0, 7, 7, 13], dtype=np.int64)
    d = oracle.linear(xb, as_w(layout, wb), variant="blocked", rows=rows, **kw)
    assert np.array_equal(d, a[rows])


def test_batched_equals_per_slice_and_strided_inputs():
    g = torch.Generator().manual_seed(12)
    B, M, N, K = 3, 10, 17, 40
    big_x = rand_bits(g, (B, M, K + 8))[0]
    xb = big_x[:, :, :K]  # ld > width
    wb = rand_bits(g, (B, K, N))[0]
    y = oracle.linear(xb, wb)
    for b in range(B):
        yb = oracle.linear(np.ascontiguousarray(xb[b]), wb[b], variant="naive")
        assert np.array_equal(y[b], yb)


# ------------------------------------------------------------ library special case
@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_matches_library_dgemm(layout):
    g = torch.Generator().manual_seed(13)
    M, N, K = 67, 129, 1000
    xb, xt = rand_bits(g, (M, K))
    wb, wt = rand_bits(g, (K, N))
    ref = (xt.double() @ wt.double()).numpy()
    y = oracle.linear(xb, as_w(layout, wb), layout=layout)
    scale = (xt.double().abs() @ wt.double().abs()).numpy()
    assert (np.abs(y - ref) <= 1e-13 * scale + 1e-300).all()


# ------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_identity_returns_A(layout):
    g = torch.Generator().manual_seed(14)
    M, K = 37, 64
    xb, xt = rand_bits(g, (M, K))
    eye = bits_of(np.eye(K))
    y = oracle.linear(xb, as_w(layout, eye), layout=layout)
    assert np.array_equal(y, xt.double().numpy())


@pytest.mark.parametrize("K", [1, 512, 768, 3072, 4096, 14336, 131072])
def test_all_ones_gives_K(K):
    xb = bits_of(np.ones((3, K)))
    wb = bits_of(np.ones((K, 5)))
    y = oracle.linear(xb, wb)
    assert (y == float(K)).all()
    y = oracle.linear(xb, np.ascontiguousarray(wb.T), layout="NK", variant="naive" if K <= 4096 else "blocked")
    assert (y == float(K)).all()


@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_one_hot_and_positional_codes(layout):
    # non-square on purpose: a transposed operand or swapped index cannot pass
    M, N, K = 9, 14, 23
    A = np.zeros((M, K))
    B = np.zeros((K, N))
    A[4, 17] = 3.0
    B[17, 11] = -2.5
    y = oracle.linear(bits_of(A), as_w(layout, bits_of(B)), layout=layout)
    expect = np.zeros((M, N))
    expect[4, 11] = -7.5
    assert np.array_equal(y, expect)
    # A[i,k] = delta(k, k0) * (i+1), B[k0, j] = j+1  ->  C[i,j] = (i+1)(j+1)
    A = np.zeros((M, K))
    B = np.zeros((K, N))
    A[:, 5] = np.arange(1, M + 1)
    B[5, :] = np.arange(1, N + 1)
    y = oracle.linear(bits_of(A), as_w(layout, bits_of(B)), layout=layout)
    assert np.array_equal(y, np.outer(np.arange(1, M + 1), np.arange(1, N + 1)).astype(np.float64))


@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_small_integers_are_exact(layout):
    rng = np.random.default_rng(15)
    M, N, K = 33, 47, 2000
    A = rng.integers(-3, 4, size=(M, K))
    B = rng.integers(-3, 4, size=(K, N))
    y = oracle.linear(bits_of(A), as_w(layout, bits_of(B)), layout=layout)
    assert np.array_equal(y, (A.astype(np.int64) @ B.astype(np.int64)).astype(np.float64))


def test_exact_rational_brute_force():
    g = torch.Generator().manual_seed(16)
    M, N, K = 3, 4, 9
    xb, xt = rand_bits(g, (M, K))
    wb, wt = rand_bits(g, (K, N))
    y = oracle.linear(xb, wb, variant="naive")
    xs = [[Fraction(float(v)) for v in row] for row in xt.float().tolist()]
    ws = [[Fraction(float(v)) for v in row] for row in wt.float().tolist()]
    for m in range(M):
        for n in range(N):
            exact = sum(xs[m][k] * ws[k][n] for k in range(K))
            mag = sum(abs(xs[m][k] * ws[k][n]) for k in range(K))
            assert abs(Fraction(y[m, n]) - exact) <= Fraction(K, 2 ** 52) * mag


# ---------------------------------------------------------------------- epilogues
def _zero_product_inputs(M, N, K, epi):
    Nw = 2 * N if epi == "SILU_GATE" else N
    return bits_of(np.zeros((M, K))), bits_of(np.zeros((K, Nw)))


def test_bias_epilogues_against_library_functions():
    g = torch.Generator().manual_seed(17)
    M, N, K = 4, 200, 8
    bias_b, bias_t = rand_bits(g, (N,), 2.5)
    res_b, res_t = rand_bits(g, (M, N))
    x0, w0 = _zero_product_inputs(M, N, K, "BIAS")
    z = bias_t.double()
    lib = {
        "BIAS": z,
        "BIAS_RELU": torch.relu(z),
        "BIAS_GELU_TANH": torch.nn.functional.gelu(z, approximate="tanh"),
    }
    for epi, ref in lib.items():
        y = oracle.linear(x0, w0, epilogue=epi, bias=bias_b)
        assert np.allclose(y, np.broadcast_to(ref.numpy(), (M, N)), rtol=1e-14, atol=1e-300), epi
    y = oracle.linear(x0, w0, epilogue="BIAS_RESIDUAL", bias=bias_b, residual=res_b)
    assert np.array_equal(y, (z[None, :] + res_t.double()).numpy())
    y = oracle.linear(x0, w0, epilogue="BIAS_RESIDUAL", bias=None, residual=res_b)
    assert np.array_equal(y, res_t.double().numpy())


def test_bias_is_indexed_by_column_and_residual_by_row_and_column():
    M, N, K = 5, 7, 4
    x0, w0 = _zero_product_inputs(M, N, K, "BIAS")
    bias = bits_of(np.arange(N))
    y = oracle.linear(x0, w0, epilogue="BIAS", bias=bias)
    assert np.array_equal(y, np.broadcast_to(np.arange(N, dtype=np.float64), (M, N)))
    R = np.arange(M * N).reshape(M, N)
    y = oracle.linear(x0, w0, epilogue="BIAS_RESIDUAL", bias=bias, residual=bits_of(R))
    assert np.array_equal(y, R + np.arange(N)[None, :])


def test_gelu_tanh_identities_and_asymptotes():
    zs = np.linspace(-12, 12, 481)
    gz = np.array([oracle.gelu_tanh(z) for z in zs])
    gm = np.array([oracle.gelu_tanh(-z) for z in zs])
    # 0.5 z (1 + t) - 0.5 (-z)(1 - t) = z for any odd inner function t
    assert np.allclose(gz - gm, zs, rtol=0, atol=1e-14)
    assert oracle.gelu_tanh(0.0) == 0.0
    assert abs(oracle.gelu_tanh(12.0) - 12.0) < 1e-12
    assert abs(oracle.gelu_tanh(-12.0)) < 1e-12
    # the tanh form approximates the exact (erf) GELU to within 5e-4 everywhere
    exact = torch.nn.functional.gelu(torch.tensor(zs, dtype=torch.float64), approximate="none").numpy()
    assert np.abs(gz - exact).max() < 5e-4
    assert np.abs(gz - exact).max() > 1e-5  # ... and is not the erf form itself
    # library tanh form
    lib = torch.nn.functional.gelu(torch.tensor(zs, dtype=torch.float64), approximate="tanh").numpy()
    assert np.allclose(gz, lib, rtol=1e-14, atol=2e-15)  # 1 + tanh cancels in the negative tail


def test_silu_against_library_and_identities():
    gs = np.linspace(-30, 30, 601)
    s = np.array([oracle.silu(g) for g in gs])
    lib = torch.nn.functional.silu(torch.tensor(gs, dtype=torch.float64)).numpy()
    assert np.allclose(s, lib, rtol=1e-14, atol=1e-300)
    # silu(g) - silu(-g) = g
    assert np.allclose(s - s[::-1], gs, rtol=0, atol=1e-13)
    assert oracle.silu(0.0) == 0.0
    assert abs(oracle.silu(1.0) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16


@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_silu_gate_pairs_column_n_with_column_N_plus_n(layout):
    g = torch.Generator().manual_seed(18)
    M, N, K = 6, 10, 32
    xb, _ = rand_bits(g, (M, K))
    wb, _ = rand_bits(g, (K, 2 * N), 0.3)
    y = oracle.linear(xb, as_w(layout, wb), layout=layout, epilogue="SILU_GATE")
    both = oracle.linear(xb, as_w(layout, wb), layout=layout, epilogue="NONE")
    gate, up = both[:, :N], both[:, N:]
    ref = torch.nn.functional.silu(torch.tensor(gate)).numpy() * up
    assert y.shape == (M, N)
    assert np.allclose(y, ref, rtol=1e-13, atol=1e-300)
    # gate == 0  ->  0 whatever up is;  one-hot probe of the pairing
    A = np.zeros((M, K)); A[2, 3] = 1.0
    B = np.zeros((K, 2 * N)); B[3, 4] = 2.0; B[3, N + 4] = 3.0; B[3, N + 5] = 100.0
    y = oracle.linear(bits_of(A), as_w(layout, bits_of(B)), layout=layout, epilogue="SILU_GATE")
    expect = np.zeros((M, N)); expect[2, 4] = 2.0 / (1.0 + math.exp(-2.0)) * 3.0
    assert np.allclose(y, expect, rtol=1e-15, atol=0)


def test_relu_clamps_only_negative_sums():
    A = np.array([[1.0, 2.0]]); B = np.array([[1.0, -1.0], [1.0, -1.0]])
    y = oracle.linear(bits_of(A), bits_of(B), epilogue="BIAS_RELU", bias=bits_of(np.array([0.5, 0.5])))
    assert np.array_equal(y, np.array([[3.5, 0.0]]))


# ------------------------------------------------------------------ BF16 handling
def test_widening_and_rounding():
    allbits = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    t = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16)
    wide = oracle.bf16_to_f64(allbits)
    finite = np.isfinite(wide)
    assert np.array_equal(wide[finite], t.double().numpy()[finite])
    # every finite BF16 value rounds to itself
    for b in list(range(0, 1 << 16, 97)) + [0x0001, 0x007f, 0x0080, 0x7f7f, 0x8001, 0xff7f]:
        v = float(wide[b])
        if math.isfinite(v):
            assert oracle.round_bf16(v) == (b if v != 0 or b in (0, 0x8000) else b), hex(b)
    # ties go to even; a value just above the tie goes up although float32 would first pull it onto the tie
    assert oracle.round_bf16(1.0 + 2.0 ** -8) == 0x3F80
    assert oracle.round_bf16(1.0 + 2.0 ** -7 + 2.0 ** -8) == 0x3F82
    assert oracle.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81
    # library rounding on float32-representable values
    g = torch.Generator().manual_seed(19)
    v = torch.randn(2000, generator=g, dtype=torch.float32) * 37.0
    lib = wl.bits(v.to(torch.bfloat16))
    mine = np.array([oracle.round_bf16(float(x)) for x in v.tolist()], dtype=np.uint16)
    assert np.array_equal(lib, mine)


# ----------------------------------------------------------- the paper's accounting
def test_flop_accounting_matches_the_paper_printed_throughput():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_throughput_crosscheck.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for batch, M, N, K, ms, tflops in rows:
        case = wl.Case("x", "gemm", int(M), int(N), int(K), batch=int(batch))
        got = case.flops / (float(ms) * 1e-3) / 1e12
        assert abs(got - float(tflops)) / float(tflops) < 5e-3


def test_rejects_bad_arguments():
    x = bits_of(np.zeros((2, 4))); w = bits_of(np.zeros((4, 6)))
    with pytest.raises(ValueError):
        oracle.linear(x, w, epilogue="BIAS")  # missing bias
    with pytest.raises(ValueError):
        oracle.linear(x, w, epilogue="BIAS_RESIDUAL")  # missing residual
    with pytest.raises(ValueError):
        oracle.linear(x, w, rows=np.array([2]))  # row out of range
    assert oracle.linear(x[:0], w).shape == (0, 6)


def test_linear_grouped_is_the_per_group_product():
    """oracle.linear_grouped against numpy's FP64 matmul group by group (a library routine), with empty groups, and
    against oracle.linear when there is one group."""
    rng = np.random.default_rng(11)
    rows = [5, 0, 17, 1, 0, 9]
    M, N, K = sum(rows), 12, 40
    X = rng.integers(0x3C00, 0x4100, size=(M, K)).astype(np.uint16) | (rng.integers(0, 2, size=(M, K)).astype(np.uint16) << 15)
    W = rng.integers(0x3C00, 0x4100, size=(len(rows), N, K)).astype(np.uint16)
    bias = rng.integers(0x3C00, 0x4000, size=(N,)).astype(np.uint16)
    got = oracle.linear_grouped(X, W, rows, layout="NK", epilogue="BIAS", bias=bias)
    xf, wf, bf = oracle.bf16_to_f64(X), oracle.bf16_to_f64(W), oracle.bf16_to_f64(bias)
    r0 = 0
    for g, n in enumerate(rows):
        ref = xf[r0:r0 + n] @ wf[g].T + bf
        assert np.allclose(got[r0:r0 + n], ref, rtol=1e-13, atol=0)
        r0 += n
    one = oracle.linear_grouped(X, W[:1], [M], layout="NK")
    assert np.array_equal(one, oracle.linear(X, W[0], layout="NK"))
    kn = oracle.linear_grouped(X, np.ascontiguousarray(W.transpose(0, 2, 1)), rows, layout="KN", epilogue="BIAS", bias=bias)
    assert np.array_equal(kn, got)
    with pytest.raises(ValueError):
        oracle.linear_grouped(X, W, rows[:-1], layout="NK")


def test_linear_softmax_pins():
    """oracle.linear_softmax: rows sum to one, invariance under a shift of the bias, scipy's softmax of the same
    logits (a library routine), and the two-column closed form (a logistic function of the difference)."""
    from scipy.special import softmax as scipy_softmax

    rng = np.random.default_rng(12)
    M, N, K = 9, 21, 33
    X = rng.integers(0x3C00, 0x4080, size=(M, K)).astype(np.uint16) | (rng.integers(0, 2, size=(M, K)).astype(np.uint16) << 15)
    W = rng.integers(0x3A00, 0x3F80, size=(N, K)).astype(np.uint16) | (rng.integers(0, 2, size=(N, K)).astype(np.uint16) << 15)
    bias = rng.integers(0x3C00, 0x4000, size=(N,)).astype(np.uint16)
    Y = oracle.linear_softmax(X, W, layout="NK", bias=bias)
    assert np.allclose(Y.sum(axis=1), 1.0, rtol=0, atol=1e-14) and (Y > 0).all()
    logits = oracle.linear(X, W, layout="NK", epilogue="BIAS", bias=bias)
    assert np.allclose(Y, scipy_softmax(logits, axis=1), rtol=1e-13, atol=0)
    shifted = np.array([oracle.round_bf16(v + 2.0) for v in oracle.bf16_to_f64(bias)], dtype=np.uint16)
    if np.array_equal(oracle.bf16_to_f64(shifted), oracle.bf16_to_f64(bias) + 2.0):  # the shift is exact in BF16 here
        assert np.allclose(oracle.linear_softmax(X, W, layout="NK", bias=shifted), Y, rtol=1e-12, atol=0)
    two = oracle.linear_softmax(X, W[:2], layout="NK")
    z = oracle.linear(X, W[:2], layout="NK")
    assert np.allclose(two[:, 0], 1.0 / (1.0 + np.exp(z[:, 1] - z[:, 0])), rtol=1e-13, atol=0)
    one = oracle.linear_softmax(X, W[:1], layout="NK")
    assert np.array_equal(one, np.ones((M, 1)))
