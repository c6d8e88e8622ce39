"""CPU pins of the oracle for a row normalisation between two linear layers (oracle/normfold.py): closed forms,
special cases that reduce to the independent C oracle of the linear layer or to a library routine, scalar loops,
and the algebraic identity that a kernel folding the normalisation into the weights relies on."""
import math

import numpy as np
import torch
import torch.nn.functional as F

import oracle
from oracle import normfold as nf


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Nearest-even BF16 bit patterns of float64 values, through torch's conversion (a library routine)."""
    return torch.from_numpy(np.asarray(a, dtype=np.float64)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def rnd_bits(shape, seed, scale=1.0, shift=0.0):
    g = np.random.default_rng(seed)
    return bf16_bits(g.standard_normal(shape) * scale + shift)


def test_row_stats_closed_form_and_totals():
    # a ramp 0, 1, ..., C-1 in every row (exact in BF16 below 256): chunk c holds 64c .. 64c+63
    C = 200
    x = bf16_bits(np.tile(np.arange(C, dtype=np.float64), (3, 1)))
    s = nf.row_stats(x)
    assert s.shape == (4, 3, 2)
    for c in range(4):
        lo, hi = 64 * c, min(64 * c + 64, C)
        n = hi - lo
        assert np.all(s[c, :, 0] == n * (lo + hi - 1) / 2)
        assert np.all(s[c, :, 1] == sum(v * v for v in range(lo, hi)))
    # the chunks add up to whole-row sums taken another way
    xb = rnd_bits((7, 333), 1, 2.0, 0.3)
    s = nf.row_stats(xb)
    xf = oracle.bf16_to_f64(xb)
    assert np.allclose(s[:, :, 0].sum(axis=0), xf @ np.ones(333), rtol=1e-13, atol=1e-12)
    assert np.allclose(s[:, :, 1].sum(axis=0), np.einsum("mc,mc->m", xf, xf), rtol=1e-13)
    # scalar loop on one entry
    assert abs(s[2, 5, 1] - math.fsum(float(v) ** 2 for v in xf[5, 128:192])) < 1e-12


def test_constant_rows_give_the_shift_only():
    # a constant row has zero variance: with eps > 0 its LayerNorm is exactly beta, so y = beta @ W^T + b
    M, K, N = 4, 64, 24
    x = bf16_bits(np.tile(np.array([[1.5], [-2.0], [0.0], [3.0]]), (1, K)))
    w, gamma, beta, bias = rnd_bits((N, K), 2), rnd_bits((K,), 3), rnd_bits((K,), 4), rnd_bits((N,), 5)
    y = nf.norm_linear(x, w, gamma, kind="layer", eps=1e-5, beta_bits=beta, bias_bits=bias, epilogue="BIAS")
    want = oracle.bf16_to_f64(w) @ oracle.bf16_to_f64(beta) + oracle.bf16_to_f64(bias)
    assert np.allclose(y, np.tile(want, (M, 1)), rtol=1e-13, atol=1e-13)


def test_already_normalised_rows_reduce_to_the_linear_oracle():
    # rows of +-1 (mean 0, variance 1), gamma = 1, beta = 0, eps = 0: the normalisation is the identity, and the
    # result must equal the C oracle of the plain linear layer (separate code) for every epilogue
    M, K, N = 6, 128, 32
    g = np.random.default_rng(6)
    signs = np.where(g.random((M, K // 2)) < 0.5, -1.0, 1.0)
    x = bf16_bits(np.concatenate([signs, -signs], axis=1))  # every row sums to zero
    ones = bf16_bits(np.ones(K))
    w, bias, res = rnd_bits((N, K), 7, 0.1), rnd_bits((N,), 8), rnd_bits((M, N), 9)
    for kind in ("layer", "rms"):
        for epi, kw, okw in (
            ("NONE", {}, {}),
            ("BIAS", {"bias_bits": bias}, {"bias": bias}),
            ("BIAS_RELU", {"bias_bits": bias}, {"bias": bias}),
            ("BIAS_GELU_TANH", {"bias_bits": bias}, {"bias": bias}),
            ("BIAS_RESIDUAL", {"bias_bits": bias, "residual_bits": res}, {"bias": bias, "residual": res}),
        ):
            got = nf.norm_linear(x, w, ones, kind=kind, eps=0.0, epilogue=epi, **kw)
            want = oracle.linear(x, w, layout="NK", epilogue=epi, **okw)
            assert np.allclose(got, want, rtol=1e-12, atol=1e-12), (kind, epi)
    wg = rnd_bits((2 * N, K), 10, 0.1)
    got = nf.norm_linear(x, wg, ones, kind="rms", eps=0.0, epilogue="SILU_GATE")
    assert np.allclose(got, oracle.linear(x, wg, layout="NK", epilogue="SILU_GATE"), rtol=1e-12, atol=1e-12)


def test_matches_library_norm_then_matmul_and_scalar_loops():
    M, K, N = 5, 96, 16
    x, w = rnd_bits((M, K), 11, 1.5, 0.4), rnd_bits((N, K), 12, 0.2)
    gamma, beta, bias = rnd_bits((K,), 13, 0.5, 1.0), rnd_bits((K,), 14, 0.3), rnd_bits((N,), 15)
    xf, wf = (torch.from_numpy(oracle.bf16_to_f64(t)) for t in (x, w))
    gf, bf, cf = (torch.from_numpy(oracle.bf16_to_f64(t)) for t in (gamma, beta, bias))
    got = nf.norm_linear(x, w, gamma, kind="layer", eps=1e-5, beta_bits=beta, bias_bits=bias, epilogue="BIAS")
    ref = F.linear(F.layer_norm(xf, (K,), gf, bf, 1e-5), wf, cf).numpy()
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)
    got_r = nf.norm_linear(x, w, gamma, kind="rms", eps=1e-6, epilogue="NONE")
    ref_r = F.linear(xf / torch.sqrt((xf * xf).mean(dim=1, keepdim=True) + 1e-6) * gf, wf).numpy()
    assert np.allclose(got_r, ref_r, rtol=1e-12, atol=1e-12)
    # one output by scalar loops
    m, n = 3, 7
    row = [float(v) for v in xf[m]]
    mean = math.fsum(row) / K
    var = math.fsum((v - mean) ** 2 for v in row) / K
    acc = math.fsum(((row[k] - mean) / math.sqrt(var + 1e-5) * float(gf[k]) + float(bf[k])) * float(wf[n, k])
                    for k in range(K)) + float(cf[n])
    assert abs(got[m, n] - acc) < 1e-12


def test_invariances():
    M, K, N = 4, 64, 8
    x, w, gamma = rnd_bits((M, K), 16), rnd_bits((N, K), 17), rnd_bits((K,), 18)
    base = nf.norm_linear(x, w, gamma, kind="layer", eps=0.0)
    x4 = bf16_bits(4.0 * oracle.bf16_to_f64(x))  # a power of two: exact in BF16
    assert np.allclose(nf.norm_linear(x4, w, gamma, kind="layer", eps=0.0), base, rtol=1e-11, atol=1e-12)
    assert np.allclose(nf.norm_linear(x4, w, gamma, kind="rms", eps=0.0),
                       nf.norm_linear(x, w, gamma, kind="rms", eps=0.0), rtol=1e-11, atol=1e-12)
    # permuting the hidden axis of x, gamma and W together changes nothing
    perm = np.random.default_rng(19).permutation(K)
    assert np.allclose(nf.norm_linear(np.ascontiguousarray(x[:, perm]), np.ascontiguousarray(w[:, perm]),
                                      np.ascontiguousarray(gamma[perm]), kind="layer", eps=0.0), base,
                       rtol=1e-11, atol=1e-12)


def test_fold_definitions_and_the_folded_identity():
    M, K, N = 9, 192, 40
    x, w = rnd_bits((M, K), 20, 1.0, 0.5), rnd_bits((N, K), 21, 0.1)
    gamma, beta, bias = rnd_bits((K,), 22, 0.2, 1.0), rnd_bits((K,), 23, 0.1), rnd_bits((N,), 24)
    prod, shift = nf.fold_norm(w, gamma, beta, bias)
    wf, gf = oracle.bf16_to_f64(w), oracle.bf16_to_f64(gamma)
    for n, k in ((0, 0), (5, 17), (39, 191)):
        assert prod[n, k] == wf[n, k] * gf[k]
        # the product of two BF16 values has at most 16 significant bits: rounding it once, by the C oracle's
        # scalar routine, equals the library's conversion
        assert oracle.round_bf16(prod[n, k]) == int(bf16_bits(np.array([prod[n, k]]))[0])
    assert abs(shift[3] - (math.fsum(float(wf[3, k]) * float(oracle.bf16_to_f64(beta)[k]) for k in range(K)) +
                           float(oracle.bf16_to_f64(bias)[3]))) < 1e-12
    assert nf.fold_norm(w, gamma)[1] is None
    # the identity behind folding: with S1, S2 the row sums, mean = S1 / K, rstd = 1 / sqrt(S2 / K - mean^2 + eps),
    #   norm(x) @ W^T + b = rstd * (x @ P^T) - rstd * mean * rowsum(P) + shift
    stats = nf.row_stats(x)
    s1, s2 = stats[:, :, 0].sum(axis=0), stats[:, :, 1].sum(axis=0)
    xf = oracle.bf16_to_f64(x)
    for kind, eps in (("layer", 1e-5), ("rms", 1e-6)):
        mean = s1 / K if kind == "layer" else np.zeros(M)
        rstd = 1.0 / np.sqrt(s2 / K - mean * mean + eps)
        if kind == "layer":
            folded = rstd[:, None] * (xf @ prod.T) - (rstd * mean)[:, None] * prod.sum(axis=1)[None, :] + shift[None, :]
            want = nf.norm_linear(x, w, gamma, kind="layer", eps=eps, beta_bits=beta, bias_bits=bias, epilogue="BIAS")
        else:
            folded = rstd[:, None] * (xf @ prod.T)
            want = nf.norm_linear(x, w, gamma, kind="rms", eps=eps)
        assert np.allclose(folded, want, rtol=1e-10, atol=1e-11), kind
