"""CPU pins of the normalisation and whole-block oracle: library routines in float64, closed forms, invariances,
scalar-loop brute force."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import block as ob


def rnd(shape, seed, scale=1.0):
    g = np.random.default_rng(seed)
    return g.standard_normal(shape) * scale


def test_layer_norm_matches_library_and_loops():
    x, gamma, beta = rnd((5, 24), 1, 3.0) + 0.7, rnd((24,), 2), rnd((24,), 3)
    got = ob.layer_norm(x, gamma, beta, 1e-5)
    ref = F.layer_norm(torch.from_numpy(x), (24,), torch.from_numpy(gamma), torch.from_numpy(beta), 1e-5).numpy()
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)
    for m in range(5):  # the definition with scalar loops
        mean = sum(x[m]) / 24
        var = sum((v - mean) ** 2 for v in x[m]) / 24
        for c in range(24):
            want = (x[m, c] - mean) / math.sqrt(var + 1e-5) * gamma[c] + beta[c]
            assert abs(got[m, c] - want) <= 1e-12 * max(1.0, abs(want))


def test_layer_norm_closed_forms_and_invariances():
    x = rnd((4, 16), 4)
    ones, zeros = np.ones(16), np.zeros(16)
    y = ob.layer_norm(x, ones, zeros, 0.0)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-14) and np.allclose((y * y).mean(axis=1), 1, rtol=1e-12)
    # shift and positive scale of the input change nothing when eps = 0; a negative scale flips the sign
    assert np.allclose(ob.layer_norm(3.5 * x + 11.0, ones, zeros, 0.0), y, rtol=1e-11, atol=1e-12)
    assert np.allclose(ob.layer_norm(-2.0 * x, ones, zeros, 0.0), -y, rtol=1e-11, atol=1e-12)
    # a two-valued row: +-1 after normalisation
    row = np.array([[2.0, 6.0] * 8])
    assert np.allclose(ob.layer_norm(row, ones, zeros, 0.0), np.array([[-1.0, 1.0] * 8]), atol=1e-14)
    # eps dominates a constant row: output = beta
    beta = rnd((16,), 5)
    assert np.allclose(ob.layer_norm(np.full((2, 16), 4.25), ones, beta, 1e-5), np.broadcast_to(beta, (2, 16)))


def test_rms_norm_pins():
    x, gamma = rnd((6, 32), 6, 2.0), rnd((32,), 7)
    got = ob.rms_norm(x, gamma, 1e-6)
    ref = F.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(gamma), 1e-6).numpy()
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)
    y = ob.rms_norm(x, np.ones(32), 0.0)
    assert np.allclose((y * y).mean(axis=1), 1, rtol=1e-12)           # unit mean square
    assert np.allclose(ob.rms_norm(5.0 * x, np.ones(32), 0.0), y)     # scale invariance
    assert np.allclose(ob.rms_norm(np.full((1, 32), -3.0), gamma, 0.0), -gamma[None, :])  # constant row: sign * gamma
    for m in range(2):
        ms = sum(v * v for v in x[m]) / 32
        for c in range(32):
            want = x[m, c] / math.sqrt(ms + 1e-6) * gamma[c]
            assert abs(got[m, c] - want) <= 1e-12 * max(1.0, abs(want))


def test_activations():
    z = np.linspace(-6, 6, 41)
    assert np.allclose(ob.gelu_tanh(z), F.gelu(torch.from_numpy(z), approximate="tanh").numpy(), rtol=1e-12, atol=2e-15)
    assert np.allclose(ob.silu(z), F.silu(torch.from_numpy(z)).numpy(), rtol=1e-12, atol=1e-15)
    assert np.allclose(ob.gelu_tanh(z) - ob.gelu_tanh(-z), z, atol=1e-14)
    assert np.allclose(ob.silu(z) - ob.silu(-z), z, atol=1e-14)


def _weights(kind, C, Hq, Hkv, D, ffn, seed):
    g = np.random.default_rng(seed)
    qc = (Hq + 2 * Hkv) * D
    w = {"norm1_gamma": 1 + 0.1 * g.standard_normal(C), "norm2_gamma": 1 + 0.1 * g.standard_normal(C),
         "wqkv": 0.2 * g.standard_normal((qc, C)), "wo": 0.2 * g.standard_normal((C, C)),
         "w1": 0.2 * g.standard_normal(((2 if kind == "llama" else 1) * ffn, C)), "w2": 0.2 * g.standard_normal((C, ffn))}
    if kind == "gpt":
        w.update({"norm1_beta": 0.1 * g.standard_normal(C), "norm2_beta": 0.1 * g.standard_normal(C),
                  "bqkv": 0.1 * g.standard_normal(qc), "bo": 0.1 * g.standard_normal(C),
                  "b1": 0.1 * g.standard_normal(ffn), "b2": 0.1 * g.standard_normal(C)})
    return w


def _torch_block(kind, x, w, B, T, Hq, Hkv, D, eps):
    """The block as PyTorch eager would run it in float64 (library layer_norm / rms_norm / linear / SDPA / gelu)."""
    t = {k: torch.from_numpy(np.asarray(v)) for k, v in w.items()}
    x = torch.from_numpy(x)
    C = Hq * D
    norm = (lambda v, g, b: F.layer_norm(v, (C,), g, b, eps)) if kind == "gpt" else (lambda v, g, b: F.rms_norm(v, (C,), g, eps))
    n1 = norm(x, t["norm1_gamma"], t.get("norm1_beta"))
    qkv = F.linear(n1, t["wqkv"], t.get("bqkv")).view(B, T, Hq + 2 * Hkv, D)
    q, k, v = qkv[:, :, :Hq], qkv[:, :, Hq:Hq + Hkv], qkv[:, :, Hq + Hkv:]
    k, v = (u.repeat_interleave(Hq // Hkv, dim=2) for u in (k, v))  # what the paper's Llama wrapper does
    a = F.scaled_dot_product_attention(q.transpose(1, 2), k.transpose(1, 2), v.transpose(1, 2), is_causal=True)
    a = a.transpose(1, 2).reshape(B * T, C)
    x1 = F.linear(a, t["wo"], t.get("bo")) + x
    n2 = norm(x1, t["norm2_gamma"], t.get("norm2_beta"))
    if kind == "gpt":
        h = F.gelu(F.linear(n2, t["w1"], t["b1"]), approximate="tanh")
    else:
        gu = F.linear(n2, t["w1"])
        h = F.silu(gu[:, : gu.shape[1] // 2]) * gu[:, gu.shape[1] // 2:]
    return (F.linear(h, t["w2"], t.get("b2")) + x1).numpy()


def test_block_matches_the_library_chain():
    for kind, (B, T, Hq, Hkv, D, ffn) in (("gpt", (2, 7, 3, 3, 8, 40)), ("llama", (2, 9, 4, 2, 8, 24))):
        w = _weights(kind, Hq * D, Hq, Hkv, D, ffn, 11)
        x = rnd((B * T, Hq * D), 12)
        y, mid = ob.block_forward(kind, x, w, batch=B, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
        assert np.allclose(y, _torch_block(kind, x, w, B, T, Hq, Hkv, D, 1e-5), rtol=1e-11, atol=1e-12)
        assert mid["qkv"].shape == (B * T, (Hq + 2 * Hkv) * D) and mid["h"].shape == (B * T, ffn)


def test_block_special_cases():
    B, T, Hq, Hkv, D, ffn = 1, 6, 2, 1, 8, 16
    x = rnd((B * T, Hq * D), 13)
    w = _weights("llama", Hq * D, Hq, Hkv, D, ffn, 14)
    # zero output projections: both residual branches vanish, the block is the identity
    w0 = dict(w, wo=np.zeros_like(w["wo"]), w2=np.zeros_like(w["w2"]))
    y, _ = ob.block_forward("llama", x, w0, batch=B, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
    assert np.array_equal(y, x)
    # causality: the output at position i does not depend on later tokens
    y_full, _ = ob.block_forward("llama", x, w, batch=B, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
    x2 = x.copy()
    x2[4:] += 1.0
    y_pert, _ = ob.block_forward("llama", x2, w, batch=B, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
    assert np.allclose(y_full[:4], y_pert[:4], rtol=1e-12, atol=1e-13) and not np.allclose(y_full[4:], y_pert[4:])
    # batches are independent: two sequences in one call = two calls
    xb = rnd((2 * T, Hq * D), 15)
    yb, _ = ob.block_forward("llama", xb, w, batch=2, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
    for b in range(2):
        yi, _ = ob.block_forward("llama", xb[b * T:(b + 1) * T], w, batch=1, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D)
        assert np.allclose(yb[b * T:(b + 1) * T], yi, rtol=1e-12, atol=1e-13)
    # the `store` hook is applied to exactly the six stored intermediates
    seen = []
    ob.block_forward("llama", x, w, batch=B, seq=T, heads_q=Hq, heads_kv=Hkv, head_dim=D,
                     store=lambda t: (seen.append(t.shape), t)[1])
    assert len(seen) == 6
