"""FP64 CPU oracle for the row normalisations and the whole transformer block -- TEST INFRASTRUCTURE (see
oracle/__init__.py: only tests, the smoke check and the benchmark's CPU baseline may import this).

What it computes (Section 5.2: the two Level-3 blocks the paper composes from its attention pattern p1 and its
MLP pattern p2; the paper describes them as "a causal self-attention block paired with a two-layer MLP (expansion
to 3072, GELU, projection to 768)" and "a causal self-attention block with grouped-query attention paired with a
SwiGLU feed-forward network"; the surrounding normalisations and residual adds are those of a pre-norm block):

    n1  = norm1(x)                                  LayerNorm (GPT) or RMSNorm (Llama), over the hidden axis
    qkv = n1 @ Wqkv^T (+ bqkv)                      columns: Q heads | K heads | V heads
    a   = causal softmax(Q K^T / sqrt(d)) V         per batch and head, query head h -> key/value head h // group
    x1  = a @ Wo^T (+ bo) + x
    n2  = norm2(x1)
    h   = gelu_tanh(n2 @ W1^T + b1)                                  (GPT)
        = silu(n2 @ Wg^T) * (n2 @ Wu^T),  W1 = [Wg; Wu]              (Llama)
    y   = h @ W2^T (+ b2) + x1

Every step is the plain definition in float64 (numpy matmul is a step, not a reordering); nothing is rounded
between steps unless the caller passes `store`, a function applied to each stored intermediate (the tests use it
to round where the device stores BF16, which separates "the chain is wrong" from "BF16 storage moved a value").
"""
from __future__ import annotations

import numpy as np

from .attention import attention_f64


def layer_norm(x, gamma, beta, eps):
    """(x - mean) / sqrt(var + eps) * gamma + beta over the last axis, biased variance."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    y = (x - mean) / np.sqrt(var + eps) * np.asarray(gamma, dtype=np.float64)
    return y if beta is None else y + np.asarray(beta, dtype=np.float64)


def rms_norm(x, gamma, eps):
    """x / sqrt(mean(x^2) + eps) * gamma over the last axis."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * np.asarray(gamma, dtype=np.float64)


def gelu_tanh(z):
    z = np.asarray(z, dtype=np.float64)
    return 0.5 * z * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (z + 0.044715 * z ** 3)))


def silu(g):
    g = np.asarray(g, dtype=np.float64)
    return g / (1.0 + np.exp(-g))


def block_forward(kind, x, w, *, batch, seq, heads_q, heads_kv, head_dim, eps=1e-5, store=None):
    """x: float64 [batch * seq, hidden]; w: dict of float64 arrays named like fact_block_t's pointer fields
    (missing or None = absent).  Returns y float64 [batch * seq, hidden] and the dict of stored intermediates."""
    if kind not in ("gpt", "llama"):
        raise ValueError(kind)
    st = (lambda t: t) if store is None else store
    g = lambda name: None if w.get(name) is None else np.asarray(w[name], dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    hidden = heads_q * head_dim

    def norm(t, gamma, beta):
        return layer_norm(t, gamma, beta, eps) if kind == "gpt" else rms_norm(t, gamma, eps)

    def linear(t, weight, bias):
        y = t @ weight.T
        return y if bias is None else y + bias

    n1 = st(norm(x, g("norm1_gamma"), g("norm1_beta")))
    qkv = st(linear(n1, g("wqkv"), g("bqkv")))
    q = qkv[:, : hidden].reshape(batch, seq, heads_q, head_dim)
    k = qkv[:, hidden: hidden + heads_kv * head_dim].reshape(batch, seq, heads_kv, head_dim)
    v = qkv[:, hidden + heads_kv * head_dim:].reshape(batch, seq, heads_kv, head_dim)
    a = st(attention_f64(q, k, v, causal=True).reshape(batch * seq, hidden))
    x1 = st(linear(a, g("wo"), g("bo")) + x)
    n2 = st(norm(x1, g("norm2_gamma"), g("norm2_beta")))
    if kind == "gpt":
        h = st(gelu_tanh(linear(n2, g("w1"), g("b1"))))
    else:
        gu = linear(n2, g("w1"), None)
        ffn = gu.shape[1] // 2
        h = st(silu(gu[:, :ffn]) * gu[:, ffn:])
    y = linear(h, g("w2"), g("b2")) + x1
    return y, {"n1": n1, "qkv": qkv, "a": a, "x1": x1, "n2": n2, "h": h}
