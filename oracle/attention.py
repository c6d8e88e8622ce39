"""FP64 CPU oracle for fused multi-head attention -- TEST INFRASTRUCTURE (see oracle/__init__.py).

What it computes (the paper's pattern p1 of Section 5.2: causal fused multi-head attention for the MiniGPT
block; grouped-query attention with 32 query heads over 8 key/value heads for the Llama block, where the paper
expands K/V with repeat_interleave before its kernel):

    for every batch b, query head h, query position i:
        kv = h // (heads_q // heads_kv)                      (query heads share key/value heads in order)
        s_j = scale * <Q[b,i,h,:], K[b,j,kv,:]>              for the allowed key positions j
        p   = softmax_j(s)                                   (allowed: all j, or j <= i when causal)
        O[b,i,h,:] = sum_j p_j V[b,j,kv,:]

written out as that definition: the scores of one (b, h) as a matrix product in float64 (a library matmul is a
step, not a reordering), the row-wise softmax with the row maximum subtracted, the weighted sum as a second
product.  Inputs are BF16 bit patterns widened exactly; the result is float64.  No tiling, no online softmax.
"""
from __future__ import annotations

import numpy as np


def _widen(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits)
    if b.dtype != np.uint16:
        raise TypeError("expected BF16 bit patterns as uint16")
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def attention(Q, K, V, *, causal: bool, scale: float | None = None, rows=None) -> np.ndarray:
    """Q: uint16 [B, Tq, Hq, D];  K, V: uint16 [B, Tk, Hkv, D];  returns float64 [B, Tq (or len(rows)), Hq, D].
    `rows`: optional query positions to compute (all batches and heads)."""
    return attention_f64(_widen(Q), _widen(K), _widen(V), causal=causal, scale=scale, rows=rows)


def attention_f64(q, k, v, *, causal: bool, scale: float | None = None, rows=None) -> np.ndarray:
    """The same definition on float64 operands (used where attention is one stage of a longer float64 chain)."""
    q, k, v = (np.asarray(t, dtype=np.float64) for t in (q, k, v))
    B, Tq, Hq, D = q.shape
    Bk, Tk, Hkv, Dk = k.shape
    if (Bk, Dk) != (B, D) or v.shape != k.shape or Hq % Hkv:
        raise ValueError("inconsistent attention shapes")
    if causal and Tq != Tk:
        raise ValueError("causal attention is defined here for Tq == Tk")
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    idx = np.arange(Tq) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.empty((B, len(idx), Hq, D), dtype=np.float64)
    group = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            kv = h // group
            s = scale * (q[b, idx, h, :] @ k[b, :, kv, :].T)  # [rows, Tk]
            if causal:
                s = np.where(np.arange(Tk)[None, :] <= idx[:, None], s, -np.inf)
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            out[b, :, h, :] = p @ v[b, :, kv, :]
    return out
