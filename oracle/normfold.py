"""FP64 CPU oracle for a row normalisation between two linear layers -- TEST INFRASTRUCTURE (see
oracle/__init__.py: only tests, the smoke check and the benchmark's CPU baseline may import this).

The paper's Table 1 lists "GEMM-LayerNorm-GEMM fusion" among the Level-2 kernels of its registry, and the blocks of
Section 5.2 have a normalisation between the attention output projection and the MLP.  What such a fusion computes
has a plain definition, and that definition is what stands here: normalise every row of the activations over the
hidden axis, then apply the linear layer and its epilogue,

    n = (x - mean(x)) / sqrt(var(x) + eps) * gamma + beta        LayerNorm, biased variance
    n =  x / sqrt(mean(x^2) + eps) * gamma                        RMSNorm
    y = epilogue(n @ W^T + b)

in float64 with nothing rounded in between.  Whatever algebra a device kernel uses to avoid the separate pass
(folding gamma into W, correcting the accumulator per row) is the kernel's business and is NOT done here.

Also here, as definitions: the partial row sums a producing layer leaves for the normalisation (`row_stats`), and the
folded weights (`fold_norm`: the element-wise products, their row sums, the shift moved into the bias).
"""
from __future__ import annotations

import numpy as np

from . import bf16_to_f64
from .block import gelu_tanh, layer_norm, rms_norm, silu


def row_stats(x_bits) -> np.ndarray:
    """x_bits: uint16 BF16 bits [M, C].  Returns float64 [ceil(C / 64), M, 2]: for every row and every chunk of 64
    consecutive columns (the last one may be short), the sum and the sum of squares of the chunk's values."""
    x = bf16_to_f64(np.asarray(x_bits))
    M, C = x.shape
    chunks = (C + 63) // 64
    out = np.zeros((chunks, M, 2), dtype=np.float64)
    for c in range(chunks):
        part = x[:, 64 * c:64 * c + 64]
        out[c, :, 0] = part.sum(axis=1)
        out[c, :, 1] = (part * part).sum(axis=1)
    return out


def norm_linear(x_bits, w_bits, gamma_bits, *, kind, eps, beta_bits=None, bias_bits=None, residual_bits=None,
                epilogue="NONE") -> np.ndarray:
    """epilogue(norm(x) @ W^T + b), the definition.  x: [M, K]; W: [Nw, K] (nn.Linear weight; for SILU_GATE the
    gate rows first, then the up rows, Nw = 2 N_out); gamma, beta: [K]; bias: [N_out]; residual: [M, N_out].
    kind: "layer" or "rms" (beta must be None for "rms").  Returns float64 [M, N_out]."""
    x = bf16_to_f64(np.asarray(x_bits))
    w = bf16_to_f64(np.asarray(w_bits))
    gamma = bf16_to_f64(np.asarray(gamma_bits))
    beta = None if beta_bits is None else bf16_to_f64(np.asarray(beta_bits))
    if kind == "layer":
        n = layer_norm(x, gamma, beta, eps)
    elif kind == "rms":
        if beta is not None:
            raise ValueError("an RMS norm has no shift")
        n = rms_norm(x, gamma, eps)
    else:
        raise ValueError(kind)
    z = n @ w.T
    if epilogue == "SILU_GATE":
        half = w.shape[0] // 2
        return silu(z[:, :half]) * z[:, half:]
    if bias_bits is not None:
        z = z + bf16_to_f64(np.asarray(bias_bits))
    if epilogue in ("NONE", "BIAS"):
        return z
    if epilogue == "BIAS_RELU":
        return np.maximum(z, 0.0)
    if epilogue == "BIAS_GELU_TANH":
        return gelu_tanh(z)
    if epilogue == "BIAS_RESIDUAL":
        return z + bf16_to_f64(np.asarray(residual_bits))
    raise ValueError(epilogue)


def fold_norm(w_bits, gamma_bits, beta_bits=None, bias_bits=None):
    """The folded weights, as definitions: P[n, k] = gamma[k] * W[n, k] (exact in float64: two 8-bit significands),
    and the shifted bias b[n] + sum_k beta[k] W[n, k] (None without beta).  Returns (P float64 [Nw, K], shifted bias
    float64 [Nw] or None).  Rounding P to BF16 and summing its rows is left to the caller: those are statements about
    a storage format, not part of the definition."""
    w = bf16_to_f64(np.asarray(w_bits))
    gamma = bf16_to_f64(np.asarray(gamma_bits))
    prod = w * gamma[None, :]
    if beta_bits is None:
        return prod, None
    shift = w @ bf16_to_f64(np.asarray(beta_bits))
    if bias_bits is not None:
        shift = shift + bf16_to_f64(np.asarray(bias_bits))
    return prod, shift
