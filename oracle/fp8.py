"""FP64 CPU oracle for the FP8 (E4M3) fused linear layer -- TEST INFRASTRUCTURE (see oracle/__init__.py).

What it computes: ``Y = epilogue(scale * (X @ W^T) + bias)`` where X [M, K] and W [N, K] are FP8 E4M3 codes
(one byte per element), every product and sum is taken in double, and the epilogue is the one of the BF16
linear layers (Section 5.2's pattern p2).  The paper lists an FP8 GEMM among the kernels its pattern registry
holds (Table 1, Level 1); it fixes no scaling convention, so the usual one is taken: one FP32 scale for the
whole product (the product of the operands' per-tensor scales), applied to the accumulator before the bias.

E4M3 (the "fn" variant of the OCP 8-bit floating-point specification): 1 sign bit, 4 exponent bits with
bias 7, 3 mantissa bits; exponent 0 holds subnormals m/8 * 2^-6; there are no infinities, and the all-ones
pattern S.1111.111 is NaN, so the largest magnitude is 1.75 * 2^8 = 448.
"""
from __future__ import annotations

import numpy as np


def e4m3_to_f64(codes) -> np.ndarray:
    """Exact value of every E4M3 code, written out from the format's definition."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    subnormal = (m / 8.0) * 2.0 ** -6
    v = sign * np.where(e == 0, subnormal, normal)
    return np.where((e == 15) & (m == 7), np.nan, v)


def gelu_tanh(z: np.ndarray) -> np.ndarray:
    """0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))  (Section 5.2, MiniGPT pattern p2)."""
    return 0.5 * z * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (z + 0.044715 * z ** 3)))


def linear_fp8(X, W, scale: float = 1.0, bias=None, epilogue: str = "NONE", rows=None) -> np.ndarray:
    """``epilogue(scale * X @ W^T + bias)`` in FP64.

    X : uint8 E4M3 codes [M, K];  W : uint8 E4M3 codes [N, K] (nn.Linear weight).
    bias : float64-convertible [N] or None (required by the BIAS* epilogues).
    epilogue : "NONE" | "BIAS" | "BIAS_RELU" | "BIAS_GELU_TANH".
    rows : optional row indices; only those output rows are computed.
    """
    x = e4m3_to_f64(X)
    w = e4m3_to_f64(W)
    if rows is not None:
        x = x[np.asarray(rows, dtype=np.int64)]
    acc = x @ w.T  # FP64 matmul: products of E4M3 values are exact, sums are rounded at 2^-53
    z = float(scale) * acc
    if epilogue == "NONE":
        if bias is not None:
            raise ValueError("NONE takes no bias")
        return z
    if bias is None:
        raise ValueError(f"{epilogue} needs a bias")
    z = z + np.asarray(bias, dtype=np.float64)[None, :]
    if epilogue == "BIAS":
        return z
    if epilogue == "BIAS_RELU":
        return np.maximum(z, 0.0)
    if epilogue == "BIAS_GELU_TANH":
        return gelu_tanh(z)
    raise ValueError(f"unknown epilogue {epilogue}")
