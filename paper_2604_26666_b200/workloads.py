"""Seeded synthetic inputs and the shape table of the benchmark configurations.

This module holds NO arithmetic of the method (no product, no epilogue): it
only names shapes and draws random BF16 tensors on the CPU.  Both the CUDA
path and the CPU oracle are fed from here, so that they see the same bits.

The shapes stand in for the workloads of the paper's evaluation (Section 5.1
"Benchmark problems": square, batched and large-K matrix products; Section 5.2:
the linear layers of the MiniGPT block and of the Llama-3-8B decoder block),
at the sizes and value distributions the benchmark configurations state.
None of the original benchmark files or model weights is used.

Recipe (identical for every case): draw FP32 values from a
``torch.Generator(device="cpu")`` seeded with the case's seed, in the order
X/A, W/B, bias, residual; scale in FP32; round once to BF16 (nearest even).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import torch


@dataclass(frozen=True)
class Case:
    """One GEMM-family problem.  ``N`` is the number of OUTPUT columns; the
    weight has ``2 * N`` columns for SILU_GATE (gate first, then up)."""

    name: str
    op: str  # "gemm" | "gemm_batched" | "gemm_splitk" | "linear"
    M: int
    N: int
    K: int
    batch: int = 1
    epilogue: str = "NONE"
    layout: str = "KN"  # "KN": B[K x N] (torch.matmul);  "NK": W[N x K] (nn.Linear.weight)
    out: str = "bf16"  # "bf16" | "f32"
    has_bias: bool = False
    has_residual: bool = False
    seed: int = 0
    x_dist: str = "normal"  # "normal" | "uniform"  (uniform = U(-1, 1))
    w_dist: str = "normal"
    x_scale: float = 1.0
    w_scale: float = 1.0
    config: int = 0  # 1-based index of the benchmark configuration this case belongs to

    @property
    def n_weight_cols(self) -> int:
        return 2 * self.N if self.epilogue == "SILU_GATE" else self.N

    @property
    def flops(self) -> float:
        """2 * batch * M * (weight columns) * K -- the accounting of the paper's
        Section 5.2 throughput figures (epilogue work is not counted)."""
        return 2.0 * self.batch * self.M * self.n_weight_cols * self.K

    @property
    def out_bytes_per_elem(self) -> int:
        return 4 if self.out == "f32" else 2

    @property
    def algorithmic_bytes(self) -> float:
        """Each operand read once plus the output written once."""
        b = self.batch * (self.M * self.K + self.K * self.n_weight_cols) * 2
        b += self.batch * self.M * self.N * self.out_bytes_per_elem
        if self.has_bias:
            b += self.N * 2
        if self.has_residual:
            b += self.batch * self.M * self.N * 2
        return float(b)


def _k_inv_sqrt(k: int) -> float:
    return float(k) ** -0.5


def benchmark_cases(layout_linear: str = "NK") -> list[Case]:
    """The thirteen shapes of the five benchmark configurations."""
    c: list[Case] = []
    # config 1: C = ReLU(A.B + bias), 512^3, U(-1,1) operands, N(0,1) bias, seed 0
    c.append(Case("c1_512_bias_relu", "linear", 512, 512, 512, epilogue="BIAS_RELU", layout="KN",
                  has_bias=True, seed=0, x_dist="uniform", w_dist="uniform", config=1))
    # config 2: square GEMMs, operands N(0,1)/sqrt(K), seed 1
    for n in (4096, 8192):
        c.append(Case(f"c2_square_{n}", "gemm", n, n, n, layout="KN", seed=1,
                      x_scale=_k_inv_sqrt(n), w_scale=_k_inv_sqrt(n), config=2))
    # config 3: batched GEMM + large-K FP32-output split-K GEMM, seed 2
    c.append(Case("c3_batched_128x512x512x1024", "gemm_batched", 512, 512, 1024, batch=128, layout="KN",
                  seed=2, config=3))
    c.append(Case("c3_splitk_256x256x131072", "gemm_splitk", 256, 256, 131072, layout="KN", out="f32",
                  seed=2, x_dist="uniform", w_dist="uniform", config=3))
    # config 4: GPT-style block linears, 16384 tokens, d_model 768, MLP 3072, seed 3
    L = layout_linear
    c.append(Case("c4_qkv", "linear", 16384, 2304, 768, epilogue="BIAS", layout=L, has_bias=True,
                  seed=3, w_scale=0.02, config=4))
    c.append(Case("c4_out_proj", "linear", 16384, 768, 768, epilogue="BIAS_RESIDUAL", layout=L,
                  has_bias=True, has_residual=True, seed=3, w_scale=0.02, config=4))
    c.append(Case("c4_mlp_up_gelu", "linear", 16384, 3072, 768, epilogue="BIAS_GELU_TANH", layout=L,
                  has_bias=True, seed=3, w_scale=0.02, config=4))
    c.append(Case("c4_mlp_down", "linear", 16384, 768, 3072, epilogue="BIAS_RESIDUAL", layout=L,
                  has_bias=True, has_residual=True, seed=3, w_scale=0.02, config=4))
    # config 5: Llama-3-8B-shaped linears, 8192 tokens, hidden 4096, MLP 14336, seed 4
    c.append(Case("c5_qkv", "linear", 8192, 6144, 4096, epilogue="NONE", layout=L, seed=4,
                  w_scale=0.02, config=5))
    c.append(Case("c5_o_proj", "linear", 8192, 4096, 4096, epilogue="BIAS_RESIDUAL", layout=L,
                  has_residual=True, seed=4, w_scale=0.02, config=5))
    c.append(Case("c5_gate_up_silu", "linear", 8192, 14336, 4096, epilogue="SILU_GATE", layout=L,
                  seed=4, w_scale=0.02, config=5))
    c.append(Case("c5_down", "linear", 8192, 4096, 14336, epilogue="BIAS_RESIDUAL", layout=L,
                  has_residual=True, seed=4, w_scale=0.02, config=5))
    return c


def paper_cases() -> list[Case]:
    """The paper's own Level-1 shapes where they differ from the benchmark configurations (Section 5.1): Problem 3,
    a batch of 128 products 512 x 1024 . 1024 x 2048, and Problem 6, 256 x 524288 . 524288 x 256 with FP32 output.
    (Problem 1, 4096^3, is configuration 2.)  config = 0 marks them as extras."""
    return [Case("p3_batched_128x512x2048x1024", "gemm_batched", 512, 2048, 1024, batch=128, layout="KN", seed=12,
                 config=0),
            Case("p6_splitk_256x256x524288", "gemm_splitk", 256, 256, 524288, layout="KN", out="f32", seed=16,
                 x_dist="uniform", w_dist="uniform", config=0)]


def case_by_name(name: str, layout_linear: str = "NK") -> Case:
    for cs in benchmark_cases(layout_linear) + paper_cases():
        if cs.name == name:
            return cs
    raise KeyError(name)


def _draw(gen: torch.Generator, shape, dist: str, scale: float) -> torch.Tensor:
    if dist == "normal":
        t = torch.randn(shape, generator=gen, dtype=torch.float32)
    elif dist == "uniform":
        t = torch.rand(shape, generator=gen, dtype=torch.float32) * 2.0 - 1.0
    else:
        raise ValueError(dist)
    if scale != 1.0:
        t = t * scale
    return t.to(torch.bfloat16)


@dataclass
class Inputs:
    X: torch.Tensor  # bf16 [M,K] or [batch,M,K]
    W: torch.Tensor  # bf16 [K,Nw] / [Nw,K] (or batched)
    bias: Optional[torch.Tensor] = None  # bf16 [N]
    residual: Optional[torch.Tensor] = None  # bf16 [M,N] (or batched)
    extra: dict = field(default_factory=dict)


def make_inputs(case: Case, gen: Optional[torch.Generator] = None, pin: bool = False) -> Inputs:
    """Draw the case's inputs on the CPU (BF16).  ``gen`` lets a caller continue
    one generator across the cases of a configuration; by default a fresh
    generator seeded with ``case.seed`` is used."""
    if gen is None:
        gen = torch.Generator(device="cpu")
        gen.manual_seed(case.seed)
    b = (case.batch,) if case.batch > 1 else ()
    Nw = case.n_weight_cols
    X = _draw(gen, b + (case.M, case.K), case.x_dist, case.x_scale)
    wshape = (case.K, Nw) if case.layout == "KN" else (Nw, case.K)
    W = _draw(gen, b + wshape, case.w_dist, case.w_scale)
    bias = _draw(gen, (case.N,), "normal", 1.0) if case.has_bias else None
    residual = _draw(gen, b + (case.M, case.N), "normal", 1.0) if case.has_residual else None
    ins = Inputs(X, W, bias, residual)
    if pin:
        for f in ("X", "W", "bias", "residual"):
            t = getattr(ins, f)
            if t is not None:
                setattr(ins, f, t.pin_memory())
    return ins


def bits(t: torch.Tensor):
    """BF16 tensor (CPU) -> numpy uint16 view of its bit patterns (no copy)."""
    import numpy as np

    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------------------------------------
# Attention (the fused multi-head attention entry point; Section 5.2's transformer blocks)
@dataclass(frozen=True)
class AttentionCase:
    """One attention problem: Q [B, T, Hq, D], K and V [B, T, Hkv, D], BF16."""
    name: str
    B: int
    T: int
    Hq: int
    Hkv: int
    D: int
    causal: bool
    seed: int

    @property
    def flops(self) -> float:
        """Algorithmic FLOPs: two products of 2*D FLOPs per (query, visible key) pair."""
        pairs = self.T * (self.T + 1) / 2 if self.causal else self.T * self.T
        return 4.0 * self.D * pairs * self.B * self.Hq

    @property
    def algorithmic_bytes(self) -> int:
        """Q and O once, K and V once (BF16)."""
        return 2 * self.B * self.T * self.D * (2 * self.Hq + 2 * self.Hkv)


def attention_cases():
    """The attention shapes of the two transformer blocks: GPT-2-like (12 heads of 64) and LLaMA-like (32 query
    heads over 8 key/value heads of 128), at the benchmark's token counts (16 x 1024 and 4 x 2048 tokens) and at
    the paper's (128 x 512 and 16 x 2048), causal and not."""
    shapes = [("gpt2_16x1024", 16, 1024, 12, 12, 64), ("llama_4x2048", 4, 2048, 32, 8, 128),
              ("gpt2_128x512", 128, 512, 12, 12, 64), ("llama_16x2048", 16, 2048, 32, 8, 128)]
    out = []
    for i, (name, B, T, Hq, Hkv, D) in enumerate(shapes):
        for causal in (True, False):
            out.append(AttentionCase(f"{name}_{'causal' if causal else 'full'}", B, T, Hq, Hkv, D, causal, 7000 + i))
    return out


def make_attention_inputs(case, device="cpu"):
    """Seeded N(0, 1) BF16 Q, K, V (unit-variance activations, as after a layer norm and a projection)."""
    import torch

    gen = torch.Generator(device="cpu")
    gen.manual_seed(case.seed)
    q = torch.randn(case.B, case.T, case.Hq, case.D, generator=gen).to(torch.bfloat16)
    k = torch.randn(case.B, case.T, case.Hkv, case.D, generator=gen).to(torch.bfloat16)
    v = torch.randn(case.B, case.T, case.Hkv, case.D, generator=gen).to(torch.bfloat16)
    return q.to(device), k.to(device), v.to(device)


# ------------------------------------------------------------------------------------------------
# Whole transformer blocks (Section 5.2: the MiniGPT block at (128, 512, 768), the Llama-3-8B block at (16, 2048, 4096))
@dataclass(frozen=True)
class BlockCase:
    """One pre-norm transformer block: x [B * T, Hq * D] BF16 and its weights."""
    name: str
    kind: str  # "gpt": layer norms, biases, GELU MLP;  "llama": RMS norms, no biases, SwiGLU, grouped queries
    B: int
    T: int
    Hq: int
    Hkv: int
    D: int
    ffn: int
    seed: int

    @property
    def hidden(self) -> int:
        return self.Hq * self.D

    @property
    def flops(self) -> float:
        """Algorithmic FLOPs of the four linears and the causal attention (normalisations not counted)."""
        tok, C = self.B * self.T, self.hidden
        qc = (self.Hq + 2 * self.Hkv) * self.D
        mlp = (2 if self.kind == "llama" else 1) * self.ffn * C + C * self.ffn
        lin = 2.0 * tok * (qc * C + C * C + mlp)
        att = 4.0 * self.D * (self.T * (self.T + 1) / 2) * self.B * self.Hq
        return lin + att


def block_cases():
    """The paper's two block shapes."""
    return [BlockCase("gpt_block_128x512x768", "gpt", 128, 512, 12, 12, 64, 3072, 7100),
            BlockCase("llama_block_16x2048x4096", "llama", 16, 2048, 32, 8, 128, 14336, 7101)]


BLOCK_WEIGHT_NAMES = ("norm1_gamma", "norm1_beta", "wqkv", "bqkv", "wo", "bo", "norm2_gamma", "norm2_beta", "w1", "b1",
                      "w2", "b2")


def make_block_inputs(case, device="cpu"):
    """Seeded BF16 x ~ N(0, 1) and weights: linear weights N(0, 0.02^2) (the configurations' weight scale), norm
    gains 1 + N(0, 0.1^2), norm offsets and biases N(0, 0.02^2); a Llama block has gains and weights only.
    Returns (x, dict name -> tensor), drawn in the order of BLOCK_WEIGHT_NAMES after x."""
    import torch

    gen = torch.Generator(device="cpu")
    gen.manual_seed(case.seed)
    C, qc = case.hidden, (case.Hq + 2 * case.Hkv) * case.D
    shapes = {"norm1_gamma": (C,), "norm1_beta": (C,), "wqkv": (qc, C), "bqkv": (qc,), "wo": (C, C), "bo": (C,),
              "norm2_gamma": (C,), "norm2_beta": (C,), "w1": ((2 if case.kind == "llama" else 1) * case.ffn, C),
              "b1": (case.ffn,), "w2": (C, case.ffn), "b2": (C,)}
    x = torch.randn(case.B * case.T, C, generator=gen).to(torch.bfloat16).to(device)
    w = {}
    for name in BLOCK_WEIGHT_NAMES:
        vector = len(shapes[name]) == 1
        if case.kind == "llama" and vector and "gamma" not in name:
            continue
        t = torch.randn(*shapes[name], generator=gen)
        t = 1.0 + 0.1 * t if "gamma" in name else 0.02 * t
        w[name] = t.to(torch.bfloat16).to(device)
    return x, w


# ---------------------------------------------------------------------------------------------
# FP8 (E4M3) linear layers: the paper's pattern table is indexed by (rule, data type, architecture) and lists
# an FP8 GEMM among its Level-1 kernels (Section 3, Table 1); it gives no FP8 shapes, so the BF16 shapes are reused.
@dataclass(frozen=True)
class Fp8Case:
    name: str
    M: int
    N: int
    K: int
    epilogue: str = "NONE"
    has_bias: bool = False
    seed: int = 0
    x_amax: float = 4.0   # activations are scaled so that this many standard deviations reach the format's 448
    w_std: float = 0.02

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> float:
        return float(self.M * self.K + self.N * self.K + self.M * self.N * 2 + (self.N * 2 if self.has_bias else 0))


def fp8_cases() -> list[Fp8Case]:
    """The square 8192 problem, and the Llama-shaped and GPT-shaped MLP up-projections of the BF16 configurations."""
    return [
        Fp8Case("f8_square_8192", 8192, 8192, 8192, seed=7200),
        Fp8Case("f8_llama_qkv", 8192, 6144, 4096, seed=7201),
        Fp8Case("f8_gpt_up_gelu", 16384, 3072, 768, epilogue="BIAS_GELU_TANH", has_bias=True, seed=7202),
    ]


@dataclass
class Fp8Inputs:
    X: torch.Tensor                 # uint8 E4M3 codes [M, K]
    W: torch.Tensor                 # uint8 E4M3 codes [N, K]
    scale: float                    # the product of the two per-tensor scales
    bias: Optional[torch.Tensor]    # BF16 [N] or None


def make_fp8_inputs(case: Fp8Case) -> Fp8Inputs:
    """Per-tensor scaled quantisation of N(0,1) activations and N(0, w_std^2) weights, as an FP8 inference stack
    would store them: x_q = e4m3(x * sx), w_q = e4m3(w * sw) with the scales chosen so that `x_amax` standard
    deviations map to the format's largest value; the kernel is given 1 / (sx * sw).  Values beyond that clip
    to +-448 (torch's conversion saturates).  No arithmetic of the method: rounding random numbers to the
    storage format is input generation."""
    g = torch.Generator(device="cpu").manual_seed(case.seed)
    x = torch.randn((case.M, case.K), generator=g, dtype=torch.float32)
    w = torch.randn((case.N, case.K), generator=g, dtype=torch.float32) * case.w_std
    bias = torch.randn((case.N,), generator=g, dtype=torch.float32).to(torch.bfloat16) if case.has_bias else None
    sx = 448.0 / case.x_amax
    sw = 448.0 / (case.x_amax * case.w_std)
    xq = (x * sx).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
    wq = (w * sw).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
    return Fp8Inputs(xq, wq, 1.0 / (sx * sw), bias)


# ---------------------------------------------------------------------------------------------
# Grouped linear layers ("Grouped GEMM" in the paper's Table 1): the paper gives no shapes; these are the expert
# projections of a mixture-of-experts layer with the Llama-shaped hidden sizes of configuration 5.
@dataclass(frozen=True)
class GroupedCase:
    name: str
    tokens: int
    groups: int
    N: int
    K: int
    epilogue: str = "NONE"
    seed: int = 0

    @property
    def n_weight_cols(self) -> int:
        return 2 * self.N if self.epilogue == "SILU_GATE" else self.N

    @property
    def flops(self) -> float:
        return 2.0 * self.tokens * self.n_weight_cols * self.K

    @property
    def algorithmic_bytes(self) -> float:
        return 2.0 * (self.tokens * self.K + self.groups * self.n_weight_cols * self.K + self.tokens * self.N)


def grouped_cases() -> list[GroupedCase]:
    return [
        # (the short one first: timed right after the millisecond-long ones it inherits their power-limited clocks)
        GroupedCase("g8_short_k_gelu", 16384, 8, 3072, 768, epilogue="BIAS_GELU_TANH", seed=7303),
        GroupedCase("g8_moe_up_silu", 16384, 8, 14336, 4096, epilogue="SILU_GATE", seed=7300),
        GroupedCase("g8_moe_down", 16384, 8, 4096, 14336, seed=7301),
        GroupedCase("g64_small_experts", 16384, 64, 2048, 2048, seed=7302),
    ]


def grouped_rows(case: GroupedCase) -> list[int]:
    """Rows per group: every token picks a group uniformly at random (seeded), as a router without load balancing
    would: the counts are uneven and none is a multiple of the tile height."""
    g = torch.Generator(device="cpu").manual_seed(case.seed)
    pick = torch.randint(0, case.groups, (case.tokens,), generator=g)
    return torch.bincount(pick, minlength=case.groups).tolist()


def make_grouped_inputs(case: GroupedCase, device="cpu"):
    """X ~ N(0,1) [tokens, K], W ~ N(0, 0.02^2) [groups, Nw, K], BF16; drawn on the device when one is given (the
    weights alone are up to 1.9 GB)."""
    g = torch.Generator(device=device).manual_seed(case.seed + 1)
    X = torch.randn((case.tokens, case.K), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    W = torch.empty((case.groups, case.n_weight_cols, case.K), dtype=torch.bfloat16, device=device)
    for i in range(case.groups):
        W[i] = (torch.randn((case.n_weight_cols, case.K), generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    return X, W


# A row normalisation between two linear layers ("GEMM-LayerNorm-GEMM fusion" in the paper's Table 1): the paper
# gives no shapes; these are the attention output projection -> norm -> first MLP layer of its two blocks
# (Section 5.2), at the token counts of configurations 4 and 5.
@dataclass(frozen=True)
class NormChainCase:
    name: str
    tokens: int
    hidden: int
    ffn: int
    kind: str       # "layer": LayerNorm, biases, GELU;  "rms": RMSNorm, no biases, SiLU-gated
    seed: int = 0

    @property
    def gated(self) -> bool:
        return self.kind == "rms"

    @property
    def epilogue(self) -> str:
        return "SILU_GATE" if self.gated else "BIAS_GELU_TANH"

    @property
    def flops(self) -> float:
        return 2.0 * self.tokens * self.hidden * (self.hidden + (2 if self.gated else 1) * self.ffn)


def norm_chain_cases() -> list[NormChainCase]:
    return [
        NormChainCase("n_gpt2_out_ln_up", 16384, 768, 3072, "layer", seed=7400),
        NormChainCase("n_llama_o_rms_gate_up", 8192, 4096, 14336, "rms", seed=7401),
    ]


def make_norm_chain_inputs(case: NormChainCase, device="cpu") -> dict:
    """Attention output a and block input x0 ~ N(0,1) (x0 with a mean of 0.1: residual streams are not centred),
    weights ~ N(0, 0.02^2), gamma ~ N(1, 0.1^2), beta and biases ~ N(0, 0.02^2); BF16, seeded, drawn on `device`."""
    g = torch.Generator(device=device).manual_seed(case.seed)

    def draw(shape, scale, shift=0.0):
        return (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * scale + shift).to(torch.bfloat16)

    H, F, T = case.hidden, case.ffn, case.tokens
    t = {"a": draw((T, H), 1.0), "x0": draw((T, H), 1.0, 0.1), "wo": draw((H, H), 0.02), "gamma": draw((H,), 0.1, 1.0),
         "w1": draw(((2 * F) if case.gated else F, H), 0.02)}
    if not case.gated:
        t.update(bo=draw((H,), 0.02), beta=draw((H,), 0.02), b1=draw((F,), 0.02))
    return t
