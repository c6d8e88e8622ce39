"""GPU parity of fact_norm and fact_block_forward against the FP64 block oracle."""
import numpy as np
import pytest
import torch

from oracle import block as ob
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def rnd(shape, seed, scale=1.0, shift=0.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale + shift).to(torch.bfloat16)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """float64 -> nearest-even BF16 -> float64 (what storing an intermediate as BF16 does)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).double().numpy()


# ---------------------------------------------------------------------------------------------- fact_norm
@pytest.mark.parametrize("kind", ["layer", "rms"])
@pytest.mark.parametrize("M,C", [(1, 8), (37, 64), (300, 768), (129, 1032), (64, 4096), (19, 5000), (9, 8192)])
def test_norm_matches_the_oracle(h, kind, M, C):
    x = rnd((M, C), 1, 2.0, 0.5)
    gamma, beta = rnd((C,), 2, 0.1, 1.0), (rnd((C,), 3, 0.1) if kind == "layer" else None)
    got = to_f64(h.norm(x.to(DEV), gamma.to(DEV), None if beta is None else beta.to(DEV), kind=kind, eps=1e-5))
    xf, gf = to_f64(x), to_f64(gamma)
    ref = ob.layer_norm(xf, gf, to_f64(beta), 1e-5) if kind == "layer" else ob.rms_norm(xf, gf, 1e-5)
    # one BF16 rounding of an FP32 result: 2^-9 relative, plus FP32 noise of the statistics (C <= 8192 terms)
    assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-6).all()


def test_norm_strided_rows_in_place_and_errors(h):
    from paper_2604_26666_b200.binding import FactError
    M, C = 50, 256
    big = rnd((M, 3 * C), 4).to(DEV)
    x = big[:, C:2 * C]  # rows 3C apart: a column slice of a wider activation
    gamma = rnd((C,), 5, 0.1, 1.0).to(DEV)
    ref = ob.rms_norm(to_f64(x), to_f64(gamma), 1e-6)
    before = big.clone()
    h.norm(x, gamma, kind="rms", eps=1e-6, out=x)  # in place
    assert (np.abs(to_f64(x) - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-6).all()
    assert torch.equal(big[:, :C], before[:, :C]) and torch.equal(big[:, 2 * C:], before[:, 2 * C:])  # neighbours untouched
    with pytest.raises(FactError) as e:
        h.norm(rnd((4, 12), 6).to(DEV), rnd((12,), 7).to(DEV), kind="rms")
    assert e.value.code == 3  # C not a multiple of 8
    with pytest.raises(FactError) as e:
        h.norm(rnd((4, 16), 6).to(DEV), rnd((16,), 7).to(DEV), rnd((16,), 8).to(DEV), kind="rms")
    assert e.value.code == 1  # RMSNorm takes no beta
    assert h.norm(torch.empty((0, 64), dtype=torch.bfloat16, device=DEV), rnd((64,), 9).to(DEV)).shape == (0, 64)


# ---------------------------------------------------------------------------------------------- fact_block_forward
def run_block(h, case, x, w):
    """Returns y and the intermediates the call left in its workspace (cloned)."""
    from ctypes import byref

    from paper_2604_26666_b200.binding import lib
    wd = {k: v.to(DEV).contiguous() for k, v in w.items()}
    desc = h.block_desc(case.kind, case.B, case.T, case.Hq, case.Hkv, case.D, case.ffn, wd)
    ws = torch.empty(int(lib().fact_block_workspace_bytes(byref(desc))), dtype=torch.uint8, device=DEV)
    y = h.block_forward(desc, x.to(DEV), workspace=ws)
    assert h.device_status() == 0
    return y, {k: v.clone() for k, v in h.block_intermediates(desc, ws).items()}


def check_end_to_end(case, x, w, y, batches):
    """Against the exact FP64 chain (nothing rounded in between).  The device stores six intermediates and the
    output as BF16; each storage perturbs a value by up to 2^-9 of its size, and a perturbation keeps roughly its
    relative size through the sums that follow, so the output is off by about sqrt(7/3) 2^-9 rms(y) = 3e-3 rms(y)
    on average and, over millions of outputs with heavy-tailed activations, by ten times that at worst (the exact
    chain and the same chain with BF16 storage differ by up to 2.8e-2 rms(y) at the Llama shape).  Gates:
    mean |err| <= 6e-3 rms(ref) and |err| <= 1e-2 |ref| + 5e-2 rms(ref)."""
    wf = {k: to_f64(v) for k, v in w.items()}
    T = case.T
    for b in batches:
        ref, _ = ob.block_forward(case.kind, to_f64(x[b * T:(b + 1) * T]), wf, batch=1, seq=T, heads_q=case.Hq,
                                  heads_kv=case.Hkv, head_dim=case.D, eps=1e-5)
        err = np.abs(to_f64(y[b * T:(b + 1) * T]) - ref)
        rms = float(np.sqrt(np.mean(ref * ref)))
        assert err.mean() <= 6e-3 * rms, (err.mean() / rms)
        worst = float((err / (1e-2 * np.abs(ref) + 5e-2 * rms)).max())
        assert worst <= 1.0, worst


def check_stages(case, x, w, y, mid, batches):
    """Every stage against its definition applied to the inputs the device really had (its own stored BF16
    intermediates), with the single-operator gates: this is the tight check, free of the drift that BF16 storage
    causes along the chain."""
    from oracle.attention import attention_f64
    wf = {k: to_f64(v) for k, v in w.items()}
    g = lambda name: wf.get(name)
    T, C, D, Hq, Hkv = case.T, case.hidden, case.D, case.Hq, case.Hkv
    norm = (lambda t, ga, be: ob.layer_norm(t, ga, be, 1e-5)) if case.kind == "gpt" else (lambda t, ga, be: ob.rms_norm(t, ga, 1e-5))
    lin = lambda t, wt, bias: t @ wt.T + (0.0 if bias is None else bias)

    def gate(ref, got, epilogue, what):
        c, t = gates(ref, got, "bf16", epilogue)
        assert c <= 1.0 and t <= 1.0, (what, c, t)

    for b in batches:
        sl = slice(b * T, (b + 1) * T)
        xb = to_f64(x[sl])
        m = {k: to_f64(v[sl]) for k, v in mid.items()}
        yb = to_f64(y[sl])
        # qkv from x: the norm output was overwritten, so two stages at once (its BF16 storage is mirrored)
        gate(lin(bf16_round(norm(xb, g("norm1_gamma"), g("norm1_beta"))), g("wqkv"), g("bqkv")), m["qkv"], "BIAS", "qkv")
        q = m["qkv"][:, :C].reshape(1, T, Hq, D)
        k = m["qkv"][:, C:C + Hkv * D].reshape(1, T, Hkv, D)
        v = m["qkv"][:, C + Hkv * D:].reshape(1, T, Hkv, D)
        ref_a = attention_f64(q, k, v, causal=True).reshape(T, C)
        abs_a = attention_f64(q, k, np.abs(v), causal=True).reshape(T, C)
        err = np.abs(m["a"] - ref_a)  # the attention gate of tests/test_attention_gpu.py
        assert (err <= 2.0 ** -8 * np.abs(ref_a) + 2.0 ** -8 * abs_a + 1e-30).all(), ("a", float(err.max()))
        gate(lin(m["a"], g("wo"), g("bo")) + xb, m["x1"], "BIAS_RESIDUAL", "x1")
        ref_n2 = norm(m["x1"], g("norm2_gamma"), g("norm2_beta"))
        assert (np.abs(m["n"] - ref_n2) <= 2.0 ** -8 * np.abs(ref_n2) + 1e-6).all(), "n2"
        if case.kind == "gpt":
            gate(ob.gelu_tanh(lin(m["n"], g("w1"), g("b1"))), m["h"], "BIAS_GELU_TANH", "h")
        else:
            gu = lin(m["n"], g("w1"), None)
            gate(ob.silu(gu[:, :case.ffn]) * gu[:, case.ffn:], m["h"], "SILU_GATE", "h")
        gate(lin(m["h"], g("w2"), g("b2")) + m["x1"], yb, "BIAS_RESIDUAL", "y")


@pytest.mark.parametrize("case", [
    wl.BlockCase("gpt_small", "gpt", 2, 200, 4, 4, 64, 512, 7200),
    wl.BlockCase("gpt_one_token", "gpt", 3, 1, 2, 2, 64, 136, 7201),
    wl.BlockCase("llama_small", "llama", 2, 300, 4, 2, 128, 768, 7202),
    wl.BlockCase("llama_mqa_ragged", "llama", 1, 131, 4, 1, 64, 264, 7203),
], ids=lambda c: c.name)
def test_block_matches_the_oracle(h, case):
    x, w = wl.make_block_inputs(case)
    y, mid = run_block(h, case, x, w)
    check_stages(case, x, w, y, mid, range(case.B))
    check_end_to_end(case, x, w, y, range(case.B))


@pytest.mark.parametrize("case", wl.block_cases(), ids=lambda c: c.name)
def test_paper_block_shapes_on_sampled_sequences(h, case):
    """The paper's two block shapes in the configuration bench.py times, checked on whole sequences of the batch
    (a sequence is the unit the oracle can compute by itself)."""
    x, w = wl.make_block_inputs(case)
    y, mid = run_block(h, case, x, w)
    batches = [0, case.B - 1] if case.kind == "gpt" else [case.B // 2]
    check_stages(case, x, w, y, mid, batches)
    check_end_to_end(case, x, w, y, batches)


def test_block_errors_and_workspace(h):
    from paper_2604_26666_b200.binding import FactError, lib
    from ctypes import byref
    case = wl.BlockCase("e", "gpt", 1, 16, 2, 2, 64, 128, 7204)
    x, w = wl.make_block_inputs(case)
    wd = {k: v.to(DEV) for k, v in w.items()}
    desc = h.block_desc("gpt", 1, 16, 2, 2, 64, 128, wd)
    need = int(lib().fact_block_workspace_bytes(byref(desc)))
    assert need >= 16 * (128 * 3 + 384 + 128) * 2
    small = torch.empty(need - 256, dtype=torch.uint8, device=DEV)
    with pytest.raises(FactError) as e:
        h.block_forward(desc, x.to(DEV), workspace=small)
    assert e.value.code == 5
    bad = h.block_desc("llama", 1, 16, 2, 2, 64, 128, wd)  # a Llama block takes no biases
    with pytest.raises(FactError) as e:
        h.block_forward(bad, x.to(DEV))
    assert e.value.code == 1
    # y may alias x
    xin = x.to(DEV).clone()
    y1 = h.block_forward(desc, x.to(DEV))
    h.block_forward(desc, xin, out=xin)
    assert torch.equal(y1, xin)
