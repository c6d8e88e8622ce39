"""CPU pins of the attention oracle: library SDPA in float64, closed forms and invariances."""
import numpy as np
import pytest
import torch

from oracle.attention import attention
from paper_2604_26666_b200 import workloads as wl


def bits(t):
    return wl.bits(t.to(torch.bfloat16).contiguous())


def rnd(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2)])
def test_matches_library_sdpa_in_float64(causal, hq, hkv):
    B, T, D = 2, 37, 16
    q, k, v = rnd((B, T, hq, D), 1), rnd((B, T, hkv, D), 2), rnd((B, T, hkv, D), 3)
    got = attention(bits(q), bits(k), bits(v), causal=causal)
    # library routine: [B, H, T, D] layout, K/V heads repeated for grouped queries (as the paper does)
    qd, kd, vd = (x.double().permute(0, 2, 1, 3) for x in (q, k, v))
    kd = kd.repeat_interleave(hq // hkv, dim=1)
    vd = vd.repeat_interleave(hq // hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qd, kd, vd, is_causal=causal).permute(0, 2, 1, 3).numpy()
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_closed_forms():
    B, T, H, D = 1, 9, 2, 8
    q, k = rnd((B, T, H, D), 4), rnd((B, T, H, D), 5)
    # every value row equal -> the output is that row, whatever the weights (they sum to one)
    row = rnd((D,), 6)
    v = row.expand(B, T, H, D).contiguous()
    out = attention(bits(q), bits(k), bits(v), causal=False)
    assert np.allclose(out, np.broadcast_to(row.double().numpy(), out.shape), rtol=1e-14, atol=1e-15)
    # causal: the first query position sees only key 0
    v = rnd((B, T, H, D), 7)
    out = attention(bits(q), bits(k), bits(v), causal=True)
    assert np.allclose(out[:, 0], v.double().numpy()[:, 0], rtol=1e-14, atol=1e-15)
    # all-zero queries -> uniform weights -> the mean of the visible value rows
    z = torch.zeros(B, T, H, D, dtype=torch.bfloat16)
    out = attention(bits(z), bits(k), bits(v), causal=True)
    vd = v.double().numpy()
    for i in range(T):
        assert np.allclose(out[:, i], vd[:, : i + 1].mean(axis=1), rtol=1e-13, atol=1e-14)
    # one dominating key: a huge score on key 3 -> the output is value row 3
    kk = torch.zeros(B, T, H, D)
    kk[:, 3] = 16.0
    qq = torch.ones(B, T, H, D) * 16.0
    out = attention(bits(qq), bits(kk), bits(v), causal=False, scale=1.0)
    assert np.allclose(out, np.broadcast_to(vd[:, 3:4], out.shape), rtol=0, atol=1e-12)


def test_invariances():
    B, T, H, D = 1, 12, 3, 8
    q, k, v = rnd((B, T, H, D), 8), rnd((B, T, H, D), 9), rnd((B, T, H, D), 10)
    base = attention(bits(q), bits(k), bits(v), causal=False)
    perm = torch.randperm(T, generator=torch.Generator().manual_seed(11))
    shuffled = attention(bits(q), bits(k[:, perm]), bits(v[:, perm]), causal=False)
    assert np.allclose(base, shuffled, rtol=1e-12, atol=1e-13)  # keys are a set when nothing is masked
    sub = attention(bits(q), bits(k), bits(v), causal=True, rows=[0, 5, 11])
    full = attention(bits(q), bits(k), bits(v), causal=True)
    assert np.array_equal(sub, full[:, [0, 5, 11]])
    # grouped queries == the same attention on repeat-interleaved key/value heads
    k2, v2 = rnd((B, T, 1, D), 12), rnd((B, T, 1, D), 13)
    g = attention(bits(q), bits(k2), bits(v2), causal=True)
    e = attention(bits(q), bits(k2.repeat_interleave(3, dim=2)), bits(v2.repeat_interleave(3, dim=2)), causal=True)
    assert np.array_equal(g, e)
    # the default scale is 1/sqrt(D): doubling Q and halving the scale changes nothing
    a = attention(bits(q * 2), bits(k), bits(v), causal=False, scale=0.5 / np.sqrt(D))
    assert np.allclose(a, base, rtol=1e-12, atol=1e-13)


def test_brute_force_python_loops_on_a_tiny_case():
    """The definition written out with scalar loops and math.exp: softmax(scale q.k + mask) v, grouped queries."""
    import math

    B, T, Hq, Hkv, D = 1, 5, 4, 2, 4
    q, k, v = rnd((B, T, Hq, D), 14), rnd((B, T, Hkv, D), 15), rnd((B, T, Hkv, D), 16)
    qf, kf, vf = (x.double().tolist() for x in (q, k, v))
    for causal in (False, True):
        got = attention(bits(q), bits(k), bits(v), causal=causal)
        for h in range(Hq):
            g = h // (Hq // Hkv)
            for i in range(T):
                keys = range(i + 1) if causal else range(T)
                s = [sum(qf[0][i][h][d] * kf[0][j][g][d] for d in range(D)) / math.sqrt(D) for j in keys]
                w = [math.exp(x - max(s)) for x in s]
                for d in range(D):
                    want = sum(wj * vf[0][j][g][d] for wj, j in zip(w, keys)) / sum(w)
                    assert abs(got[0, i, h, d] - want) <= 1e-13 * max(1.0, abs(want))


def test_key_set_split_and_merge():
    """Attention over a key set equals the log-sum-exp weighted mix of attention over its two halves."""
    B, T, H, D = 1, 10, 2, 8
    q, k, v = rnd((B, T, H, D), 17), rnd((B, T, H, D), 18), rnd((B, T, H, D), 19)
    full = attention(bits(q), bits(k), bits(v), causal=False)
    a = attention(bits(q), bits(k[:, :4]), bits(v[:, :4]), causal=False)
    b = attention(bits(q), bits(k[:, 4:]), bits(v[:, 4:]), causal=False)
    qd, kd = q.double().numpy(), k.double().numpy()
    s = np.einsum("bihd,bjhd->bihj", qd, kd) / np.sqrt(D)
    za, zb = np.exp(s[..., :4]).sum(-1), np.exp(s[..., 4:]).sum(-1)  # partition sums of the halves
    mix = (a * za[..., None] + b * zb[..., None]) / (za + zb)[..., None]
    assert np.allclose(full, mix, rtol=1e-12, atol=1e-13)
    # a key that the query scores hugely negative has weight ~ 0: the result equals attention without that key
    far = k.clone()
    far[:, -1] = -(q[:, 0] * 64)
    near = attention(bits(q[:, :1]), bits(far), bits(v), causal=False)
    drop = attention(bits(q[:, :1]), bits(k[:, :-1]), bits(v[:, :-1]), causal=False)
    assert np.allclose(near, drop, rtol=1e-9, atol=1e-10)
