"""GPU parity of fact_attention against the FP64 attention oracle."""
import numpy as np
import pytest
import torch

from oracle.attention import attention as oracle_attention
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import gates, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def rnd(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


def attention_gates(q, k, v, causal, got, rows=None, scale=0.0):
    """(contract ratio, tight ratio).  Contract: |err| <= 1e-2 + 1e-2 |ref| (BF16 output).
    Tight: |err| <= 2^-8 |ref| + 2^-8 A with A = sum_j p_j |v_j| (the oracle run on |V|): the kernel rounds each
    probability to BF16 (relative 2^-9) before the second product, so the weighted sum is off by at most 2^-9 A;
    the row sum is taken from the unrounded probabilities (a normalisation mismatch of at most 2^-9 |ref|) and
    the result is rounded once more to BF16 (2^-9 |ref|)."""
    sc = None if scale <= 0 else scale
    qb, kb, vb = wl.bits(q.contiguous()), wl.bits(k.contiguous()), wl.bits(v.contiguous())
    ref = oracle_attention(qb, kb, vb, causal=causal, scale=sc, rows=rows)
    absv = oracle_attention(qb, kb, vb & np.uint16(0x7FFF), causal=causal, scale=sc, rows=rows)
    err = np.abs(got - ref)
    contract = float((err / (1e-2 + 1e-2 * np.abs(ref))).max())
    tight = float((err / (2.0 ** -8 * np.abs(ref) + 2.0 ** -8 * absv + 1e-30)).max())
    return contract, tight


def check(h, q, k, v, causal, rows=None, scale=0.0):
    dev = "cuda:0"
    out = h.attention(q.to(dev), k.to(dev), v.to(dev), causal=causal, scale=scale)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    got = to_f64(out)
    if rows is not None:
        got = got[:, rows]
    assert np.isfinite(got).all()
    c, t = attention_gates(q, k, v, causal, got, rows=rows, scale=scale)
    assert c <= 1.0, f"contract gate ratio {c:.3f}"
    assert t <= 1.0, f"tight gate ratio {t:.3f}"
    return out


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("T", [128, 200, 513])
def test_mha_small(h, causal, D, T):
    B, H = 2, 3
    check(h, rnd((B, T, H, D), 1), rnd((B, T, H, D), 2), rnd((B, T, H, D), 3), causal)


@pytest.mark.parametrize("causal", [True, False])
def test_grouped_queries(h, causal):
    B, T, Hq, Hkv, D = 2, 300, 8, 2, 128
    check(h, rnd((B, T, Hq, D), 4), rnd((B, T, Hkv, D), 5), rnd((B, T, Hkv, D), 6), causal)


def test_cross_attention_lengths(h):
    # non-causal with different query and key lengths, both ragged
    B, H, D = 1, 2, 64
    check(h, rnd((B, 77, H, D), 7), rnd((B, 391, H, D), 8), rnd((B, 391, H, D), 9), False)


def test_views_into_a_fused_qkv_projection(h):
    # Q, K, V are column slices of one [tokens, (Hq + 2 Hkv) D] matrix, as the QKV linear produces them
    B, T, Hq, Hkv, D = 2, 260, 4, 2, 64
    fused = rnd((B, T, (Hq + 2 * Hkv) * D), 10)
    q = fused[..., : Hq * D].view(B, T, Hq, D)
    k = fused[..., Hq * D: (Hq + Hkv) * D].view(B, T, Hkv, D)
    v = fused[..., (Hq + Hkv) * D:].view(B, T, Hkv, D)
    dev = "cuda:0"
    fd = fused.to(dev)
    qd = fd[..., : Hq * D].view(B, T, Hq, D)
    kd = fd[..., Hq * D: (Hq + Hkv) * D].view(B, T, Hkv, D)
    vd = fd[..., (Hq + Hkv) * D:].view(B, T, Hkv, D)
    out = h.attention(qd, kd, vd, causal=True)
    torch.cuda.synchronize()
    c, t = attention_gates(q, k, v, True, to_f64(out))
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_heads_first_storage(h):
    # [B, H, T, D] storage viewed as [B, T, H, D]: the head stride is larger than the token stride
    B, T, H, D = 1, 140, 3, 128
    qs, ks, vs = (rnd((B, H, T, D), s) for s in (11, 12, 13))
    dev = "cuda:0"
    out_store = torch.empty((B, H, T, D), dtype=torch.bfloat16, device=dev)
    h.attention(qs.to(dev).permute(0, 2, 1, 3), ks.to(dev).permute(0, 2, 1, 3), vs.to(dev).permute(0, 2, 1, 3),
                causal=True, out=out_store.permute(0, 2, 1, 3))
    torch.cuda.synchronize()
    c, t = attention_gates(qs.permute(0, 2, 1, 3), ks.permute(0, 2, 1, 3), vs.permute(0, 2, 1, 3), True,
                           to_f64(out_store.permute(0, 2, 1, 3)))
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_closed_forms(h):
    B, T, H, D = 1, 300, 2, 64
    q, k = rnd((B, T, H, D), 14), rnd((B, T, H, D), 15)
    row = rnd((D,), 16)
    v = row.expand(B, T, H, D).contiguous()
    out = check(h, q, k, v, True)
    # weights sum to one: every output row is the common value row up to the rounding of P
    assert (out.float().cpu() - row.float()).abs().max() <= 2.0 ** -7 * row.float().abs().max() + 1e-3
    # first causal row sees only key 0: exact
    v2 = rnd((B, T, H, D), 17)
    out = check(h, q, k, v2, True)
    assert torch.equal(out[:, 0].cpu(), v2[:, 0])


def test_large_scores_do_not_overflow(h):
    B, T, H, D = 1, 256, 1, 64
    check(h, rnd((B, T, H, D), 18, 6.0), rnd((B, T, H, D), 19, 6.0), rnd((B, T, H, D), 20), True)


@pytest.mark.parametrize("name", ["gpt", "llama"])
def test_block_shapes_sampled_rows(h, name):
    # the attention shapes of the two transformer blocks at the benchmark token counts
    if name == "gpt":
        B, T, Hq, Hkv, D = 16, 1024, 12, 12, 64
    else:
        B, T, Hq, Hkv, D = 4, 2048, 32, 8, 128
    q, k, v = rnd((B, T, Hq, D), 21), rnd((B, T, Hkv, D), 22), rnd((B, T, Hkv, D), 23)
    rows = np.array(sorted({0, 1, 127, 128, 129, T // 2, T - 129, T - 2, T - 1}), dtype=np.int64)
    check(h, q, k, v, True, rows=rows)


@pytest.mark.parametrize("causal", [True, False])
def test_many_ragged_tiles_per_cta(h, causal):
    """960 work items over 148 persistent CTAs: every CTA walks several tiles, the last tile of each sequence is
    ragged (333 = 2 * 128 + 77) and, when causal, the tiles of one CTA have different numbers of key blocks."""
    B, T, Hq, Hkv, D = 40, 333, 8, 2, 64
    q, k, v = rnd((B, T, Hq, D), 31), rnd((B, T, Hkv, D), 32), rnd((B, T, Hkv, D), 33)
    check(h, q, k, v, causal)
    # 384 items of four different weights at head_dim 128: causal, the host deals them out (fact_attention_deal) and
    # the kernel walks the list it was handed; the same rows must come out as for any other order
    B, T, Hq, Hkv, D = 6, 1000, 16, 4, 128
    q, k, v = rnd((B, T, Hq, D), 131), rnd((B, T, Hkv, D), 132), rnd((B, T, Hkv, D), 133)
    rows = np.array(sorted({0, 1, 127, 128, 255, 256, 500, 767, 768, 998, 999}), dtype=np.int64)
    check(h, q, k, v, causal, rows=rows)


def test_long_sequence_sampled_rows(h):
    # 8192 keys: 64 key blocks per tile; reference maxima move late in the row for some rows (scores scaled up)
    B, T, Hq, Hkv, D = 1, 8192, 4, 1, 128
    q, k, v = rnd((B, T, Hq, D), 34, 1.5), rnd((B, T, Hkv, D), 35, 1.5), rnd((B, T, Hkv, D), 36)
    rows = np.array(sorted({0, 127, 128, 4095, 4096, 8000, 8191}), dtype=np.int64)
    check(h, q, k, v, True, rows=rows)
    check(h, q, k, v, False, rows=rows)


def test_reference_that_keeps_rising(h):
    """Keys sorted by growing norm: the row maximum rises block after block, so the output accumulator is
    rescaled repeatedly (the rare path of the lazy rescaling) -- and once by a large step."""
    B, T, H, D = 1, 1024, 2, 64
    q = rnd((B, T, H, D), 37)
    ramp = torch.linspace(0.2, 6.0, T).view(1, T, 1, 1)
    k = (q.float() * ramp).to(torch.bfloat16)  # key j is query j scaled up: scores grow with j
    k[:, 900:] = (k[:, 900:].float() * 3).to(torch.bfloat16)
    v = rnd((B, T, H, D), 38)
    check(h, q, k, v, True)
    check(h, q, k, v, False)


def test_repeated_calls_are_bitwise_identical(h):
    B, T, Hq, Hkv, D = 3, 700, 8, 4, 128
    q, k, v = rnd((B, T, Hq, D), 39).to("cuda:0"), rnd((B, T, Hkv, D), 40).to("cuda:0"), rnd((B, T, Hkv, D), 41).to("cuda:0")
    a = h.attention(q, k, v, causal=True).clone()
    for _ in range(3):
        assert torch.equal(a, h.attention(q, k, v, causal=True))
    assert h.device_status() == 0


def test_host_dealt_causal_calls_in_a_cuda_graph_and_between_other_shapes(h):
    """A causal problem whose items the host deals out (the list travels as a kernel parameter, so a captured launch
    keeps its own copy): replayed from a CUDA graph, and interleaved with another dealt shape and a shape that is
    not dealt, every call gives the bits of its first run."""
    dev = "cuda:0"
    shapes = [(16, 1024, 12, 12, 64), (6, 1000, 16, 4, 128), (2, 300, 4, 4, 64)]
    ins, first = [], []
    for i, (B, T, Hq, Hkv, D) in enumerate(shapes):
        q, k, v = (rnd((B, T, Hq, D), 50 + i).to(dev), rnd((B, T, Hkv, D), 60 + i).to(dev),
                   rnd((B, T, Hkv, D), 70 + i).to(dev))
        ins.append((q, k, v))
        first.append(h.attention(q, k, v, causal=True).clone())
    for _ in range(2):
        for (q, k, v), want in zip(ins, first):
            assert torch.equal(h.attention(q, k, v, causal=True), want)
    outs = [torch.empty_like(f) for f in first]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream(dev)):
        for (q, k, v), o in zip(ins, outs):
            h.attention(q, k, v, causal=True, out=o)
    for _ in range(2):
        for o in outs:
            o.zero_()
        g.replay()
        torch.cuda.synchronize()
        for o, want in zip(outs, first):
            assert torch.equal(o, want)
    assert h.device_status() == 0
    rows = np.array([0, 127, 128, 511, 512, 1023], dtype=np.int64)
    c, t = attention_gates(ins[0][0].cpu(), ins[0][1].cpu(), ins[0][2].cpu(), True, to_f64(first[0])[:, rows], rows=rows)
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_error_codes(h):
    from paper_2604_26666_b200.binding import FactError
    dev = "cuda:0"
    q = torch.zeros(1, 128, 2, 96, dtype=torch.bfloat16, device=dev)
    with pytest.raises(FactError) as e:
        h.attention(q, q, q)
    assert e.value.code == 3  # head_dim 96
    q = torch.zeros(1, 128, 3, 64, dtype=torch.bfloat16, device=dev)
    k = torch.zeros(1, 128, 2, 64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(FactError) as e:
        h.attention(q, k, k)
    assert e.value.code == 1  # 3 query heads over 2 key/value heads
    k = torch.zeros(1, 64, 3, 64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(FactError) as e:
        h.attention(q, k, k, causal=True)
    assert e.value.code == 3  # causal with different lengths


def _sweep_cases():
    rng = np.random.default_rng(2024)
    cases = []
    for i in range(28):
        D = int(rng.choice([64, 128]))
        causal = bool(rng.integers(0, 2))
        Hkv = int(rng.integers(1, 4))
        Hq = Hkv * int(rng.choice([1, 2, 4]))
        B = int(rng.integers(1, 4))
        # lengths around the tile (128), item (256) and key-block (64 / 128) borders, and a few larger ones
        pool = [1, 2, 63, 64, 65, 127, 128, 129, 191, 192, 255, 256, 257, 320, 383, 384, 385, 511, 512, 600, 769]
        Tq = int(rng.choice(pool))
        Tk = Tq if causal else int(rng.choice(pool))
        cases.append((i, B, Tq, Tk, Hq, Hkv, D, causal))
    return cases


@pytest.mark.parametrize("i,B,Tq,Tk,Hq,Hkv,D,causal", _sweep_cases(),
                         ids=[f"{c[0]}-B{c[1]}-Tq{c[2]}-Tk{c[3]}-H{c[4]}/{c[5]}-D{c[6]}-{'c' if c[7] else 'f'}" for c in _sweep_cases()])
def test_random_shapes(h, i, B, Tq, Tk, Hq, Hkv, D, causal):
    """Seeded random shapes: lengths on and around every border the kernel has (tile of 128 query rows, item of two
    tiles, key blocks of 64 or 128, a second tile wholly past the end), grouped queries, both head sizes."""
    check(h, rnd((B, Tq, Hq, D), 500 + i), rnd((B, Tk, Hkv, D), 600 + i), rnd((B, Tk, Hkv, D), 700 + i), causal)
