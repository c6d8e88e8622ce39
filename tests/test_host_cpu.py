"""CPU-only checks of the host side: the library loads and exports every symbol the header declares,
the header and the binding agree, the workload table matches the benchmark configurations."""
import re
from pathlib import Path

import pytest

from paper_2604_26666_b200 import workloads as wl

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def libfact():
    from paper_2604_26666_b200 import build
    from paper_2604_26666_b200.binding import lib

    build.build()  # nvcc cross-compiles for sm_100a without a GPU
    return lib()


def declared_symbols():
    text = (ROOT / "include" / "fact.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fact_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(libfact):
    from paper_2604_26666_b200.binding import EXPORTED

    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(libfact, n), f"{n} is declared in fact.h but not exported"
    assert sorted(EXPORTED) == names, "binding.EXPORTED and fact.h disagree"


def test_status_strings(libfact):
    assert libfact.fact_status_string(0) == b"FACT_OK"
    assert libfact.fact_status_string(7) == b"FACT_ERR_DEVICE_TIMEOUT"
    assert libfact.fact_status_string(99) == b"FACT_ERR_UNKNOWN"


def test_calls_without_a_handle_fail_cleanly(libfact):
    from ctypes import byref, c_int, c_size_t

    n = c_size_t(0)
    assert libfact.fact_workspace_bytes(None, 0, 1, 8, 8, 8, 0, 0, 0, None, byref(n)) == 1
    assert libfact.fact_gemm(None, 8, 8, 8, None, 8, None, 8, 0, None, 8, 0, None, None, 0, None) == 1
    assert libfact.fact_launch_count(None) == 0
    assert libfact.fact_destroy(None) == 0
    v = c_int(0)
    assert libfact.fact_device_status(None, None, byref(v)) == 1


def test_no_product_module_imports_the_oracle():
    for f in (ROOT / "paper_2604_26666_b200").glob("*.py"):
        assert not re.search(r"^\s*(import|from)\s+oracle\b", f.read_text(), flags=re.M), f
    for f in (ROOT / "paper_2604_26666_b200" / "csrc").iterdir():
        assert "oracle" not in f.read_text().lower(), f
    assert "paper_2604_26666_b200" not in (ROOT / "oracle" / "__init__.py").read_text().replace(
        "CUDA package", "")


def test_workload_table_matches_the_configurations():
    cases = {c.name: c for c in wl.benchmark_cases()}
    assert len(cases) == 13
    c = cases["c1_512_bias_relu"]
    assert (c.M, c.N, c.K, c.epilogue, c.layout, c.seed) == (512, 512, 512, "BIAS_RELU", "KN", 0)
    assert [cases[f"c2_square_{n}"].flops for n in (4096, 8192)] == [2.0 * 4096 ** 3, 2.0 * 8192 ** 3]
    c = cases["c3_batched_128x512x512x1024"]
    assert (c.batch, c.M, c.N, c.K) == (128, 512, 512, 1024)
    c = cases["c3_splitk_256x256x131072"]
    assert (c.M, c.N, c.K, c.out) == (256, 256, 131072, "f32")
    c = cases["c5_gate_up_silu"]
    assert c.n_weight_cols == 28672 and c.N == 14336 and c.flops == 2.0 * 8192 * 28672 * 4096
    c = cases["c4_mlp_up_gelu"]
    # X + W + bias read once, Y written once
    assert c.algorithmic_bytes == 2 * (16384 * 768 + 768 * 3072 + 3072 + 16384 * 3072)


def test_inputs_are_reproducible_and_scaled():
    import torch

    c = wl.case_by_name("c2_square_4096")
    small = wl.Case("s", "gemm", 64, 48, 4096, seed=c.seed, x_scale=c.x_scale, w_scale=c.w_scale)
    a = wl.make_inputs(small)
    b = wl.make_inputs(small)
    assert torch.equal(a.X, b.X) and torch.equal(a.W, b.W)
    assert a.X.dtype == torch.bfloat16 and a.W.shape == (4096, 48)
    assert abs(float(a.X.float().std()) * 64.0 - 1.0) < 0.05  # N(0,1)/sqrt(4096)


def test_block_workspace_layout_is_host_only_and_consistent():
    """fact_block_workspace_bytes / _offsets need no GPU: sizes, order, alignment, rejection of bad descriptors."""
    from ctypes import byref, c_size_t

    from paper_2604_26666_b200 import binding

    L = binding.lib()
    b = binding.Block()
    b.kind, b.batch, b.seq, b.hidden, b.heads_q, b.heads_kv, b.head_dim, b.ffn = 1, 16, 2048, 4096, 32, 8, 128, 14336
    tok = 16 * 2048
    off = (c_size_t * 5)()
    assert L.fact_block_workspace_offsets(byref(b), off) == 0
    o = [int(v) for v in off]
    sizes = [tok * 4096 * 2, tok * 6144 * 2, tok * 4096 * 2, tok * 4096 * 2, tok * 14336 * 2]
    assert o[0] == 0 and all(x % 256 == 0 for x in o)
    for i in range(4):
        assert o[i + 1] >= o[i] + sizes[i]  # buffers in order, no overlap
    total = int(L.fact_block_workspace_bytes(byref(b)))
    assert total >= o[4] + sizes[4] and total - (o[4] + sizes[4]) < 256
    b.heads_kv = 5  # 32 query heads cannot share 5 key/value heads
    assert int(L.fact_block_workspace_bytes(byref(b))) == 0
    assert L.fact_block_workspace_offsets(byref(b), off) == 1  # FACT_ERR_INVALID_ARG
    b.heads_kv, b.hidden = 8, 4000  # hidden != heads_q * head_dim
    assert int(L.fact_block_workspace_bytes(byref(b))) == 0


def test_attention_and_block_workloads():
    cases = {c.name: c for c in wl.attention_cases()}
    assert len(cases) == 8
    c = cases["llama_4x2048_causal"]
    assert c.flops == 4.0 * 128 * (2048 * 2049 / 2) * 4 * 32
    assert cases["llama_4x2048_full"].algorithmic_bytes == 2 * 4 * 2048 * 128 * (2 * 32 + 2 * 8)
    q, k, v = wl.make_attention_inputs(wl.AttentionCase("t", 1, 5, 4, 2, 8, True, 3))
    assert q.shape == (1, 5, 4, 8) and k.shape == v.shape == (1, 5, 2, 8)
    q2, _, _ = wl.make_attention_inputs(wl.AttentionCase("t", 1, 5, 4, 2, 8, True, 3))
    assert (wl.bits(q) == wl.bits(q2)).all()
    gpt, llama = wl.block_cases()
    assert (gpt.B, gpt.T, gpt.hidden, gpt.ffn) == (128, 512, 768, 3072)
    assert (llama.B, llama.T, llama.hidden, llama.Hq, llama.Hkv, llama.ffn) == (16, 2048, 4096, 32, 8, 14336)
    x, w = wl.make_block_inputs(wl.BlockCase("t", "llama", 1, 4, 2, 1, 8, 16, 5))
    assert sorted(w) == ["norm1_gamma", "norm2_gamma", "w1", "w2", "wo", "wqkv"] and w["w1"].shape == (32, 16)
    x, w = wl.make_block_inputs(wl.BlockCase("t", "gpt", 1, 4, 2, 2, 8, 16, 5))
    assert len(w) == 12 and w["w1"].shape == (16, 16) and w["bqkv"].shape == (48,)
    assert [c.name for c in wl.paper_cases()] == ["p3_batched_128x512x2048x1024", "p6_splitk_256x256x524288"]


@pytest.mark.parametrize("groups,sk_tiles,k_blocks", [
    (74, 44, 48), (74, 44 + 74, 12), (148, 1, 2048), (148, 147, 3), (74, 73, 1), (7, 3, 5), (5, 12, 4), (3, 2, 1),
    (148, 20, 11), (2, 1, 1),
])
def test_stream_k_partition_covers_every_k_block_once(libfact, groups, sk_tiles, k_blocks):
    """The stream-K schedule the kernels walk (fact_stream_k_pieces): runs are contiguous and balanced, every
    k-block of every tile is in exactly one piece, every tile has exactly one finishing piece, and the pieces it
    waits for are the first work of the groups right after it."""
    from paper_2604_26666_b200.binding import stream_k_pieces

    per_group = [stream_k_pieces(groups, sk_tiles, k_blocks, g) for g in range(groups)]
    lengths = [sum(k1 - k0 for (_, k0, k1, _, _) in ps) for ps in per_group]
    assert sum(lengths) == sk_tiles * k_blocks
    assert max(lengths) - min(lengths) <= 1
    assert lengths == sorted(lengths, reverse=True)  # the longer runs come first
    covered = {}
    pos = 0
    for g, ps in enumerate(per_group):
        for i, (tile, k0, k1, role, peers) in enumerate(ps):
            assert 0 <= tile < sk_tiles and 0 <= k0 < k1 <= k_blocks
            assert tile * k_blocks + k0 == pos, "runs are contiguous in (tile, k) order"
            pos += k1 - k0
            for k in range(k0, k1):
                assert (tile, k) not in covered
                covered[(tile, k)] = g
            if role == 0:
                assert (k0, k1) == (0, k_blocks) and peers == 0
            elif role == 1:
                assert k0 == 0 and k1 < k_blocks and peers >= 1
                assert i == len(ps) - 1, "a run can only end inside a tile with its last piece"
            else:
                assert role == 2 and k0 > 0 and peers == 0
                assert i == 0, "a parked piece is the first thing its group does"
    assert len(covered) == sk_tiles * k_blocks
    for tile in range(sk_tiles):
        owners = sorted({covered[(tile, k)] for k in range(k_blocks)})
        assert owners == list(range(owners[0], owners[-1] + 1)), "a tile's pieces belong to consecutive groups"
        first = per_group[owners[0]][-1] if len(owners) > 1 else None
        if first is not None:
            assert first[0] == tile and first[3] == 1 and first[4] == len(owners) - 1


def test_stream_k_pieces_rejects_bad_arguments(libfact):
    import ctypes

    n = ctypes.c_int(0)
    buf = (ctypes.c_int32 * 5)()
    assert libfact.fact_stream_k_pieces(0, 1, 1, 0, 1, buf, ctypes.byref(n)) == 1
    assert libfact.fact_stream_k_pieces(4, 1, 0, 0, 1, buf, ctypes.byref(n)) == 1
    assert libfact.fact_stream_k_pieces(4, 1, 1, 4, 1, buf, ctypes.byref(n)) == 1
    assert libfact.fact_stream_k_pieces(4, 1, 1, 0, 1, buf, None) == 1
    assert libfact.fact_stream_k_pieces(4, 1, 8, 3, 0, None, ctypes.byref(n)) == 0 and n.value == 1


def test_binding_rejects_mismatched_shapes_without_launching_anything():
    """A Python shape mistake must be a ValueError, not an out-of-bounds device access: the binding checks inner
    dimensions, the output's shape and the devices before it hands a pointer to the library.  CPU tensors reach
    the shape checks (the CUDA requirement comes last), so nothing can launch here."""
    import torch

    from paper_2604_26666_b200 import binding as bd

    bf, f32 = torch.bfloat16, torch.float32
    A = torch.zeros(64, 128, dtype=bf)
    with pytest.raises(ValueError, match="inner dimensions"):
        bd._validate_matmul(A, torch.zeros(120, 96, dtype=bf), None, "KN")
    with pytest.raises(ValueError, match="inner dimensions"):
        bd._validate_matmul(A, torch.zeros(96, 120, dtype=bf), None, "NK")
    with pytest.raises(ValueError, match="shape"):  # too small an output would be written past its end
        bd._validate_matmul(A, torch.zeros(128, 96, dtype=bf), torch.zeros(32, 96, dtype=f32), "KN")
    with pytest.raises(ValueError, match="shape"):
        bd._validate_matmul(torch.zeros(2, 64, 128, dtype=bf), torch.zeros(2, 128, 96, dtype=bf),
                            torch.zeros(64, 96, dtype=bf), "KN", batched=True)
    with pytest.raises(ValueError, match="batch"):
        bd._validate_matmul(torch.zeros(2, 64, 128, dtype=bf), torch.zeros(3, 128, 96, dtype=bf), None, "KN", batched=True)
    with pytest.raises(TypeError):  # wrong operand dtype
        bd._validate_matmul(A.float(), torch.zeros(128, 96, dtype=bf), None, "KN")
    with pytest.raises(ValueError, match="operands are on"):
        bd._need_out(torch.zeros(64, 96, dtype=f32, device="meta"), (64, 96), A)
    with pytest.raises(ValueError, match="contiguous"):
        bd._need_out(torch.zeros(96, 64, dtype=f32).t(), (64, 96), A)
    # consistent shapes pass the shape checks and stop at the CUDA requirement
    with pytest.raises(TypeError, match="CUDA"):
        bd._validate_matmul(A, torch.zeros(128, 96, dtype=bf), torch.zeros(64, 96, dtype=f32), "KN")
    # the allocation-free entry point goes through the same checks before it calls the library
    with pytest.raises(ValueError, match="inner dimensions"):
        bd.gemm_splitk_static(A, torch.zeros(120, 96, dtype=bf), torch.zeros(64, 96, dtype=f32))
    with pytest.raises(ValueError, match="shape"):
        bd.gemm_splitk_static(A, torch.zeros(128, 96, dtype=bf), torch.zeros(64, 90, dtype=f32))
    with pytest.raises(TypeError):
        bd.gemm_splitk_static(A, torch.zeros(128, 96, dtype=bf), None)


def test_static_status_query_without_a_device(libfact):
    from ctypes import byref, c_int

    v = c_int(5)
    assert libfact.fact_gemm_splitk_static_status(0, None, byref(v)) == 0 and v.value == 0  # no call has run yet
    assert libfact.fact_gemm_splitk_static_status(-1, None, byref(v)) == 1
    assert libfact.fact_gemm_splitk_static_status(0, None, None) == 1
    assert libfact.fact_debug_flags(None) == 0


@pytest.mark.parametrize("ctas,bh,seq,hd", [(148, 192, 1024, 64), (148, 128, 2048, 128), (148, 20, 4000, 64),
                                            (7, 5, 1500, 128), (148, 149, 300, 64), (3, 1, 2048, 64)])
def test_attention_deal_gives_every_item_to_one_cta_and_balances_the_key_blocks(libfact, ctas, bh, seq, hd):
    """The host's deal of a causal attention problem (fact_attention_deal): every item goes to exactly one CTA, the
    first round is CTA c <- item c, and no CTA carries more than the mean plus one item's weight (what giving every
    item, heaviest first, to the CTA with the least so far guarantees)."""
    from paper_2604_26666_b200.binding import attention_deal

    bk = 128 if hd == 64 else 64
    q_pairs = (seq + 255) // 256
    items = bh * q_pairs
    kv_blocks = (seq + bk - 1) // bk

    def weight(idx):
        qp = q_pairs - 1 - idx // bh
        return min(kv_blocks, (qp * 256 + 255) // bk + 1) + (1.0 if bk == 128 else 2.0)

    per_cta = [attention_deal(ctas, bh, seq, hd, c) for c in range(ctas)]
    seen = sorted(i for lst in per_cta for i in lst)
    assert seen == list(range(items))
    for c in range(min(ctas, items)):
        assert per_cta[c][0] == c
    loads = [sum(weight(i) for i in lst) for lst in per_cta]
    mean = sum(loads) / ctas
    assert max(loads) <= mean + weight(0) + 1e-9
    # heaviest first inside every CTA
    for lst in per_cta:
        assert lst == sorted(lst)


def test_attention_deal_argument_errors(libfact):
    import ctypes

    n = ctypes.c_int(0)
    buf = (ctypes.c_int32 * 4)()
    assert libfact.fact_attention_deal(0, 4, 512, 64, 0, 4, buf, ctypes.byref(n)) == 1
    assert libfact.fact_attention_deal(4, 4, 512, 96, 0, 4, buf, ctypes.byref(n)) == 1
    assert libfact.fact_attention_deal(4, 4, 512, 64, 4, 4, buf, ctypes.byref(n)) == 1
    assert libfact.fact_attention_deal(4, 4, 512, 64, 0, 4, buf, None) == 1
    assert libfact.fact_attention_deal(148, 10000, 512, 64, 0, 4, buf, ctypes.byref(n)) == 3  # more than 8192 items
