"""GPU parity tests: libfact (through the C ABI binding) against the FP64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_26666_b200 import workloads as wl
from tests.helpers import check_case, gates, oracle_for, run_gpu, small_int_inputs, to_f64

pytestmark = pytest.mark.gpu

ALL_EPI = ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"]


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0)
    yield hd
    hd.close()


def mk(name, M, N, K, op="linear", epilogue="NONE", layout="KN", out="bf16", batch=1, seed=5, **kw):
    has_bias = epilogue in ("BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "BIAS_RESIDUAL")
    has_res = epilogue == "BIAS_RESIDUAL"
    return wl.Case(name, op, M, N, K, batch=batch, epilogue=epilogue, layout=layout, out=out, has_bias=has_bias,
                   has_residual=has_res, seed=seed, **kw)


def bit_exact(h, case, ins, cfg=None, splits=0):
    got = run_gpu(h, ins, case, cfg=cfg, splits=splits)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    ref = oracle_for(ins, case)
    if case.out == "bf16":
        want = np.vectorize(oracle.round_bf16, otypes=[np.uint16])(ref)
        gotb = wl.bits(got.cpu().contiguous())
        bad = np.argwhere(gotb != want)
    else:
        bad = np.argwhere(got.cpu().double().numpy() != ref)
    assert len(bad) == 0, f"{case.name}: {len(bad)} of {ref.size} elements differ, first at {bad[:5].tolist()}"


# ------------------------------------------------------------------ exact pins
@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_identity_is_bit_exact(h, layout):
    g = torch.Generator().manual_seed(1)
    M, K = 200, 256
    X = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = torch.eye(K).to(torch.bfloat16)
    case = mk("identity", M, K, K, layout=layout)
    got = run_gpu(h, wl.Inputs(X, W), case)
    assert torch.equal(got.cpu(), X)


@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("K", [64, 512, 768, 3072, 4096])
def test_all_ones_gives_K(h, layout, K):
    M, N = 130, 192
    X = torch.ones(M, K, dtype=torch.bfloat16)
    W = torch.ones((K, N) if layout == "KN" else (N, K), dtype=torch.bfloat16)
    got = run_gpu(h, wl.Inputs(X, W), mk("ones", M, N, K, layout=layout, out="f32"))
    assert (got.cpu() == float(K)).all()


@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_positional_probe(h, layout):
    # C[i, j] = (i % 7 + 1) * (j % 5 + 1) through a single k: locates any row/column/swizzle mix-up
    M, N, K = 256, 256, 128
    for k0 in (0, 5, 17, 63, 64, 127):
        A = torch.zeros(M, K)
        B = torch.zeros(K, N)
        A[:, k0] = (torch.arange(M) % 7 + 1).float()
        B[k0, :] = (torch.arange(N) % 5 + 1).float()
        W = B if layout == "KN" else B.t().contiguous()
        case = mk("probe", M, N, K, layout=layout, out="f32")
        got = run_gpu(h, wl.Inputs(A.to(torch.bfloat16), W.to(torch.bfloat16)), case).cpu()
        want = torch.outer(torch.arange(M) % 7 + 1, torch.arange(N) % 5 + 1).float()
        assert torch.equal(got, want), f"k0={k0}: {(got != want).sum().item()} wrong"


@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("out", ["bf16", "f32"])
def test_small_integers_bit_exact(h, layout, out):
    case = mk("ints", 300, 320, 1000 if layout == "NK" else 1000, layout=layout, out=out)
    bit_exact(h, case, small_int_inputs(case, 7))


# ------------------------------------------------------------------ epilogues, layouts, tails
@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("epi", ALL_EPI)
@pytest.mark.parametrize("out", ["bf16", "f32"])
def test_epilogues_ragged(h, layout, epi, out):
    # 3 m-tiles with a tail, 2 n-tiles with a tail, K not a multiple of 64
    case = mk(f"rag_{epi}", 300, 328, 520, epilogue=epi, layout=layout, out=out, w_scale=0.05)
    check_case(h, case)


@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("epi", ["BIAS_RELU", "SILU_GATE", "BIAS_RESIDUAL"])
def test_epilogue_exact_on_integers(h, layout, epi):
    # ReLU / residual on integer data are exact; SiLU is compared through the gate
    case = mk(f"int_{epi}", 140, 136, 200, epilogue=epi, layout=layout, out="f32")
    ins = small_int_inputs(case, 9, lo=-2, hi=2)
    if epi == "SILU_GATE":
        check_case(h, case, ins=ins)
    else:
        bit_exact(h, case, ins)


@pytest.mark.parametrize("tile_n", [32, 64, 96, 128, 192, 256])
@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_tile_widths(h, tile_n, layout):
    if layout == "KN" and tile_n % 64:
        pytest.skip("N-major B tiles are whole 64-column boxes")
    case = mk(f"tn{tile_n}", 260, 520, 384, epilogue="BIAS", layout=layout)
    check_case(h, case, cfg={"tile_n": tile_n})


@pytest.mark.parametrize("stages", [2, 3, 4, 6])
def test_stage_counts(h, stages):
    case = mk(f"st{stages}", 256, 256, 2048, layout="NK")
    check_case(h, case, cfg={"tile_n": 128, "stages": stages})


ROW_STORE_EPI = ["NONE", "BIAS", "BIAS_RELU", "BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"]


@pytest.mark.parametrize("epi", ROW_STORE_EPI)
@pytest.mark.parametrize("out", ["bf16", "f32"])
def test_register_row_stores(h, epi, out):
    """store_mode 3: the staged epilogue's arithmetic, rows stored from registers in 32-byte pieces.  Ragged M, two
    n-tiles with the second one partly past N, K not a multiple of 64; N a multiple of 32 bytes."""
    if out == "f32" and epi == "BIAS_RESIDUAL":
        pytest.skip("an FP32 output with a residual is not stageable")
    case = mk(f"rs_{epi}", 300, 336, 520, epilogue=epi, layout="NK", out=out, w_scale=0.05)
    check_case(h, case, cfg={"store_mode": 3, "tile_n": 256, "cta_group": 2})
    check_case(h, case, cfg={"store_mode": 3, "tile_n": 128, "cta_group": 1})


def test_register_row_stores_exact_batched_and_refusals(h):
    from paper_2604_26666_b200.binding import FactError
    case = mk("rs_int", 260, 256, 200, epilogue="BIAS_RESIDUAL", layout="KN", out="bf16")
    bit_exact(h, case, small_int_inputs(case, 11, lo=-2, hi=2), cfg={"store_mode": 3})
    caseb = mk("rs_batched", 200, 192, 136, op="gemm_batched", layout="NK", batch=3)
    check_case(h, caseb, cfg={"store_mode": 3})
    # refusals: rows that are not whole 32-byte pieces, K slices, stream-K
    for bad_case, cfg in ((mk("rs_n", 128, 200, 128, layout="NK"), {"store_mode": 3}),
                          (mk("rs_sp", 128, 256, 1024, layout="NK"), {"store_mode": 3, "split_k": 2}),
                          (mk("rs_sk", 300, 2304, 768, layout="NK"), {"store_mode": 3, "split_k": -1})):
        with pytest.raises(FactError) as e:
            run_gpu(h, wl.make_inputs(bad_case), bad_case, cfg=cfg)
        assert e.value.code == 3
    assert h.device_status() == 0


def test_unaligned_output_and_odd_sizes(h):
    # N odd: rows of C are not 16-byte aligned -> element-wise stores
    for (M, N, K) in [(1, 1, 8), (5, 7, 24), (129, 33, 72), (64, 250, 136)]:
        case = mk(f"odd_{M}_{N}_{K}", M, N, K, epilogue="BIAS_RESIDUAL", layout="NK")
        check_case(h, case)


def test_strided_operands(h):
    g = torch.Generator().manual_seed(3)
    M, N, K = 150, 200, 264
    Xbig = torch.randn(M, K + 24, generator=g).to(torch.bfloat16)
    Wbig = (torch.randn(N, K + 8, generator=g) * 0.1).to(torch.bfloat16)
    Cbig = torch.zeros(M, N + 16, dtype=torch.bfloat16, device="cuda")
    out = Cbig[:, :N]
    h.linear(Xbig.cuda()[:, :K], Wbig.cuda()[:, :K], layout="NK", out=out)
    torch.cuda.synchronize()
    ref = oracle.linear(wl.bits(Xbig)[:, :K], wl.bits(Wbig)[:, :K], layout="NK")
    c, t = gates(ref, to_f64(out), "bf16", "NONE")
    assert c <= 1 and t <= 1
    assert (Cbig[:, N:] == 0).all(), "wrote outside the N columns"


def test_table_entries_are_hints_for_less_aligned_outputs(h, tmp_path):
    """The tuner's table is keyed on the shape alone.  An entry that asks for staged tensor stores, 32-byte register
    row stores or K slices must not turn a call with a less aligned output, or without scratch, into an error: the
    library falls back to a store path (one K slice) that can run, and the result is still the oracle's."""
    from paper_2604_26666_b200.binding import Handle, lib
    import ctypes

    M, N, K = 384, 320, 2048 + 64
    path = tmp_path / "hints.txt"
    # op LINEAR(3) epilogue BIAS(1) layout NK(1) out BF16(0): staged stores; op GEMM(0): register row stores (mode 3);
    # op LINEAR with BIAS_RELU(2): 4 K slices
    path.write_text(f"3 1 1 0 1 {M} {N} {K} | 128 64 64 4 1 0 1 2\n"
                    f"0 0 0 0 1 {M} {N} {K} | 128 64 64 4 1 0 1 3\n"
                    f"3 2 1 0 1 {M} {N} {K} | 128 64 64 4 1 0 4 2\n")
    h2 = Handle(0, load_table=False)
    h2.tune_cache_load(str(path))
    dev = "cuda:0"
    # (a) staged entry, output with ldc = N + 2: rows are not 16-byte multiples
    case = mk("hint_staged", M, N, K, epilogue="BIAS", layout="NK")
    ins = wl.make_inputs(case)
    big = torch.zeros(M, N + 2, dtype=torch.bfloat16, device=dev)
    out = big[:, :N]
    h2.linear(ins.X.to(dev), ins.W.to(dev), bias=ins.bias.to(dev), epilogue="BIAS", layout="NK", out=out)
    torch.cuda.synchronize()
    assert h2.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", "BIAS")
    assert c <= 1 and t <= 1, (c, t)
    assert (big[:, N:] == 0).all()
    # (b) register-row-store entry, output 16-byte but not 32-byte aligned
    case = mk("hint_rows32", M, N, K, op="gemm", layout="KN")
    ins = wl.make_inputs(case)
    flat = torch.zeros(M * N + 8, dtype=torch.bfloat16, device=dev)
    out = flat[8:].view(M, N)
    assert out.data_ptr() % 32 == 16
    h2.gemm(ins.X.to(dev), ins.W.to(dev), layout="KN", out=out)
    torch.cuda.synchronize()
    assert h2.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", "NONE")
    assert c <= 1 and t <= 1, (c, t)
    assert (flat[:8] == 0).all()
    # (c) an entry with K slices, called through the raw C ABI without any workspace
    case = mk("hint_split", M, N, K, epilogue="BIAS_RELU", layout="NK")
    ins = wl.make_inputs(case)
    X, W, b = ins.X.to(dev), ins.W.to(dev), ins.bias.to(dev)
    out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    vp = ctypes.c_void_p
    rc = lib().fact_linear(h2._h, M, N, K, vp(X.data_ptr()), K, vp(W.data_ptr()), K, 1, vp(b.data_ptr()), None, 0,
                           vp(out.data_ptr()), N, 0, 2, None, None, 0, vp(torch.cuda.current_stream(0).cuda_stream))
    assert rc == 0, rc
    torch.cuda.synchronize()
    assert h2.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", "BIAS_RELU")
    assert c <= 1 and t <= 1, (c, t)
    # a caller's own configuration is still refused where it cannot run
    with pytest.raises(Exception):
        h2.linear(X, W, bias=b, epilogue="BIAS_RELU", layout="NK", out=big[:, :N], cfg={"store_mode": 2})
    h2.close()


# ------------------------------------------------------------------ batched and split-K
@pytest.mark.parametrize("layout", ["KN", "NK"])
def test_batched(h, layout):
    case = mk("batched", 136, 200, 264, op="gemm_batched", batch=5, layout=layout)
    check_case(h, case)


@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("splits", [0, 2, 7, 16])
def test_splitk_parity_and_determinism(h, layout, splits):
    case = mk("splitk", 256, 256, 8192 + 64, op="gemm_splitk", layout=layout, out="f32",
              x_dist="uniform", w_dist="uniform")
    ins = wl.make_inputs(case)
    check_case(h, case, splits=splits, ins=ins)
    a = run_gpu(h, ins, case, splits=splits).clone()
    for _ in range(3):
        b = run_gpu(h, ins, case, splits=splits)
        assert torch.equal(a, b), "split-K result changed between runs"


def test_splitk_exact_on_integers_for_any_split(h):
    case = mk("splitk_int", 200, 136, 4096, op="gemm_splitk", layout="KN", out="f32")
    ins = small_int_inputs(case, 11)
    for s in (1, 3, 8, 64):
        bit_exact(h, case, ins, splits=s)


def test_splitk_with_epilogue_through_linear(h):
    for epi in ("BIAS_GELU_TANH", "SILU_GATE", "BIAS_RESIDUAL"):
        case = mk(f"lin_split_{epi}", 200, 264, 2048, epilogue=epi, layout="NK", w_scale=0.05)
        check_case(h, case, cfg={"split_k": 5})


@pytest.mark.parametrize("out", ["bf16", "f32"])
def test_few_slices_take_the_wide_reduction_and_keep_every_bit(h, out):
    """With eight slices or fewer one thread adds all slices of 8 adjacent columns (vector or element-wise stores, a
    ragged last group); with more, four lanes share a group of 4.  Integer inputs: both must equal the oracle bit for
    bit, for aligned and unaligned outputs, with bias and residual."""
    for (M, N, K, epi) in [(200, 136, 2048, "BIAS_RESIDUAL"), (130, 102, 1024, "BIAS_RELU"), (64, 1030, 512, "BIAS")]:
        case = mk(f"wide_{N}_{epi}", M, N, K, epilogue=epi, layout="NK", out=out)
        ins = small_int_inputs(case, 21, lo=-2, hi=2)
        ref = oracle_for(ins, case)
        for splits in (2, 3, 8, 9):
            for pad in (0, 3):  # pad 3: rows of the output are not 16-byte aligned
                dt = torch.float32 if out == "f32" else torch.bfloat16
                big = torch.full((M, N + pad), -7.0, dtype=dt, device="cuda")
                got = run_gpu(h, ins, case, cfg={"split_k": splits}, out=big[:, :N])
                torch.cuda.synchronize()
                assert h.device_status() == 0
                if out == "bf16":
                    want = np.vectorize(oracle.round_bf16, otypes=[np.uint16])(ref)
                    bad = np.argwhere(wl.bits(got.cpu().contiguous()) != want)
                else:
                    bad = np.argwhere(got.cpu().double().numpy() != ref)
                assert len(bad) == 0, (case.name, splits, pad, len(bad), bad[:4].tolist())
                if pad:
                    assert (big[:, N:] == -7.0).all(), "wrote outside the N columns"


@pytest.mark.parametrize("layout", ["KN", "NK"])
@pytest.mark.parametrize("pair,slices,tile_n", [(1, 2, 64), (1, 2, 128), (1, 4, 128), (1, 2, 256), (1, 4, 256), (1, 8, 256),
                                                (2, 2, 64), (2, 2, 128), (2, 4, 128), (2, 2, 256), (2, 4, 256)])
def test_k_slices_as_a_cluster_are_exact_and_equal_the_workspace_reduction(h, layout, pair, slices, tile_n):
    """schedule 3: the K slices of a tile run as one cluster (each slice a CTA on a 128-row tile, or a CTA pair on a
    256-row tile) and are added up through distributed shared memory, in
    the order of the workspace reduction.  Integer inputs: bit-exact against the oracle, for every epilogue the
    schedule serves, several tiles per cluster (more tiles than clusters), ragged M, N and K, FP32 and BF16 outputs;
    random inputs: the same bits as the same number of slices through the workspace."""
    from paper_2604_26666_b200.binding import FactError

    kc = {"cta_group": pair, "tile_n": tile_n, "split_k": slices, "schedule": 3}
    if pair == 2 and tile_n == 64 and layout == "KN":
        # (each CTA of a pair loads half the tile's columns of B; a [K, N] operand has no 32-column box)
        case = mk("kc_pair_kn_64", 256, 256, 1024, layout=layout)
        with pytest.raises(FactError):
            run_gpu(h, wl.make_inputs(case), case, cfg=kc)
        return
    for (M, N, K, epi, out) in [(200, 520, 1096, "BIAS_RESIDUAL", "bf16"), (130, 264, 2048, "BIAS_RELU", "f32"),
                                (128 * 40 + 8, 512, 1024, "NONE", "bf16")]:
        case = mk(f"kc_{pair}_{slices}_{tile_n}_{epi}", M, N, K, epilogue=epi, layout=layout, out=out)
        bit_exact(h, case, small_int_inputs(case, 31, lo=-2, hi=2), cfg=kc)
    case = mk(f"kc_rand_{pair}_{slices}_{tile_n}", 300, 520, 4096, epilogue="BIAS_GELU_TANH", layout=layout)
    ins = wl.make_inputs(case)
    check_case(h, case, ins=ins, cfg=kc)
    a = run_gpu(h, ins, case, cfg=kc)
    b = run_gpu(h, ins, case, cfg={"cta_group": pair, "tile_n": tile_n, "split_k": slices})
    torch.cuda.synchronize()
    assert torch.equal(a, b), "cluster and workspace reductions of the same slices differ"
    assert h.workspace_bytes("linear", 1, 300, 520, 4096, "BIAS_GELU_TANH", layout, torch.bfloat16, kc) == 0
    # what the schedule does not serve is refused before any launch
    gate = mk("kc_gate", 128, 256, 1024, epilogue="SILU_GATE", layout=layout)
    with pytest.raises(FactError):
        run_gpu(h, wl.make_inputs(gate), gate, cfg=kc)
    # (a cluster holds at most 8 CTAs: 8 slices of pairs would be 16)
    for bad in ({"cta_group": 2, "split_k": 8, "tile_n": 256}, {"split_k": 3}, {"tile_n": 96}):
        with pytest.raises(FactError):
            run_gpu(h, ins, case, cfg={**kc, **bad})
    assert h.device_status() == 0


@pytest.mark.parametrize("pair", [1, 2])
def test_k_slices_as_a_cluster_serve_the_batched_and_the_sliced_entry_points(h, pair):
    kc = {"cta_group": pair, "tile_n": 128, "split_k": 4, "schedule": 3}
    for layout in ("KN", "NK"):
        case = mk("kc_batched", 200, 264, 1536, op="gemm_batched", batch=5, layout=layout, out="f32")
        bit_exact(h, case, small_int_inputs(case, 41, lo=-2, hi=2), cfg=kc)
        case = mk("kc_splitk_op", 256, 256, 8192 + 64, op="gemm_splitk", layout=layout, out="f32")
        bit_exact(h, case, small_int_inputs(case, 42, lo=-2, hi=2), cfg=kc, splits=4)
    assert h.device_status() == 0


@pytest.mark.parametrize("pair", [1, 2])
def test_k_slices_as_a_cluster_in_a_cuda_graph_and_back_to_back(h, pair):
    """Cluster launches can be captured and replayed, and launches that follow one another on a stream (each may move
    onto the SMs while its predecessor's last CTAs leave) -- of the cluster kernel and of the persistent kernel in
    turn -- give the same bits every time."""
    case = mk("kc_graph", 384, 512, 4096, epilogue="BIAS_RELU", layout="NK")
    ins = wl.make_inputs(case)
    X, W, b = ins.X.cuda(), ins.W.cuda(), ins.bias.cuda()
    kc = {"cta_group": pair, "tile_n": 128, "split_k": 4, "schedule": 3}
    first_kc = h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", cfg=kc)
    first_dp = h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", cfg={"split_k": 1})
    torch.cuda.synchronize()
    out_kc, out_dp = torch.empty_like(first_kc), torch.empty_like(first_dp)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream("cuda:0")):
        for _ in range(3):
            h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", out=out_kc, cfg=kc)
            h.linear(X, W, bias=b, epilogue=case.epilogue, layout="NK", out=out_dp, cfg={"split_k": 1})
    for _ in range(3):
        out_kc.zero_()
        out_dp.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out_kc, first_kc) and torch.equal(out_dp, first_dp)
    assert h.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out_kc), "bf16", case.epilogue)
    assert c <= 1 and t <= 1, (c, t)


def test_untuned_few_tiles_long_k_takes_k_slices_when_it_has_the_scratch(h):
    """The library's own choice for an untuned product of few tiles and long K is K slices (Section 4.2, Action 2:
    the grid-level policy is a design choice) -- with the workspace the binding brings; the same call through the C
    ABI without a workspace runs in one slice.  Both are checked against the oracle."""
    import ctypes

    from paper_2604_26666_b200.binding import lib

    case = mk("few_tiles_long_k", 256, 512, 16384, op="gemm", layout="NK")
    cfg = h.get_config("gemm", 1, case.M, case.N, case.K, "NONE", "NK", torch.bfloat16).as_dict()
    assert cfg["split_k"] > 1, cfg
    # (slices through the workspace, or -- schedule 3 -- as a cluster, which needs none)
    assert (h.workspace_bytes("gemm", 1, case.M, case.N, case.K, "NONE", "NK", torch.bfloat16) > 0) != (cfg["schedule"] == 3)
    ins = wl.make_inputs(case)
    check_case(h, case, ins=ins)
    # an explicit single slice is respected, and a short K is never sliced
    assert h.get_config("gemm", 1, 256, 512, 512, "NONE", "NK", torch.bfloat16).as_dict()["split_k"] == 1
    X, W = ins.X.cuda(), ins.W.cuda()
    out = torch.full((case.M, case.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    rc = lib().fact_gemm(h._h, case.M, case.N, case.K, ctypes.c_void_p(X.data_ptr()), X.stride(0),
                         ctypes.c_void_p(W.data_ptr()), W.stride(0), 1, ctypes.c_void_p(out.data_ptr()), out.stride(0), 0,
                         None, None, 0, None)
    assert rc == 0, rc
    torch.cuda.synchronize()
    assert h.device_status() == 0
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", "NONE")
    assert c <= 1.0 and t <= 1.0, (c, t)


def test_diagnostic_switches_change_no_bit(h, monkeypatch):
    """FACT_DEBUG_FLAGS (read once, when a handle is created): without the downward K walk of every second tile the
    sums of those tiles are taken in the other order, which integer inputs do not see; without programmatic dependent
    launch and without the L2 eviction priority of the operand loads nothing about the arithmetic changes at all, so
    random inputs give the same bits.  The default build masks every other bit."""
    from paper_2604_26666_b200.binding import Handle

    case = mk("diag", 1100, 1032, 2048 + 72, epilogue="BIAS_GELU_TANH", layout="NK")
    ins = wl.make_inputs(case)
    ints = small_int_inputs(case, 77, lo=-2, hi=2)
    want = run_gpu(h, ins, case).clone()
    want_int = run_gpu(h, ints, case).clone()
    for flags in (2048, 4096, 8192, 4096 | 8192, 1 | 2 | 4):
        monkeypatch.setenv("FACT_DEBUG_FLAGS", str(flags))
        h2 = Handle(0)
        try:
            assert h2.debug_flags() == (flags & (256 | 2048 | 4096 | 8192))
            if not flags & 2048:
                assert torch.equal(run_gpu(h2, ins, case), want), flags
            assert torch.equal(run_gpu(h2, ints, case), want_int), flags
            torch.cuda.synchronize()
            assert h2.device_status() == 0
        finally:
            h2.close()


# ------------------------------------------------------------------ degenerate sizes
def test_empty_and_k_zero(h):
    dev = "cuda:0"
    A = torch.zeros(0, 64, dtype=torch.bfloat16, device=dev)
    B = torch.zeros(64, 32, dtype=torch.bfloat16, device=dev)
    assert h.gemm(A, B).shape == (0, 32)
    # K == 0: the epilogue of a zero accumulator
    X = torch.zeros(10, 0, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(24, 0, dtype=torch.bfloat16, device=dev)
    bias = torch.arange(24, dtype=torch.float32).to(torch.bfloat16).to(dev)
    y = h.linear(X, W, bias=bias, epilogue="BIAS_RELU", layout="NK")
    assert torch.equal(y.cpu(), bias.cpu().expand(10, 24))


# ------------------------------------------------------------------ host-side error paths
def test_error_codes(h):
    from paper_2604_26666_b200.binding import FactError
    dev = "cuda:0"
    A = torch.zeros(64, 72, dtype=torch.bfloat16, device=dev)
    B = torch.zeros(72, 64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(FactError) as e:
        h.gemm(A[:, 1:65], B[:64])  # operand pointer not 16-byte aligned
    assert e.value.code == 2
    with pytest.raises(FactError) as e:
        h.linear(A, B, epilogue="BIAS", layout="KN")  # missing bias
    assert e.value.code == 1
    with pytest.raises(FactError) as e:
        h.gemm(A, B, cfg={"tile_n": 48})  # not a multiple of 32
    assert e.value.code == 3
    with pytest.raises(FactError) as e:
        h.gemm(A, B, cfg={"tile_n": 256, "stages": 8})  # over the shared-memory budget
    assert e.value.code == 3
    # split-K without enough workspace, through the raw C entry point
    from ctypes import c_void_p
    from paper_2604_26666_b200.binding import lib
    C = torch.zeros(64, 64, dtype=torch.float32, device=dev)
    rc = lib().fact_gemm_splitk(h._h, 64, 64, 72, c_void_p(A.data_ptr()), 72, c_void_p(B.data_ptr()), 64, 0,
                                c_void_p(C.data_ptr()), 64, 1, 2, None, None, 0, None)
    assert rc == 5
    assert (C == 0).all()


# ------------------------------------------------------------------ bounded waits, tuner, raster direction
def test_an_expired_device_wait_is_reported_and_the_context_survives(h):
    """Nothing is hung or faulted: a warp waits on a barrier that is never completed, with a 5 ms limit."""
    assert h.device_status() == 0
    h.selftest_wait_timeout(5.0)
    assert h.device_status() == 7  # FACT_ERR_DEVICE_TIMEOUT, reported once ...
    assert h.device_status() == 0  # ... and cleared
    case = mk("after_timeout", 200, 264, 520, epilogue="BIAS", layout="NK")
    check_case(h, case)  # the handle and the context still work


def test_raster_along_n_and_along_m_agree(h):
    case = mk("raster", 1100, 1300, 264, layout="NK")
    ins = wl.make_inputs(case)
    outs = [run_gpu(h, ins, case, cfg={"raster_group": g, "tile_n": 128, "cta_group": 1}).clone() for g in (1, 3, -1, -4)]
    for o in outs[1:]:
        assert torch.equal(outs[0], o)  # the raster changes the order of tiles, never a value
    check_case(h, case, cfg={"raster_group": -3}, ins=ins)


def test_tuner_returns_a_runnable_config_and_the_table_round_trips(h, tmp_path):
    case = mk("tune", 512, 384, 520, epilogue="BIAS_RELU", layout="NK")
    ins = wl.make_inputs(case)
    dev = "cuda:0"
    X, W, b = ins.X.to(dev), ins.W.to(dev), ins.bias.to(dev)
    cfg, ms, n = h.tune("linear", X, W, layout="NK", bias=b, epilogue="BIAS_RELU", warmup=2, iters=5)
    assert n >= 4 and ms > 0
    d = cfg.as_dict()
    assert d["tile_m"] == 128 * d["cta_group"] and d["tile_n"] % 32 == 0 and d["stages"] >= 2
    got = h.get_config("linear", 1, case.M, case.N, case.K, "BIAS_RELU", "NK").as_dict()
    assert {k: got[k] for k in ("tile_n", "cta_group", "stages", "split_k")} == \
           {k: d[k] for k in ("tile_n", "cta_group", "stages", "split_k")}
    check_case(h, case, ins=ins)  # runs with the tuned entry
    path = tmp_path / "table.txt"
    h.tune_cache_save(str(path))
    from paper_2604_26666_b200.binding import Handle
    h2 = Handle(0, load_table=False)
    before = h2.get_config("linear", 1, case.M, case.N, case.K, "BIAS_RELU", "NK").as_dict()
    h2.tune_cache_load(str(path))
    after = h2.get_config("linear", 1, case.M, case.N, case.K, "BIAS_RELU", "NK").as_dict()
    assert {k: after[k] for k in ("tile_n", "cta_group", "stages")} == {k: d[k] for k in ("tile_n", "cta_group", "stages")}
    assert isinstance(before, dict)
    h2.close()


def test_tuner_verifies_before_it_times_and_records_every_candidate(h):
    """Section 4.2: verify, then benchmark.  Every candidate's output is compared on the device with the default
    configuration's before it is timed; the record says what happened to each.  The gate itself is tested by letting
    one candidate (a correct one) be compared with a deliberately wrong reference: it must be rejected, untimed."""
    case = mk("tune_gate", 640, 384, 1024 + 64, epilogue="BIAS_GELU_TANH", layout="NK")
    ins = wl.make_inputs(case)
    dev = "cuda:0"
    X, W, b = ins.X.to(dev), ins.W.to(dev), ins.bias.to(dev)
    out = torch.empty(case.M, case.N, dtype=torch.bfloat16, device=dev)
    cfg, ms, n, recs = h.tune("linear", X, W, layout="NK", bias=b, epilogue=case.epilogue, out=out, warmup=1, iters=3,
                              records=True)
    outcomes = [r["outcome"] for r in recs]
    assert n == outcomes.count("timed") and n >= 4
    assert "verify_failed" not in outcomes and "launch_failed" not in outcomes
    assert all(0 <= r["verify_err"] <= 1 and r["ms"] > 0 and r["rel"] > 0 for r in recs if r["outcome"] == "timed")
    assert all(r["ms"] < 0 for r in recs if r["outcome"] != "timed")
    # the output is left holding the winner's result: the oracle's, within the gates
    torch.cuda.synchronize()
    c, t = gates(oracle_for(ins, case), to_f64(out), "bf16", case.epilogue)
    assert c <= 1 and t <= 1, (c, t)
    # the gate's own test: the k-th feasible candidate is checked against a wrong reference
    k = outcomes.index("timed")
    cfg2, ms2, n2, recs2 = h.tune("linear", X, W, layout="NK", bias=b, epilogue=case.epilogue, out=out, warmup=1,
                                  iters=3, records=True, inject_fault=k)
    assert recs2[k]["outcome"] == "verify_failed" and recs2[k]["verify_err"] > 1 and recs2[k]["ms"] < 0
    assert n2 == n - 1 and [r["outcome"] for i, r in enumerate(recs2) if i != k] == \
           [o for i, o in enumerate(outcomes) if i != k]
    # cold-L2 timing and FP32 output through the same gate
    case3 = mk("tune_gate_f32", 256, 256, 8192, op="gemm_splitk", layout="KN", out="f32", x_dist="uniform",
               w_dist="uniform")
    ins3 = wl.make_inputs(case3)
    cfg3, ms3, n3, recs3 = h.tune("gemm_splitk", ins3.X.to(dev), ins3.W.to(dev), layout="KN",
                                  out_dtype=torch.float32, warmup=1, iters=3, cold_l2=True, records=True)
    assert n3 >= 2 and "verify_failed" not in [r["outcome"] for r in recs3]
    check_case(h, case3, ins=ins3)  # runs with the tuned entry
