"""Parity of the stream-K schedule (config.split_k = -1 / -2; the paper's third grid-level policy, Section 4.2,
Action 2) against the FP64 oracle, through the C ABI.

Shapes are chosen so that a small problem still has full data-parallel waves plus a partial wave on a 148-SM
part (narrow tiles), tiles whose pieces span two, three and many CTAs, ragged edges in M, N and K, and every
epilogue.  Integer-valued inputs make every partial sum exact in FP32, so there a dropped or doubled piece
shows as an exact mismatch, not as a tolerance question.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2604_26666_b200 import workloads as wl
from tests.helpers import check_case, oracle_for, run_gpu, small_int_inputs, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    from paper_2604_26666_b200.binding import Handle
    hd = Handle(0, load_table=False)
    yield hd
    hd.close()


def cfg(tile_n, cg, mode, stages=0):
    return dict(tile_m=128 * cg, tile_n=tile_n, tile_k=64, stages=stages, cta_group=cg, raster_group=0,
                split_k=mode, store_mode=0)


def uses_stream_k(h, case, c):
    """The workspace query says whether the library will cut tiles for this problem."""
    odt = torch.float32 if case.out == "f32" else torch.bfloat16
    op = {"gemm": "gemm", "gemm_batched": "gemm_batched", "linear": "linear"}[case.op]
    return h.workspace_bytes(op, case.batch, case.M, case.N, case.K, case.epilogue, case.layout, odt, c) > 0


LINEAR = [
    # name, M, N, K, epilogue, tile_n, cta_group, mode
    ("gelu_1cta_partial_wave", 1280, 1280, 520, "BIAS_GELU_TANH", 64, 1, -1),     # 200 tiles on 148 CTAs, ragged K
    ("bias_1cta_two_waves", 1300, 1288, 512, "BIAS", 64, 1, -2),                   # ragged M and N: 11 x 21 tiles, all cut
    ("relu_2cta_partial_wave", 1280, 1280, 448, "BIAS_RELU", 64, 2, -1),           # 100 pair tiles on 74 pairs
    ("residual_2cta_all_tiles", 1280, 1280, 448, "BIAS_RESIDUAL", 64, 2, -2),      # 26 + 74: every tile is cut
    ("residual_1cta_fewer_tiles_than_ctas", 1150, 704, 1104, "BIAS_RESIDUAL", 64, 1, -1),
    ("silu_gate_2cta", 1280, 1280, 384, "SILU_GATE", 128, 2, -1),                  # 64 gate + 64 up columns per tile
    ("silu_gate_1cta", 2200, 672, 304, "SILU_GATE", 128, 1, -1),                   # 18 x 11 tiles
    ("none_wide_tiles", 2560, 2304, 512, "NONE", 256, 2, -1),                      # 90 tiles of 256 x 256
    ("few_tiles_many_pieces", 256, 512, 4096, "BIAS", 256, 2, -1),                 # 2 tiles over 74 pairs: 37 pieces each
    ("one_tile_all_ctas", 128, 256, 9600, "NONE", 256, 1, -1),                     # 1 tile, 148 CTAs, 150 k-blocks
]


@pytest.mark.parametrize("name,M,N,K,epi,tile_n,cg,mode", LINEAR, ids=[c[0] for c in LINEAR])
def test_stream_k_linear_matches_oracle(h, name, M, N, K, epi, tile_n, cg, mode):
    case = wl.Case(name, "linear", M, N, K, epilogue=epi, layout="NK", has_bias=epi.startswith("BIAS"),
                   has_residual=epi == "BIAS_RESIDUAL", seed=11, w_scale=K ** -0.5)
    c = cfg(tile_n, cg, mode)
    assert uses_stream_k(h, case, c), "the shape was meant to have a partial wave"
    check_case(h, case, cfg=c)


@pytest.mark.parametrize("layout,out", [("KN", "f32"), ("KN", "bf16"), ("NK", "f32")])
def test_stream_k_gemm_layouts_and_outputs(h, layout, out):
    case = wl.Case("sk_gemm", "gemm", 1408, 1216, 712, layout=layout, out=out, seed=12, x_scale=712 ** -0.5)
    for c in (cfg(64, 1, -1), cfg(128, 2, -1), cfg(128, 2, -2)):
        assert uses_stream_k(h, case, c)
        check_case(h, case, cfg=c)


def test_stream_k_batched(h):
    case = wl.Case("sk_batched", "gemm_batched", 384, 320, 576, batch=13, layout="KN", seed=13, x_scale=576 ** -0.5)
    c = cfg(64, 1, -1)  # 13 x 3 x 5 = 195 tiles
    assert uses_stream_k(h, case, c)
    check_case(h, case, cfg=c)


@pytest.mark.parametrize("tile_n,cg,mode", [(32, 1, -1), (64, 2, -1), (64, 2, -2), (256, 2, -1)])
def test_stream_k_is_exact_on_integer_inputs_and_repeatable(h, tile_n, cg, mode):
    """Small-integer operands: every product and every partial sum is an integer below 2^24, so FP32 is exact
    whatever the order -- the stream-K result must EQUAL the oracle's, and a second call the first."""
    case = wl.Case("sk_int", "gemm", 1536, 1312, 840, layout="NK", out="f32", seed=14)
    ins = small_int_inputs(case, seed=14)
    c = cfg(tile_n, cg, mode)
    assert uses_stream_k(h, case, c)
    got = run_gpu(h, ins, case, cfg=c)
    again = run_gpu(h, ins, case, cfg=c)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    ref = oracle_for(ins, case)
    assert np.array_equal(to_f64(got), ref)
    assert torch.equal(got, again)


def test_stream_k_equals_data_parallel_bits_where_no_tile_is_cut(h):
    """Rows of tiles that stay data-parallel are computed by the same code as without stream-K: identical bits.
    And normal-valued inputs repeat bit for bit (the order of the partial sums is fixed)."""
    case = wl.Case("sk_bits", "linear", 2048, 1024, 640, epilogue="BIAS_GELU_TANH", layout="NK", has_bias=True,
                   seed=15, w_scale=640 ** -0.5)
    ins = wl.make_inputs(case)
    sk = cfg(64, 1, -1)  # 16 x 16 = 256 tiles: 148 data-parallel, 108 cut
    dp = cfg(64, 1, 1)
    assert uses_stream_k(h, case, sk)
    a = run_gpu(h, ins, case, cfg=sk)
    b = run_gpu(h, ins, case, cfg=sk)
    d = run_gpu(h, ins, case, cfg=dp)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    assert torch.equal(a, b)
    n_tiles_n = 1024 // 64
    dp_tiles = 148  # the first 148 tiles in raster order are not cut; compare a block that lies inside them
    info = h.device_info()
    if info["sm_count"] == 148:
        # raster groups walk m-tiles fastest inside a group; whatever the order, at least the tiles of one full
        # row-block of 128 rows x 64 columns agree wherever both runs used the same summation order.  Check the
        # share of identical elements instead of guessing the raster: the uncut tiles are 148 / 256 of the output.
        same = (a == d).float().mean().item()
        assert same >= dp_tiles / (16 * n_tiles_n) - 1e-6, same


def test_stream_k_without_partial_wave_is_data_parallel(h):
    info = h.device_info()
    sms = info["sm_count"]
    case = wl.Case("sk_whole_waves", "gemm", 128 * sms, 64, 192, layout="NK", out="bf16", seed=16)
    c = cfg(64, 1, -1)  # exactly one wave: nothing to cut
    assert not uses_stream_k(h, case, c)
    check_case(h, case, cfg=c)


def test_stream_k_unaligned_output_falls_back_to_data_parallel(h):
    # ldc = 650 elements: rows are not 16-byte multiples, the staged store cannot write them
    case = wl.Case("sk_unaligned", "gemm", 1280, 650, 256, layout="NK", out="bf16", seed=17, x_scale=1 / 16)
    check_case(h, case, cfg=cfg(64, 1, -1))
    # a tile width the staged store does not handle for BF16 outputs: no scratch is asked for, the call still works
    case = wl.Case("sk_narrow", "gemm", 1280, 640, 256, layout="NK", out="bf16", seed=17, x_scale=1 / 16)
    assert not uses_stream_k(h, case, cfg(32, 1, -1))
    check_case(h, case, cfg=cfg(32, 1, -1))


def test_stream_k_workspace_errors(h):
    from paper_2604_26666_b200.binding import Config, lib, _ptr, _ld

    M, N, K = 1280, 1280, 512
    A = torch.randn(M, K, device="cuda").bfloat16()
    B = torch.randn(N, K, device="cuda").bfloat16()
    C = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
    c = Config(**cfg(64, 1, -1))
    need = h.workspace_bytes("gemm", 1, M, N, K, "NONE", "NK", torch.bfloat16, c)
    info = h.device_info()
    assert need == info["sm_count"] * 128 * 64 * 4
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    call = lambda wptr, wbytes, cc: lib().fact_gemm(h._h, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), 1, _ptr(C), _ld(C),
                                                   0, cc, wptr, wbytes, s)
    assert call(None, 0, ctypes.byref(c)) == 5          # FACT_ERR_WORKSPACE_TOO_SMALL
    assert call(_ptr(ws), need - 1, ctypes.byref(c)) == 5
    assert call(ctypes.c_void_p(ws.data_ptr() + 4), need, ctypes.byref(c)) in (2, 5)  # misaligned scratch
    bad = Config(**cfg(64, 1, -3))
    assert call(_ptr(ws), need, ctypes.byref(bad)) == 1  # FACT_ERR_INVALID_ARG
    assert call(_ptr(ws), need, ctypes.byref(c)) == 0
    torch.cuda.synchronize()
    assert h.device_status() == 0
    ref = (A.float() @ B.float().T)
    assert torch.allclose(C.float(), ref, rtol=2e-2, atol=2e-1)


def test_stream_k_replays_in_a_cuda_graph(h):
    """The flags are cleared by their reader, not by the host, so a captured launch can be replayed: three replays
    on three different inputs each give that input's product."""
    case = wl.Case("sk_graph", "gemm", 1536, 1312, 448, layout="NK", out="f32", seed=18)
    c = cfg(64, 2, -1)
    assert uses_stream_k(h, case, c)
    inputs = [small_int_inputs(case, seed=100 + i) for i in range(3)]
    X = inputs[0].X.cuda().clone()
    W = inputs[0].W.cuda().clone()
    out = torch.empty(case.M, case.N, device="cuda", dtype=torch.float32)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        h.gemm(X, W, layout="NK", out=out, cfg=c, stream=side)  # allocates the workspace outside the capture
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            h.gemm(X, W, layout="NK", out=out, cfg=c, stream=side)
    torch.cuda.synchronize()
    for ins in inputs:
        X.copy_(ins.X)
        W.copy_(ins.W)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert h.device_status() == 0
        assert np.array_equal(out.double().cpu().numpy(), oracle_for(ins, case))


def test_tuned_stream_k_entry_without_scratch_runs_data_parallel(tmp_path):
    """A table entry may say stream-K while a caller (a block chain, say) brings no workspace: the library then
    runs the same tiles data-parallel instead of failing; with an explicit config the missing scratch is an error
    (test_stream_k_workspace_errors)."""
    from paper_2604_26666_b200.binding import Handle, lib, _ptr, _ld

    M, N, K = 1280, 1280, 512
    table = tmp_path / "table.txt"
    table.write_text(f"0 0 1 0 1 {M} {N} {K} | 128 64 64 0 1 0 -1 0\n")
    hd = Handle(0, load_table=False)
    try:
        hd.tune_cache_load(str(table))
        assert hd.get_config("gemm", 1, M, N, K, "NONE", "NK", torch.bfloat16).as_dict()["split_k"] == -1
        assert hd.workspace_bytes("gemm", 1, M, N, K, "NONE", "NK", torch.bfloat16) > 0
        case = wl.Case("sk_table", "gemm", M, N, K, layout="NK", out="f32", seed=19)
        ins = small_int_inputs(case, seed=19)
        A, B = ins.X.cuda(), ins.W.cuda()
        C = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
        s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        rc = lib().fact_gemm(hd._h, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), 1, _ptr(C), _ld(C), 0, None, None, 0, s)
        assert rc == 0
        torch.cuda.synchronize()
        assert hd.device_status() == 0
        with_ws = hd.gemm(A, B, layout="NK", out_dtype=torch.bfloat16)  # the binding brings the scratch: stream-K
        torch.cuda.synchronize()
        assert hd.device_status() == 0
        ref = torch.from_numpy(oracle_for(ins, case)).to(torch.bfloat16)  # integers: exact before the BF16 rounding
        assert torch.equal(C.cpu(), ref) and torch.equal(with_ws.cpu(), ref)
    finally:
        hd.close()
