"""The N > 1 plumbing on CPU: two gloo ranks agree on the max-over-ranks time and the whole-job rate,
and a row-sharded product assembled from the ranks' slabs equals the unsharded oracle (the path has
no exchange step, so sharding rows must change nothing)."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2604_26666_b200 import dist_util, workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import oracle

    dist = dist_util.init("gloo")
    assert dist is not None and dist.get_world_size() == world
    # every rank is timed differently; all must see the slowest
    mine = 1.0 + rank
    assert dist_util.max_over_ranks(mine, dist) == float(world)
    rate = dist_util.whole_job_rate(10.0, mine, world, dist)
    assert abs(rate - world * 10.0 / world) < 1e-12
    # a row shard of one problem, computed independently
    case = wl.Case("shard", "linear", 37, 24, 40, epilogue="BIAS", layout="NK", has_bias=True, seed=21)
    ins = wl.make_inputs(case)
    b, e = dist_util.shard_rows(case.M, rank, world, multiple=8)
    y = oracle.linear(wl.bits(ins.X)[b:e], wl.bits(ins.W), layout="NK", epilogue="BIAS", bias=wl.bits(ins.bias))
    np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    import oracle

    case = wl.Case("shard", "linear", 37, 24, 40, epilogue="BIAS", layout="NK", has_bias=True, seed=21)
    ins = wl.make_inputs(case)
    full = oracle.linear(wl.bits(ins.X), wl.bits(ins.W), layout="NK", epilogue="BIAS", bias=wl.bits(ins.bias))
    parts = [np.load(tmp_path / f"y{r}.npy") for r in range(world)]
    assert np.array_equal(np.concatenate(parts, axis=0), full)


def test_shard_rows_covers_everything_once():
    for total in (0, 1, 37, 128, 16384):
        for world in (1, 2, 3, 8):
            for mult in (1, 8, 128):
                spans = [dist_util.shard_rows(total, r, world, mult) for r in range(world)]
                assert spans[0][0] == 0 and spans[-1][1] == total
                for (b0, e0), (b1, e1) in zip(spans, spans[1:]):
                    assert e0 == b1 and b0 <= e0
                assert all((b % mult == 0) for b, _ in spans if b < total)


def test_single_process_is_identity():
    assert dist_util.init("gloo") is None
    assert dist_util.max_over_ranks(3.5, None) == 3.5
