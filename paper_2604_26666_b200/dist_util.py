"""Process-group plumbing for the multi-GPU benchmark: one process per GPU, no data-path collective.

The GEMM path shards by rows / batch entries with nothing to exchange, so the only
communication is a barrier around the timed region and a max-reduction of the per-rank
times (the job is as slow as its slowest rank).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple


def env_ranks() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) outside it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Initialise torch.distributed when WORLD_SIZE > 1.  Returns the module, or None for one process."""
    rank, world, _ = env_ranks()
    if world <= 1:
        return None
    import torch.distributed as dist

    if not dist.is_initialized():
        kw = {}
        if device is not None and backend == "nccl":
            kw["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return dist


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The largest `value` any rank holds (identity for a single process)."""
    if dist is None:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, seconds_per_rank: float, world: int, dist, device="cpu") -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: every rank does
    `units_per_rank`)."""
    return world * units_per_rank / max_over_ranks(seconds_per_rank, dist, device)


def shard_rows(total_rows: int, rank: int, world: int, multiple: int = 1) -> Tuple[int, int]:
    """[begin, end) of the rows rank `rank` owns when `total_rows` are split over `world` ranks in
    contiguous blocks whose sizes are multiples of `multiple` (the last rank takes the remainder)."""
    if world <= 0 or not (0 <= rank < world) or multiple <= 0:
        raise ValueError("bad rank/world/multiple")
    blocks = (total_rows + multiple - 1) // multiple
    per = (blocks + world - 1) // world
    begin = min(total_rows, rank * per * multiple)
    end = min(total_rows, (rank + 1) * per * multiple)
    return begin, end
