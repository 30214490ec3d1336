"""Multi-GPU plumbing of the benchmark and of data-parallel use: one process per GPU, batches are
independent (the layer's statistics are per-GPU batch statistics), so ranks share nothing on the data
path.  The only exchanges are the max-over-ranks of a device time and the split of work units."""
from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment (torch.distributed.run)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def shard_units(total: int, rank: int, world: int):
    """[begin, end) of the `total` independent units (images, problems) that `rank` processes: contiguous,
    sizes differ by at most one, the union over ranks is exactly range(total)."""
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time (all-reduce MAX); identity for a single process."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
