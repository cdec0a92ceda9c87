"""Host-side helpers for running the path on several GPUs.

Contexts (and with them every (context, head) attention unit) are independent, so the path
shards by contexts: each rank owns a contiguous slice of the global batch, holds a replica of
the datastore, and exchanges nothing on the data path.  Timing is the maximum over ranks."""
from __future__ import annotations


def shard_bounds(n_items: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of rank's contiguous slice; sizes differ by at most one, earlier ranks
    take the larger slices."""
    if world < 1 or not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(seconds: float, dist=None, device=None) -> float:
    """All-reduce(max) of a per-rank duration; identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(seconds)
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_step: int, steps: int, world: int, seconds_max: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank_step * steps * world / seconds_max
