"""Multi-GPU plumbing of the benchmark: the path shards by images only (every GPU holds the whole encoded layers and
runs its own batch; there is no collective on the data path), so all that crosses ranks is timing bookkeeping."""
from __future__ import annotations

from typing import List, Sequence, Tuple


def shard_batch(total: int, world: int, rank: int) -> Tuple[int, int]:
    """Half-open image range [lo, hi) of `rank` when `total` images are split over `world` replicas."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(values: Sequence[float], device=None) -> List[float]:
    """Element-wise maximum of `values` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_value(units_per_rank: float, seconds_max: float, world: int) -> float:
    """Aggregate throughput of `world` replicas that each processed `units_per_rank` in at most `seconds_max`."""
    return world * units_per_rank / seconds_max
