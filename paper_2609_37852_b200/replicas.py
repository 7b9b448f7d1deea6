"""Multi-GPU helpers.  The attention path has no exchange step: every (batch, KV group) is an
independent unit, so N GPUs run N independent replicas (or disjoint shards of batch x KV heads)
and only the timing is reduced across ranks."""
from typing import Sequence, Tuple

import torch


def shard_units(n_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) range of independent units (batch x KV-head groups) owned by ``rank``;
    the first ``n_units % world_size`` ranks take one extra unit.  No unit is shared, so no data
    ever crosses ranks."""
    if not 0 <= rank < world_size:
        raise ValueError("rank outside the world")
    base, extra = divmod(n_units, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values: Sequence[float], device=None, group=None) -> list:
    """Element-wise maximum of per-rank timings (a job is as slow as its slowest rank).  Uses the
    default process group when one is initialised; otherwise returns the values unchanged."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return [float(x) for x in t.cpu()]


def aggregate_rate(work_per_rank: float, world_size: int, seconds_max: float) -> float:
    """Whole-job rate of ``world_size`` replicas that each did ``work_per_rank`` in at most ``seconds_max``."""
    return world_size * work_per_rank / seconds_max
