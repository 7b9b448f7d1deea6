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


def free_port() -> int:
    """A TCP port that is free on 127.0.0.1 right now (for the rendezvous of a local launch)."""
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def launch_local(n_ranks: int, script: str, argv: Sequence[str], env=None) -> int:
    """Runs ``script argv`` as ``n_ranks`` processes of one node, one rank per GPU, the way the
    benchmark is launched for N > 1 (``python -m torch.distributed.run --nnodes=1 --nproc-per-node N``,
    rendezvous on 127.0.0.1).  Returns the launcher's exit code.  The ranks find RANK, LOCAL_RANK,
    WORLD_SIZE and MASTER_* in their environment."""
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(argv)
    return subprocess.call(cmd, env=env)
