"""One process per GPU: rank bookkeeping for the benchmark's N > 1 runs.

One problem's traces share one pool and the prune decision is global to it, so the hot path has no
exchange step between GPUs: N GPUs run N independent problems (replicas).  What the ranks do share is
the measurement: a barrier on both sides of the timed region, the MAX over ranks of every time, the MIN
of the health flag.  The helpers below work on any torch.distributed backend (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def rank_env():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(values, ok: bool, device):
    """Every time in `values` becomes the slowest rank's; `ok` becomes true only if every rank's is.

    Returns (values, ok); with no process group (one rank) the inputs come back unchanged.
    """
    values = [float(x) for x in values]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return values, bool(ok)
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    f = torch.tensor([1 if ok else 0], dtype=torch.int32, device=device)
    dist.all_reduce(f, op=dist.ReduceOp.MIN)
    return [float(x) for x in t.tolist()], bool(int(f.item()))


def whole_job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Weak scaling: every rank processed `units_per_rank` units in the (max over ranks) time."""
    return world * units_per_rank / seconds
