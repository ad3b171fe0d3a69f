"""Replica bookkeeping of the benchmark: the path does not shard (one GPU per problem), so N GPUs run N
independent replicas.  Each rank times its own steps; the job's time is the slowest rank's and the job's
work is the sum.  The only communication is one all-reduce of two scalars, outside any timed region."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Replicas draw different inputs."""
    return base_seed + rank


def aggregate(local_ms: float, local_work: float, device=None):
    """(max over ranks of local_ms, sum over ranks of local_work); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms), float(local_work)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    w = torch.tensor([local_work], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return float(t.item()), float(w.item())


def throughput(total_work: float, max_ms: float) -> float:
    return total_work / (max_ms * 1e-3)
