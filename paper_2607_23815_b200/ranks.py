"""Multi-rank plumbing for replicas-only scaling: the path has no exchange step, so ranks only agree on a
seed per replica and reduce (max time, summed work) for reporting."""
from __future__ import annotations

import torch


def replica_seed(seed: int, rank: int) -> int:
    return seed + 7919 * rank


def aggregate(ms: float, work: float, world: int, device="cuda"):
    """(max over ranks of ms, sum over ranks of work); identity for a single rank."""
    if world == 1:
        return ms, work
    import torch.distributed as dist
    t_max = torch.tensor([ms], dtype=torch.float64, device=device)
    t_sum = torch.tensor([work], dtype=torch.float64, device=device)
    dist.all_reduce(t_max, op=dist.ReduceOp.MAX)
    dist.all_reduce(t_sum, op=dist.ReduceOp.SUM)
    return float(t_max.item()), float(t_sum.item())
