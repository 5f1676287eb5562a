"""Host-side helpers for running the step on several GPUs of one node.

The method has no exchange step: every targeted matrix is updated on its own (Algorithm 1's loop over the
targeted matrices), so ranks either run independent replicas or own disjoint sets of whole matrices. The only
quantity that would ever cross ranks is one scalar, the squared global norm used by gradient clipping.
Everything here is plain torch.distributed and runs on any backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def shard_matrices(shapes: Sequence[Tuple[int, int]], world: int) -> List[List[int]]:
    """Partition matrix indices over `world` ranks, whole matrices only, balancing element counts.

    Longest-processing-time greedy: biggest matrix first onto the lightest rank; ties go to the lower rank, so the
    result is deterministic. Every index appears exactly once; lists are returned in ascending index order.
    """
    if world < 1:
        raise ValueError("world must be >= 1")
    order = sorted(range(len(shapes)), key=lambda i: (-shapes[i][0] * shapes[i][1], i))
    load = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        out[r].append(i)
        load[r] += shapes[i][0] * shapes[i][1]
    return [sorted(x) for x in out]


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Largest `value` over all ranks (how a multi-GPU step time is reported). Identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def global_sqnorm(local_sqnorm: float, device=None, group=None) -> float:
    """Sum of per-rank squared gradient norms: the one scalar global-norm clipping needs when matrices are sharded."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(local_sqnorm)
    t = torch.tensor([float(local_sqnorm)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())


def whole_job_throughput(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (units per second)."""
    return world * units_per_rank / (ms_max * 1e-3)
