"""Multi-GPU plumbing: the pass has no exchange step (units are independent), so ranks only need
a partition of the work and a max-reduction of their timings."""
from __future__ import annotations

import copy
from typing import List, Tuple


def shard_range(count: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [begin, end) share of `count` items for `rank`; shares differ by at most one."""
    base, extra = divmod(count, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_layers(layers: int, rank: int, world: int) -> List[int]:
    """The layers of one model that `rank` compresses when a single job is split (strong scaling)."""
    begin, end = shard_range(layers, rank, world)
    return list(range(begin, end))


def rank_workload(w, rank: int):
    """Weak scaling: every rank compresses its own copy of the workload, drawn with its own seed."""
    w = copy.deepcopy(w)
    w.seed = w.seed + 1000 * rank
    return w


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_second(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    return tokens_per_rank * world / (ms_per_step * 1e-3)
