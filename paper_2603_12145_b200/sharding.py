"""Host-side logic of the multi-GPU run: how envs are split over ranks and how
per-rank results are combined.  Envs are independent, so each rank owns a
contiguous range of global env ids and there is no data-path collective; only
the timing (max over ranks) and the three int64 episode counters (sum) cross
ranks.  Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

from typing import Sequence, Tuple


def shard(rank: int, world: int, n_per_rank: int) -> Tuple[int, int]:
    """(env_id_base, n_envs) of a rank under weak scaling: every rank simulates
    n_per_rank envs with global ids rank*n_per_rank ..."""
    if not (0 <= rank < world) or n_per_rank < 1:
        raise ValueError("bad rank / world / n_per_rank")
    if world * n_per_rank > 0x7FFFFFFF:
        raise ValueError("global env ids must fit in 31 bits")
    return rank * n_per_rank, n_per_rank


def split(n_total: int, world: int) -> Sequence[Tuple[int, int]]:
    """Strong-scaling split of n_total envs into `world` contiguous ranges whose
    sizes differ by at most one: [(env_id_base, n_envs), ...]."""
    if world < 1 or n_total < world:
        raise ValueError("need at least one env per rank")
    q, r = divmod(n_total, world)
    out, base = [], 0
    for k in range(world):
        n = q + (1 if k < r else 0)
        out.append((base, n))
        base += n
    return out


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar (the timed interval) over all ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_stats(stats: Tuple[int, int, int], device=None) -> Tuple[int, int, int]:
    """Sum of the (episodes, sum_return, sum_length) counters over all ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return tuple(int(x) for x in stats)
    t = torch.tensor(list(stats), dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return tuple(int(x) for x in t.tolist())
