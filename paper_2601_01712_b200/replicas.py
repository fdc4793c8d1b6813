"""Scale-out as the paper does it: independent replicas, users placed by a hash of their id.

The path shards by user - a pre-infer / rank pair touches one user's cached prefix and nothing else - and the
paper routes every request of a user to the instance that holds the cache by consistent hashing of the user id
(Section 3.3, "Affinity routing").  There is no data-path collective: each GPU runs the whole library on its own
users.  ``torch.distributed`` is used only to agree on a timing (max over ranks) and to barrier.
"""
from __future__ import annotations

from typing import Iterable, List

_MIX = 0x9E3779B97F4A7C15


def owner_rank(user_id: int, world_size: int) -> int:
    """The replica that holds (or will hold) this user's prefix cache."""
    h = ((int(user_id) * _MIX) & 0xFFFFFFFFFFFFFFFF) >> 33      # multiplicative hash modulo 2^64
    return h % int(world_size)


def users_of_rank(user_ids: Iterable[int], rank: int, world_size: int) -> List[int]:
    return [int(u) for u in user_ids if owner_rank(int(u), world_size) == rank]


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Max of a per-rank scalar over all ranks (the job's time is its slowest replica's)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, seconds_per_rank: float, dist=None, device=None) -> float:
    """Whole-job units per second: every rank's units over the slowest rank's time."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return units_per_rank / seconds_per_rank
    import torch
    u = torch.tensor([float(units_per_rank)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / max_over_ranks(seconds_per_rank, dist, device)
