"""Multi-GPU plumbing: the recall path shards by session, with no collective on the data path.

Sessions are independent problems (each softmax runs over its own blocks, a physical page belongs
to one session), so N GPUs simply own disjoint sets of sessions.  The only communication is the
benchmark's bookkeeping: a barrier around the timed region and the maximum of the per-rank times.
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def sessions_for_rank(n_sessions: int, rank: int, world: int) -> List[int]:
    """Contiguous, balanced partition of session ids; every session has exactly one owner."""
    if not (0 <= rank < world) or n_sessions < 0:
        raise ValueError("rank must be in [0, world) and n_sessions non-negative")
    lo = n_sessions * rank // world
    hi = n_sessions * (rank + 1) // world
    return list(range(lo, hi))


def owner_of(session: int, n_sessions: int, world: int) -> int:
    """Rank that owns `session` under sessions_for_rank."""
    if not (0 <= session < n_sessions):
        raise ValueError("session out of range")
    for r in range(world):
        if session < n_sessions * (r + 1) // world:
            return r
    raise AssertionError("unreachable")


def max_over_ranks(values: Sequence[float], device="cpu") -> List[float]:
    """Element-wise maximum of per-rank timings (identity when no process group is up)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank: int, world: int, max_ms: float) -> float:
    """Units per second over all ranks, given the slowest rank's time for `units_per_rank` units."""
    return world * units_per_rank / (max_ms * 1e-3)
