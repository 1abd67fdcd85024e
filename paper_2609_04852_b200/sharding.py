"""Multi-GPU plumbing.  The recall path shards two ways.

By session (weak scaling): sessions are independent problems (each softmax runs over its own blocks, a
physical page belongs to one session), so N GPUs own disjoint sets of sessions and the data path has no
collective; the only communication is the benchmark's bookkeeping (a barrier around the timed region and
the maximum of the per-rank times).

By KV head inside one session (strong scaling): the softmax of the block score (Eq. "kvmem-block-score",
Sec. 4.3) is taken per (layer, query token, query head), so a GPU that holds the pages and index rows of
KV heads [g0, g1) and the query heads that map to them computes its heads' share of R_b without seeing
the others.  R_b is a mean over heads: one all-reduce (sum) of the NB fp32 partial scores, each scaled by
its share of the heads inside the scoring kernel (kvmem_score's score_scale), gives every rank the same R bit for bit; every rank then runs the same
deterministic top-k and gathers and attends over its own heads.  Outputs are head-disjoint: no second
exchange.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

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


# ---- sharding by KV head inside a session ---------------------------------------------------------

def kv_heads_for_rank(n_kv_heads: int, rank: int, world: int) -> Tuple[int, int]:
    """[g0, g1): equal contiguous slices, so that every rank's share of the head mean is 1/world."""
    if not (0 <= rank < world):
        raise ValueError("rank must be in [0, world)")
    if n_kv_heads % world != 0:
        raise ValueError(f"{n_kv_heads} KV heads do not split evenly over {world} ranks")
    per = n_kv_heads // world
    return rank * per, (rank + 1) * per


def query_heads_of(kv_range: Tuple[int, int], q_per_kv: int) -> Tuple[int, int]:
    """[h0, h1): the query heads whose KV head g(h) = h // q_per_kv lies in kv_range."""
    return kv_range[0] * q_per_kv, kv_range[1] * q_per_kv


def combine_head_shard_scores(r_share: torch.Tensor, world: int, group=None,
                              all_reduce: Optional[Callable[[torch.Tensor], None]] = None) -> torch.Tensor:
    """In place: r_share (this rank's mean over ITS heads times 1/world, as kvmem_score writes it when given
    score_scale = 1/world) -> R (mean over all heads), identical on every rank.

    R = sum over ranks of r_share: one all-reduce and nothing else; the 1/world factor is applied by the scoring
    kernel (exact for a power-of-two world).  all_reduce overrides the collective (tests without a process group)."""
    if world < 1:
        raise ValueError("world must be positive")
    if world == 1:
        return r_share
    r_local = r_share
    if all_reduce is not None:
        all_reduce(r_local)
    else:
        dist.all_reduce(r_local, op=dist.ReduceOp.SUM, group=group)
    return r_local


def head_sharded_step(pool, q_local: torch.Tensor, params, scores: torch.Tensor, sel_ids: torch.Tensor,
                      n_sel: torch.Tensor, view, out: torch.Tensor, lse: torch.Tensor, world: int, group=None,
                      all_reduce: Optional[Callable[[torch.Tensor], None]] = None) -> None:
    """One recall step of a rank that owns a slice of the KV heads of every session in `pool`.

    pool holds only this rank's heads (created with n_kv_heads / world and n_q_heads / world); q_local is the
    matching slice of the query heads.  score (own heads) -> all-reduce of R -> top-k (same ids on every rank)
    -> view assembly and attention over the own heads.  Every step runs in the library's kernels; the only
    exchange is the all-reduce of scores ([n_sessions][max_blocks_per_session] fp32)."""
    pool.score(q_local, scores, score_scale=1.0 / world)
    combine_head_shard_scores(scores, world, group, all_reduce)
    pool.topk(scores, params, sel_ids, n_sel)
    pool.materialize_attend(q_local, sel_ids, n_sel, view, out, lse)
