"""Shared test plumbing: fill a GPU pool and an oracle repository from the same seeded bytes.

The CUDA package and the oracle never meet except here, in test code: both receive the tensors
produced by ``kvmem_workloads``.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from kvmem_workloads import WorkloadSpec, kv_blocks, make_queries, page_table
from oracle import kvmem_oracle as orc


def bits(t: torch.Tensor) -> np.ndarray:
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


@dataclass
class OracleSession:
    repo: orc.Repository
    table: np.ndarray
    idx: np.ndarray
    n_blocks: int


def fill_oracle(spec: WorkloadSpec, n_blocks: Optional[List[int]] = None, gen_device="cpu") -> List[OracleSession]:
    """Oracle-side state: one repository of physical pages shared by the sessions, one index each."""
    tables = page_table(spec).numpy()
    lens = [spec.n_blocks if n_blocks is None else n_blocks[s] for s in range(spec.n_sessions)]
    n_pages = max(int(tables[s, :lens[s]].max(initial=0)) + 1 for s in range(spec.n_sessions))
    repo = orc.Repository.empty(n_pages, spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim)
    out = []
    for s in range(spec.n_sessions):
        nb = lens[s]
        idx = np.zeros((spec.n_layers, spec.n_kv_heads, max(nb, 1), spec.head_dim), np.uint16)
        step = 512
        for b0 in range(0, nb, step):
            b1 = min(nb, b0 + step)
            K, V = kv_blocks(spec, s, b0, b1, gen_device)
            Kb, Vb = bits(K), bits(V)
            repo.place(Kb, Vb, np.ascontiguousarray(tables[s, b0:b1]))
            orc.mean_k_index(Kb, spec.block_tokens, idx, b0)
        out.append(OracleSession(repo, np.ascontiguousarray(tables[s]), idx, nb))
    return out


def fill_pool(spec: WorkloadSpec, n_blocks: Optional[List[int]] = None, extra_pages: int = 0):
    """GPU pool holding the same workspaces; keys/values are generated on the device."""
    from paper_2609_04852_b200 import Pool
    dev = torch.device("cuda", 0)
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens,
                spec.n_sessions, spec.n_sessions * spec.n_blocks + extra_pages, spec.n_blocks, 0)
    tables = page_table(spec)
    for s in range(spec.n_sessions):
        nb = spec.n_blocks if n_blocks is None else n_blocks[s]
        step = 1024
        for b0 in range(0, nb, step):
            b1 = min(nb, b0 + step)
            K, V = kv_blocks(spec, s, b0, b1, dev)
            pool.append_blocks(s, K, V, tables[s, b0:b1].tolist())
    torch.cuda.synchronize()
    return pool


def queries(spec: WorkloadSpec, qset: int = 0):
    q = make_queries(spec, qset)
    return q, bits(q)


# ---- tolerances stated by the benchmark spec -------------------------------------------------------------
SCORE_RTOL = 1e-3          # |R_gpu - R_ref| <= 1e-3 * |R_ref| (+ floor for values that underflow towards 0)
ATTN_ATOL = 2e-3           # max-abs on unit-scale values, outputs and log-sum-exp
GAP_RTOL = 1e-3            # ids must be identical where the relative gap at the k-th boundary exceeds this


def check_scores(R_gpu: np.ndarray, R_ref: np.ndarray, M: int) -> None:
    floor = 1e-6 * M / max(len(R_ref), 1)      # a millionth of the mean score: only matters near underflow
    err = np.abs(R_gpu - R_ref)
    assert np.all(err <= SCORE_RTOL * np.abs(R_ref) + floor), \
        f"score mismatch: max rel err {np.max(err / np.maximum(np.abs(R_ref), 1e-30)):.3e}"


def check_selection(sel_gpu: np.ndarray, R_ref: np.ndarray, sel_ref: np.ndarray, n_sink=0, n_recent=0) -> str:
    """Exact equality where the boundary gap is resolvable, otherwise the band rule.  Returns which applied."""
    assert len(sel_gpu) == len(sel_ref), f"selected {len(sel_gpu)} blocks, oracle {len(sel_ref)}"
    assert np.all(np.diff(sel_gpu) > 0), "ids must be strictly ascending"
    NB = len(R_ref)
    if len(sel_ref) in (0, NB):
        assert np.array_equal(sel_gpu, sel_ref)
        return "exact"
    reserved = np.zeros(NB, bool)
    reserved[:n_sink] = True
    if n_recent:
        reserved[NB - n_recent:] = True
    in_ref = np.zeros(NB, bool)
    in_ref[sel_ref] = True
    cand_in = R_ref[in_ref & ~reserved]
    cand_out = R_ref[~in_ref & ~reserved]
    if len(cand_in) == 0 or len(cand_out) == 0:
        assert np.array_equal(sel_gpu, sel_ref)
        return "exact"
    r_k, r_next = cand_in.min(), cand_out.max()
    if (r_k - r_next) > GAP_RTOL * r_k:
        assert np.array_equal(sel_gpu, sel_ref), "ids differ although the k-th boundary gap exceeds 1e-3"
        return "exact"
    in_gpu = np.zeros(NB, bool)
    in_gpu[sel_gpu] = True
    must = (~reserved & (R_ref > r_k * (1 + GAP_RTOL))) | (reserved & in_ref)
    must_not = ~reserved & (R_ref < r_k * (1 - GAP_RTOL))
    assert np.all(in_gpu[must]), "a block clearly above the boundary was not selected"
    assert not np.any(in_gpu[must_not]), "a block clearly below the boundary was selected"
    return "band"
