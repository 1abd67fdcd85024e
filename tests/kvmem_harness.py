"""Shared test plumbing: fill a GPU pool and an oracle repository from the same seeded bytes.

The CUDA package and the oracle never meet except here, in test code: both receive the tensors
produced by ``kvmem_workloads``.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from kvmem_workloads import WorkloadSpec, kv_blocks, make_queries, page_table, select_params
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


class Guards:
    """Output buffers with canary bytes in front of and behind them.

    Every buffer a GPU entry point writes (ids, counts, scores, views, outputs) is cut out of a larger allocation
    whose surroundings hold a byte pattern; ``check()`` after the call fails if any entry point wrote outside
    what it was given.  The payload starts 256 bytes into a fresh torch allocation, so it keeps the 256-byte
    alignment the views and workspaces need; the rear canary starts at the payload's last byte + 1."""
    PAD = 256
    BYTE = 0xA5

    def __init__(self, device):
        self.device = device
        self.items = []

    def empty(self, shape, dtype, fill=0) -> torch.Tensor:
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        buf = torch.full((self.PAD + n + self.PAD,), self.BYTE, dtype=torch.uint8, device=self.device)
        t = buf[self.PAD:self.PAD + n].view(dtype).view(*shape)
        if fill is not None:
            t.fill_(fill)
        self.items.append((buf, n))
        return t

    def view(self, pool, n_sessions: int, cap_tokens: int):
        from paper_2609_04852_b200.kvmem import View
        c = pool.cfg
        shape = (n_sessions, c.n_layers, c.n_kv_heads, cap_tokens, c.head_dim)
        return View(self.empty(shape, torch.bfloat16), self.empty(shape, torch.bfloat16), cap_tokens)

    def outputs(self, pool, n_sessions: int, n_q_tokens: int):
        c = pool.cfg
        return (self.empty((n_sessions, n_q_tokens, c.n_layers, c.n_q_heads, c.head_dim), torch.float32),
                self.empty((n_sessions, n_q_tokens, c.n_layers, c.n_q_heads), torch.float32))

    def check(self) -> None:
        for i, (buf, n) in enumerate(self.items):
            front, back = buf[:self.PAD], buf[self.PAD + n:]
            assert bool((front == self.BYTE).all()) and bool((back == self.BYTE).all()), \
                f"guard bytes around output buffer {i} ({n} bytes) were overwritten"


def queries(spec: WorkloadSpec, qset: int = 0):
    q = make_queries(spec, qset)
    return q, bits(q)


# ---- tolerances stated by the benchmark spec -------------------------------------------------------------
SCORE_RTOL = 1e-3          # |R_gpu - R_ref| <= 1e-3 * |R_ref| (+ floor for values that underflow towards 0)
ATTN_ATOL = 2e-3           # max-abs on unit-scale values, outputs and log-sum-exp
GAP_RTOL = 1e-3            # ids must be identical where the relative gap at the k-th boundary exceeds this


# Keys rotated by COMPOSED angles (the raw-key one-pass and copy-free modes): the kernel forms (cos, sin)(p1 + b) from the
# table rows of p1 and of b, four fp32 operations whose result is within 3 units in the last place (3 * 2^-24 relative to
# 1) of the table's own row of p1 + b.  A rotated key a*cos - b*sin therefore moves by at most 3 * 2^-24 * (|a| + |b|)
# < 4e-6 for keys below 10 in magnitude before its rounding to bf16, which shifts the stored code by at most one bf16 step
# (2^-8 relative) unless the rotated value is itself tiny next to its inputs.  An element sits that close to a rounding
# boundary with probability about (4e-6 * 2) / (2^-9 |k|), far below one in a hundred.
ROTATED_KEY_ABS = 4e-6
ROTATED_KEY_MAX_DIFFERING = 1e-2


def check_rotated_keys(view_bits: np.ndarray, ref_bits: np.ndarray) -> None:
    """view_bits, ref_bits: bf16 codes (uint16) of rotated keys; equal up to one bf16 rounding step (plus the absolute
    slack above) on a small fraction of the elements."""
    assert view_bits.shape == ref_bits.shape and view_bits.dtype == np.uint16 and ref_bits.dtype == np.uint16
    differing = view_bits != ref_bits
    if not differing.any():
        return
    frac = differing.mean()
    assert frac <= ROTATED_KEY_MAX_DIFFERING, f"{frac:.2e} of the rotated keys differ from the defined code"
    got = (view_bits[differing].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ref = (ref_bits[differing].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    bound = np.abs(ref) * 2.0 ** -7 + ROTATED_KEY_ABS     # one step of the binade above (a step doubles across a power of two)
    worst = np.abs(got - ref) - bound
    assert worst.max() <= 0, f"a rotated key is off by more than one bf16 step: {got[worst.argmax()]} against {ref[worst.argmax()]}"


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


def full_step(spec: WorkloadSpec, qsets=(0,), gap_forced_budget=None, n_sink=0, n_recent=0):
    """One whole recall step per query set, every stage against the oracle on the same bytes: index bit-exact,
    scores within SCORE_RTOL, ids exact or by the band rule, gathered view bit-exact, attention within ATTN_ATOL.
    The fused pass (what the benchmark times) and the copy-free pass must reproduce the view and the results of
    the separate calls bit for bit.  Every output buffer sits between guard bytes.  Returns the selection modes."""
    from paper_2609_04852_b200 import SelectParams, budget_blocks
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec, gen_device=dev)
    prm_d = select_params(spec)
    prm_d["n_sink_blocks"], prm_d["n_recent_blocks"] = n_sink, n_recent
    if gap_forced_budget is not None:
        prm_d["budget_blocks"] = gap_forced_budget
    prm = SelectParams(**prm_d)
    ns, B, M = spec.n_sessions, spec.block_tokens, spec.n_q_tokens
    k = budget_blocks(prm, B, spec.n_blocks)
    fast = 64 % B == 0 or B % 64 == 0   # the passes that read pages through the block table walk 64-token tiles
    guards = Guards(dev)
    sel = guards.empty((ns, k), torch.int32)
    n_sel = guards.empty((ns,), torch.int32)
    scores = guards.empty((ns, spec.n_blocks), torch.float32)
    view = guards.view(pool, ns, k * B)
    out, lse = guards.outputs(pool, ns, M)
    view2 = guards.view(pool, ns, k * B) if fast else None
    out2, lse2 = guards.outputs(pool, ns, M)
    out3, lse3 = guards.outputs(pool, ns, M)
    for s in range(ns):
        assert np.array_equal(bits(pool.index(s)), osess[s].idx), "Mean-K index differs"
    modes = []
    for qset in qsets:
        q, qb = queries(spec, qset)
        qd = q.to(dev)
        pool.select(qd, prm, sel, n_sel, scores)
        pool.materialize(sel, n_sel, view)
        if spec.attend:
            pool.view_attend(qd, view, n_sel, out, lse)
            if fast:
                view2.k.zero_(), view2.v.zero_()
                pool.materialize_attend(qd, sel, n_sel, view2, out2, lse2)
                pool.paged_attend(qd, sel, n_sel, out3, lse3)
        torch.cuda.synchronize()
        assert pool.device_status() == 0
        guards.check()
        if spec.attend and fast:
            assert torch.equal(view.k, view2.k) and torch.equal(view.v, view2.v), "fused pass left a different view"
            assert torch.equal(out, out2) and torch.equal(lse, lse2), "fused pass: different results"
            assert torch.equal(out, out3) and torch.equal(lse, lse3), "copy-free pass: different results"
        sel_h, n_h, sc_h = sel.cpu().numpy(), n_sel.cpu().numpy(), scores.cpu().numpy()
        out_h, lse_h = out.cpu().numpy(), lse.cpu().numpy()
        for s in range(ns):
            R, _ = orc.block_scores(qb[s], osess[s].idx, spec.n_blocks)
            ref_sel = orc.select(R, B, prm_d["budget_blocks"], prm_d["max_view_tokens"], 0, n_sink, n_recent)
            check_scores(sc_h[s], R, M)
            sel_gpu = sel_h[s, : n_h[s]]
            assert n_h[s] == k == len(ref_sel) and k * B <= spec.max_view_tokens
            modes.append(check_selection(sel_gpu, R, ref_sel, n_sink, n_recent))
            vK, vV = orc.gather(osess[s].repo, osess[s].table, np.ascontiguousarray(sel_gpu), k * B)
            assert np.array_equal(bits(view.k[s]), vK) and np.array_equal(bits(view.v[s]), vV), "gathered view differs"
            if not spec.attend:
                continue
            ref_out, ref_lse = orc.attend(qb[s], vK, vV, k * B)
            err_o, err_l = np.abs(out_h[s] - ref_out).max(), np.abs(lse_h[s] - ref_lse).max()
            assert err_o <= ATTN_ATOL and err_l <= ATTN_ATOL, f"attention error {err_o:.2e}, lse {err_l:.2e}"
            assert err_o <= 5e-2 * np.abs(ref_out).max(), "attention error is large relative to the output scale"
    return modes
