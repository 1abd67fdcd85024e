"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element, on
the same seeded inputs.  Index, selected ids and gathered views: bit-exact.  Scores: 1e-3
relative.  Attention outputs and log-sum-exp: 2e-3 max-abs on unit-scale values.
"""
import numpy as np
import pytest
import torch

from kvmem_harness import (ATTN_ATOL, bits, check_scores, check_selection, fill_oracle, fill_pool, queries)
from kvmem_workloads import CONFIGS, planted_blocks
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu

SMALL = CONFIGS["tiny"].with_(name="small", n_blocks=200, n_planted=6, budget_blocks=24)   # ragged: 200 = 128 + 72


def _params(**kw):
    from paper_2609_04852_b200 import SelectParams
    base = dict(budget_blocks=0, max_view_tokens=1 << 30, mandatory_tokens=0, n_sink_blocks=0, n_recent_blocks=0)
    base.update(kw)
    return SelectParams(**base)


def _run_step(pool, spec, q_dev, params, cap_blocks, n_sessions=None, attend=True):
    """select -> materialize -> attend through the C ABI; returns host copies."""
    ns = spec.n_sessions if n_sessions is None else n_sessions
    dev = q_dev.device
    sel = torch.full((ns, max(cap_blocks, 1)), -1, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(ns, dtype=torch.int32, device=dev)
    scores = torch.zeros(ns, spec.n_blocks, dtype=torch.float32, device=dev)
    view = pool.new_view(ns, max(cap_blocks, 1) * spec.block_tokens)
    pool.select(q_dev, params, sel, n_sel, scores)
    pool.materialize(sel, n_sel, view)
    out = lse = None
    if attend:
        out, lse = pool.new_outputs(ns, spec.n_q_tokens)
        pool.view_attend(q_dev, view, n_sel, out, lse)
    assert pool.device_status() == 0
    return dict(sel=sel.cpu().numpy(), n_sel=n_sel.cpu().numpy(), scores=scores.cpu().numpy(), view=view,
                out=None if out is None else out.cpu().numpy(), lse=None if lse is None else lse.cpu().numpy())


def _oracle_step(spec, osess, qb, s, budget, max_view=1 << 30, mandatory=0, sink=0, recent=0, sel_override=None):
    R, _ = orc.block_scores(qb[s], osess.idx, osess.n_blocks)
    sel = orc.select(R, spec.block_tokens, budget, max_view, mandatory, sink, recent)
    use = sel if sel_override is None else sel_override
    cap = max(len(use), 1) * spec.block_tokens
    vK, vV = orc.gather(osess.repo, osess.table, use, cap)
    out, lse = orc.attend(qb[s], vK, vV, len(use) * spec.block_tokens)
    return dict(R=R, sel=sel, vK=vK, vV=vV, out=out, lse=lse)


def _compare_step(spec, got, s, ref, sink=0, recent=0):
    n = int(got["n_sel"][s])
    sel_gpu = got["sel"][s, :n]
    check_scores(got["scores"][s, :len(ref["R"])], ref["R"], spec.n_q_tokens)
    how = check_selection(sel_gpu, ref["R"], ref["sel"], sink, recent)
    return sel_gpu, how


def _compare_view_and_attention(spec, got, s, ref_same_ids):
    n = int(got["n_sel"][s])
    T = n * spec.block_tokens
    gk, gv = bits(got["view"].k[s]), bits(got["view"].v[s])
    assert np.array_equal(gk[:, :, :T], ref_same_ids["vK"][:, :, :T]), "gathered K differs"
    assert np.array_equal(gv[:, :, :T], ref_same_ids["vV"][:, :, :T]), "gathered V differs"
    if got["out"] is not None:
        err_o = np.abs(got["out"][s] - ref_same_ids["out"]).max()
        if T == 0:                                                   # empty view: lse is -inf on both sides
            assert np.all(np.isneginf(got["lse"][s])) and np.all(np.isneginf(ref_same_ids["lse"]))
            assert err_o == 0
            return
        err_l = np.abs(got["lse"][s] - ref_same_ids["lse"]).max()
        assert err_o <= ATTN_ATOL and err_l <= ATTN_ATOL, f"attention error {err_o:.2e} / lse {err_l:.2e}"
        rel = err_o / max(np.abs(ref_same_ids["out"]).max(), 1e-30)
        assert rel < 5e-2, f"relative attention error {rel:.2e}"          # the absolute bound must not be vacuous


# ------------------------------------------------------------------ index

@pytest.mark.parametrize("spec", [SMALL, SMALL.with_(n_layers=2, n_kv_heads=4, n_q_heads=8, block_tokens=32, n_blocks=37)],
                         ids=["L1G8B64", "L2G4B32"])
def test_index_and_block_table_bit_exact(spec):
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    assert np.array_equal(bits(pool.index(0)), osess.idx)
    assert np.array_equal(pool.block_table(0).cpu().numpy(), osess.table[:spec.n_blocks])
    assert pool.device_status() == 0


# ------------------------------------------------------------------ whole step on small workspaces

@pytest.mark.parametrize("M", [1, 2, 4])
@pytest.mark.parametrize("gather_mode,score_mode", [(1, 1), (0, 0)])
def test_step_matches_oracle_small(M, gather_mode, score_mode):
    from paper_2609_04852_b200 import set_option
    spec = SMALL.with_(n_q_tokens=M)
    set_option("gather_mode", gather_mode)
    set_option("score_mode", score_mode)
    try:
        pool = fill_pool(spec)
        osess = fill_oracle(spec)[0]
        for qset in range(2):
            q, qb = queries(spec, qset)
            got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.budget_blocks), spec.budget_blocks)
            ref = _oracle_step(spec, osess, qb, 0, spec.budget_blocks)
            sel_gpu, _ = _compare_step(spec, got, 0, ref)
            same = _oracle_step(spec, osess, qb, 0, spec.budget_blocks, sel_override=sel_gpu)
            _compare_view_and_attention(spec, got, 0, same)
    finally:
        set_option("gather_mode", 1)
        set_option("score_mode", 1)


@pytest.mark.parametrize("block_tokens,budget", [(32, 21), (32, 24), (16, 37), (128, 5)])
def test_step_with_other_block_sizes(block_tokens, budget):
    # the paper's default block is 32 tokens; the view is walked in 64-token tiles, so an odd number of 32-token
    # blocks (or any count of 16-token blocks not divisible by 4) ends in a partly filled tile
    spec = SMALL.with_(block_tokens=block_tokens, budget_blocks=budget, n_q_tokens=2)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=budget), budget)
    ref = _oracle_step(spec, osess, qb, 0, budget)
    sel_gpu, _ = _compare_step(spec, got, 0, ref)
    assert len(sel_gpu) == budget
    same = _oracle_step(spec, osess, qb, 0, budget, sel_override=sel_gpu)
    _compare_view_and_attention(spec, got, 0, same)


@pytest.mark.parametrize("M,score_mode", [(8, 1), (8, 0), (16, 1), (5, 0)])
def test_scoring_with_more_than_sixteen_rows_per_kv_head(M, score_mode):
    # M * 4 rows per KV head > 16: the decode scorer walks the rows in passes of 16
    from paper_2609_04852_b200 import set_option
    spec = SMALL.with_(n_q_tokens=M, n_blocks=333)
    set_option("score_mode", score_mode)
    try:
        pool = fill_pool(spec)
        osess = fill_oracle(spec)[0]
        q, qb = queries(spec)
        got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.budget_blocks), spec.budget_blocks, attend=False)
        R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
        check_scores(got["scores"][0], R, M)
        check_selection(got["sel"][0, : int(got["n_sel"][0])], R, orc.select(R, 64, spec.budget_blocks, 1 << 30))
    finally:
        set_option("score_mode", 1)


def test_gap_forced_selection_is_identical_and_recovers_planted_blocks():
    spec = SMALL
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.n_planted), spec.n_planted)
    ref = _oracle_step(spec, osess, qb, 0, spec.n_planted)
    sel_gpu, how = _compare_step(spec, got, 0, ref)
    assert how == "exact" and np.array_equal(sel_gpu, ref["sel"])
    assert set(sel_gpu.tolist()) == set(planted_blocks(spec, 0)[0].tolist())
    _compare_view_and_attention(spec, got, 0, ref)


@pytest.mark.parametrize("budget,max_view,mandatory,sink,recent", [
    (10 ** 6, 1 << 30, 0, 0, 0),        # k >= NB: the view is the whole history
    (24, 64 * 10, 1, 0, 0),             # capacity clamp: floor((640 - 1) / 64) = 9 blocks
    (24, 1 << 30, 0, 3, 5),             # sink + recent reservation
    (6, 1 << 30, 0, 4, 4),              # reservation larger than the budget
    (0, 1 << 30, 0, 0, 0),              # empty selection
    (1, 1 << 30, 0, 0, 0),
])
def test_budget_and_reservation_edge_cases(budget, max_view, mandatory, sink, recent):
    spec = SMALL
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, qb = queries(spec, 1)
    k = orc.budget_blocks(spec.n_blocks, spec.block_tokens, budget, max_view, mandatory)
    prm = _params(budget_blocks=min(budget, 2 ** 31 - 1), max_view_tokens=max_view, mandatory_tokens=mandatory,
                  n_sink_blocks=sink, n_recent_blocks=recent)
    from paper_2609_04852_b200 import budget_blocks
    assert budget_blocks(prm, spec.block_tokens, spec.n_blocks) == k
    got = _run_step(pool, spec, q.cuda(), prm, k)
    ref = _oracle_step(spec, osess, qb, 0, budget, max_view, mandatory, sink, recent)
    assert int(got["n_sel"][0]) == k == len(ref["sel"])
    sel_gpu, _ = _compare_step(spec, got, 0, ref, sink, recent)
    same = _oracle_step(spec, osess, qb, 0, budget, max_view, mandatory, sink, recent, sel_override=sel_gpu)
    _compare_view_and_attention(spec, got, 0, same)
    if k == 0:
        assert not got["out"].any() and np.all(np.isneginf(got["lse"]))


def test_selecting_everything_equals_full_attention_over_raw_history():
    spec = SMALL.with_(n_blocks=70, n_q_tokens=4)
    pool = fill_pool(spec)
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=10 ** 6), spec.n_blocks)
    assert got["sel"][0].tolist() == list(range(spec.n_blocks))
    from kvmem_workloads import kv_blocks
    K, V = kv_blocks(spec, 0, 0, spec.n_blocks)
    vK = np.ascontiguousarray(np.transpose(bits(K), (1, 2, 0, 3)))
    vV = np.ascontiguousarray(np.transpose(bits(V), (1, 2, 0, 3)))
    out, lse = orc.attend(qb[0], vK, vV, spec.tokens)
    assert np.abs(got["out"][0] - out).max() <= ATTN_ATOL and np.abs(got["lse"][0] - lse).max() <= ATTN_ATOL


def test_duplicate_blocks_tie_break_by_lower_id():
    # identical keys in every block => identical scores: the selection must be the k lowest ids
    from paper_2609_04852_b200 import Pool
    spec = SMALL.with_(n_blocks=40)
    dev = torch.device("cuda", 0)
    pool = Pool(1, 32, 8, 128, 64, 1, 40, 40, 0)
    from kvmem_workloads import kv_blocks
    K, V = kv_blocks(spec, 0, 0, 1, dev)
    pool.append_blocks(0, K.repeat(40, 1, 1, 1).contiguous(), V.repeat(40, 1, 1, 1).contiguous())
    q, _ = queries(spec)
    got = _run_step(pool, spec.with_(n_blocks=40), q.cuda(), _params(budget_blocks=7), 7)
    assert got["sel"][0, :7].tolist() == list(range(7))
    assert np.all(got["scores"][0, :40] == got["scores"][0, 0])


def test_long_session_takes_the_general_top_k_path():
    # more than 16,384 blocks: the selector re-reads the scores from global memory in every pass
    spec = CONFIGS["tiny"].with_(name="long", n_blocks=16384 + 517, block_tokens=16, n_planted=40, budget_blocks=300)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, qb = queries(spec)
    for budget in (300, 40):
        got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=budget), budget, attend=False)
        R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
        check_scores(got["scores"][0], R, spec.n_q_tokens)
        sel_gpu = got["sel"][0, : int(got["n_sel"][0])]
        check_selection(sel_gpu, R, orc.select(R, spec.block_tokens, budget, 1 << 30))
        vK, vV = orc.gather(osess.repo, osess.table, np.ascontiguousarray(sel_gpu), budget * spec.block_tokens)
        T = len(sel_gpu) * spec.block_tokens
        assert np.array_equal(bits(got["view"].k[0])[:, :, :T], vK[:, :, :T])


@pytest.mark.parametrize("n_scores,budget,sink,recent,kind", [
    (16385, 300, 0, 0, "normal"), (50000, 4096, 3, 5, "normal"), (140000, 2048, 0, 0, "normal"),   # 2, 4 and 9 tiles
    (40000, 1000, 2, 2, "ties"), (33000, 500, 0, 0, "constant"), (20000, 19990, 4, 4, "normal"), (70000, 70000, 0, 0, "normal")])
def test_selection_from_given_scores_in_long_sessions(n_scores, budget, sink, recent, kind):
    """kvmem_topk on sessions above 16,384 blocks: the cluster kernel and the single-CTA kernel against the oracle's
    selector, bit for bit (scores are given, so there is nothing to tolerate), with heavy ties and reservations."""
    from paper_2609_04852_b200 import Pool, set_option
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(n_scores)
    if kind == "normal":
        R = rng.random(n_scores).astype(np.float32) ** 8                    # skewed, like softmax mass
    elif kind == "ties":
        R = rng.integers(0, 6, n_scores).astype(np.float32) / 8.0           # six distinct values: thousands of ties
    else:
        R = np.full(n_scores, 0.25, np.float32)
    # a pool that only carries the session length (tiny head geometry, no data needed for selection)
    pool = Pool(1, 1, 1, 128, 16, 1, n_scores, n_scores, 0)
    K = torch.zeros(n_scores * 16, 1, 1, 128, dtype=torch.bfloat16, device=dev)
    pool.append_blocks(0, K, K)
    scores = torch.from_numpy(R).view(1, -1).to(dev)
    ref = orc.select(R, 16, budget, 1 << 30, 0, sink, recent)
    for mode in (1, 0):
        set_option("topk_cluster", mode)
        try:
            sel = torch.full((1, budget), -1, dtype=torch.int32, device=dev)
            n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
            pool.topk(scores, _params(budget_blocks=budget, n_sink_blocks=sink, n_recent_blocks=recent), sel, n_sel)
            torch.cuda.synchronize()
            assert pool.device_status() == 0
            got = sel.cpu().numpy()[0, : int(n_sel[0])]
            assert np.array_equal(got, ref), f"mode {mode}: {len(got)} ids, oracle {len(ref)}"
        finally:
            set_option("topk_cluster", 1)


@pytest.mark.parametrize("n_scores,budget,sink,recent,kind", [
    (1, 1, 0, 0, "normal"), (257, 32, 0, 0, "normal"), (1024, 100, 1, 2, "ties"), (1025, 1000, 0, 0, "normal"),
    (2048, 512, 0, 0, "normal"), (2049, 7, 3, 0, "ties"), (4096, 4095, 0, 0, "normal"), (5000, 1234, 2, 9, "ties"),
    (8192, 800, 0, 0, "constant"), (8193, 4096, 0, 0, "normal"), (16384, 4096, 0, 0, "normal"), (16384, 5000, 5, 5, "ties")])
def test_selection_from_given_scores_in_short_sessions(n_scores, budget, sink, recent, kind):
    """kvmem_topk up to 16,384 blocks: the register kernel's instantiations (1, 2, 4, 8 and 16 scores per thread;
    the session picks the smallest that covers it, the switch forces larger ones) against the oracle's selector,
    bit for bit, at the sizes where the instantiation changes."""
    from paper_2609_04852_b200 import Pool, set_option
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(n_scores + budget)
    if kind == "normal":
        R = rng.random(n_scores).astype(np.float32) ** 8
    elif kind == "ties":
        R = rng.integers(0, 6, n_scores).astype(np.float32) / 8.0
    else:
        R = np.full(n_scores, 0.25, np.float32)
    pool = Pool(1, 1, 1, 128, 16, 1, n_scores, n_scores, 0)
    K = torch.zeros(n_scores * 16, 1, 1, 128, dtype=torch.bfloat16, device=dev)
    pool.append_blocks(0, K, K)
    ref = orc.select(R, 16, budget, 1 << 30, 0, sink, recent)
    # an unaligned score pointer takes the scalar loads
    for items, offset in ((0, 0), (16, 0), (4, 0), (0, 1), (8, 3)):
        buf = torch.zeros(n_scores + 8, dtype=torch.float32, device=dev)
        scores = buf[offset: offset + n_scores].view(1, -1)
        scores.copy_(torch.from_numpy(R).view(1, -1))
        set_option("topk_items", items)
        try:
            sel = torch.full((1, budget), -1, dtype=torch.int32, device=dev)
            n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
            pool.topk(scores, _params(budget_blocks=budget, n_sink_blocks=sink, n_recent_blocks=recent), sel, n_sel)
            torch.cuda.synchronize()
            assert pool.device_status() == 0
            got = sel.cpu().numpy()[0, : int(n_sel[0])]
            assert np.array_equal(got, ref), f"items {items}, offset {offset}: {len(got)} ids, oracle {len(ref)}"
        finally:
            set_option("topk_items", 0)


# ------------------------------------------------------------------ working-set delta

def test_working_set_delta_between_two_steps():
    spec = CONFIGS["batch8"].with_(name="delta", n_sessions=2, n_blocks=3000, n_planted=40, budget_blocks=1500,
                                   block_tokens=16, n_q_tokens=1, permute_pages=False)
    pool = fill_pool(spec)
    dev = torch.device("cuda", 0)
    k = spec.budget_blocks
    sels, counts = [], []
    for qset, budget in ((0, 1500), (5, 1100)):                 # two consecutive steps with different queries and budgets
        q = queries(spec, qset)[0].to(dev)
        sel = torch.full((2, k), -1, dtype=torch.int32, device=dev)
        n_sel = torch.zeros(2, dtype=torch.int32, device=dev)
        pool.select(q, _params(budget_blocks=budget), sel, n_sel)
        sels.append(sel); counts.append(n_sel)
    ret, inc, out, cnt = pool.working_set_delta(sels[0], counts[0], sels[1], counts[1])
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    for s in range(2):
        prev = sels[0][s, : int(counts[0][s])].cpu().numpy()
        nxt = sels[1][s, : int(counts[1][s])].cpu().numpy()
        r_ref, i_ref, o_ref = orc.working_set_delta(prev, nxt)
        nR, nL, nE = (int(x) for x in cnt[s].cpu())
        assert (nR, nL, nE) == (len(r_ref), len(i_ref), len(o_ref)) and nR > 0 and nL > 0 and nE > 0
        assert np.array_equal(ret[s, :nR].cpu().numpy(), r_ref)
        assert np.array_equal(inc[s, :nL].cpu().numpy(), i_ref)
        assert np.array_equal(out[s, :nE].cpu().numpy(), o_ref)


# ------------------------------------------------------------------ fused view assembly + attention

@pytest.mark.parametrize("n_sessions,M,budget", [(1, 4, 150), (3, 1, 20), (1, 2, 1)])
def test_fused_materialize_attend_equals_separate_calls_and_oracle(n_sessions, M, budget):
    spec = CONFIGS["batch8"].with_(name="fused", n_sessions=n_sessions, n_blocks=300, n_planted=6, budget_blocks=budget,
                                   n_q_tokens=M)
    lens = [300 - 41 * s for s in range(n_sessions)]
    pool = fill_pool(spec, lens)
    osess = fill_oracle(spec, lens)
    dev = torch.device("cuda", 0)
    q, qb = queries(spec)
    qd = q.to(dev)
    sel = torch.full((n_sessions, budget), -1, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(n_sessions, dtype=torch.int32, device=dev)
    pool.select(qd, _params(budget_blocks=budget), sel, n_sel)
    view_a, view_b = pool.new_view(n_sessions, budget * 64), pool.new_view(n_sessions, budget * 64)
    out_a, lse_a = pool.new_outputs(n_sessions, M)
    out_b, lse_b = pool.new_outputs(n_sessions, M)
    pool.materialize(sel, n_sel, view_a)
    pool.view_attend(qd, view_a, n_sel, out_a, lse_a)
    pool.materialize_attend(qd, sel, n_sel, view_b, out_b, lse_b)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert torch.equal(view_a.k, view_b.k) and torch.equal(view_a.v, view_b.v), "fused view differs from the gathered view"
    assert torch.equal(out_a, out_b) and torch.equal(lse_a, lse_b), "same tiles, same order: results must be identical"
    out_c, lse_c = pool.new_outputs(n_sessions, M)            # copy-free view: attention straight over the pages
    pool.paged_attend(qd, sel, n_sel, out_c, lse_c)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert torch.equal(out_a, out_c) and torch.equal(lse_a, lse_c), "paged attention differs from attention over the view"
    for s in range(n_sessions):
        ids = sel[s, : int(n_sel[s])].cpu().numpy()
        vK, vV = orc.gather(osess[s].repo, osess[s].table, np.ascontiguousarray(ids), budget * 64)
        assert np.array_equal(bits(view_b.k[s]), vK) and np.array_equal(bits(view_b.v[s]), vV)
        ref_out, ref_lse = orc.attend(qb[s], vK, vV, len(ids) * 64)
        assert np.abs(out_b[s].cpu().numpy() - ref_out).max() <= ATTN_ATOL
        assert np.abs(lse_b[s].cpu().numpy() - ref_lse).max() <= ATTN_ATOL


def test_fused_path_flags_out_of_range_ids():
    from paper_2609_04852_b200.kvmem import E_DEVICE_RANGE
    spec = SMALL
    pool = fill_pool(spec)
    dev = torch.device("cuda", 0)
    q, _ = queries(spec)
    sel = torch.tensor([[1, 5000, 7]], dtype=torch.int32, device=dev)
    n_sel = torch.tensor([3], dtype=torch.int32, device=dev)
    view = pool.new_view(1, 4 * spec.block_tokens)
    out, lse = pool.new_outputs(1, spec.n_q_tokens)
    pool.materialize_attend(q.to(dev), sel, n_sel, view, out, lse)
    assert pool.device_status() == E_DEVICE_RANGE


# ------------------------------------------------------------------ multi-token chunks (tensor-core scoring)

@pytest.mark.parametrize("M,n_blocks,n_sessions", [(32, 200, 1), (40, 300, 1), (17, 517, 2), (64, 256, 1)])
def test_chunked_scoring_matches_oracle(M, n_blocks, n_sessions):
    # M * 4 rows per KV head: one full 128-row panel, ragged panels (160, 68 rows), ragged 256-block tiles
    spec = CONFIGS["batch8"].with_(name="chunk", n_sessions=n_sessions, n_blocks=n_blocks, n_planted=6,
                                   budget_blocks=24, n_q_tokens=M, permute_pages=False)
    lens = [n_blocks - 37 * s for s in range(n_sessions)]
    pool = fill_pool(spec, lens)
    osess = fill_oracle(spec, lens)
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.budget_blocks), spec.budget_blocks, attend=False)
    for s in range(n_sessions):
        R, _ = orc.block_scores(qb[s], osess[s].idx, osess[s].n_blocks)
        assert abs(got["scores"][s, :lens[s]].sum() - M) < 1e-3 * M
        check_scores(got["scores"][s, :lens[s]], R, M)
        ref_sel = orc.select(R, spec.block_tokens, spec.budget_blocks, 1 << 30)
        sel_gpu = got["sel"][s, : int(got["n_sel"][s])]
        check_selection(sel_gpu, R, ref_sel)
        vK, vV = orc.gather(osess[s].repo, osess[s].table, np.ascontiguousarray(sel_gpu), spec.budget_blocks * spec.block_tokens)
        T = len(sel_gpu) * spec.block_tokens
        assert np.array_equal(bits(got["view"].k[s])[:, :, :T], vK[:, :, :T])
        assert np.array_equal(bits(got["view"].v[s])[:, :, :T], vV[:, :, :T])


@pytest.mark.parametrize("M,n_blocks,n_sessions", [(1, 333, 2), (4, 200, 1), (40, 300, 2)])
def test_score_alone_equals_the_scores_select_reports_and_the_oracle(M, n_blocks, n_sessions):
    spec = CONFIGS["batch8"].with_(name="score", n_sessions=n_sessions, n_blocks=n_blocks, n_planted=6,
                                   budget_blocks=24, n_q_tokens=M, permute_pages=False)
    lens = [n_blocks - 41 * s for s in range(n_sessions)]
    pool = fill_pool(spec, lens)
    osess = fill_oracle(spec, lens)
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.budget_blocks), spec.budget_blocks, attend=False)
    sc = torch.full((n_sessions, spec.n_blocks), -1.0, dtype=torch.float32, device="cuda")
    pool.score(q.cuda(), sc)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    sc = sc.cpu().numpy()
    for s in range(n_sessions):
        R, _ = orc.block_scores(qb[s], osess[s].idx, osess[s].n_blocks)
        check_scores(sc[s, :lens[s]], R, M)
        assert np.array_equal(sc[s, :lens[s]], got["scores"][s, :lens[s]])     # same kernels, fixed merge order


# ------------------------------------------------------------------ kernel-variant switches

@pytest.mark.parametrize("name,value,bit_exact", [("pdl", 0, True), ("attend_lookahead", 2, True), ("gather_ctas", 148, True),
                                                  ("attend_splits", 5, False), ("attend_splits", 37, False), ("topk_items", 16, True),
                                                  ("topk_items", 2, True), ("attend_landed", 0, True), ("attend_landed", 1, True)])
def test_kernel_variant_switches_do_not_change_results(name, value, bit_exact):
    # scheduling knobs (launch attributes, tiles in flight, CTA counts) leave every byte alone; a different split count
    # changes only the order of the split-K merge
    from paper_2609_04852_b200 import set_option
    spec = SMALL.with_(n_blocks=700, budget_blocks=333, n_q_tokens=4)
    pool = fill_pool(spec)
    q, _ = queries(spec)
    dev = torch.device("cuda", 0)

    def run():
        sel = torch.zeros(1, 333, dtype=torch.int32, device=dev)
        n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
        pool.select(q.to(dev), _params(budget_blocks=333), sel, n_sel)
        view, view2 = pool.new_view(1, 333 * 64), pool.new_view(1, 333 * 64)
        out, lse = pool.new_outputs(1, 4)
        out2, lse2 = pool.new_outputs(1, 4)
        out3, lse3 = pool.new_outputs(1, 4)
        pool.materialize(sel, n_sel, view)
        pool.view_attend(q.to(dev), view, n_sel, out, lse)
        pool.materialize_attend(q.to(dev), sel, n_sel, view2, out2, lse2)
        pool.paged_attend(q.to(dev), sel, n_sel, out3, lse3)
        torch.cuda.synchronize()
        assert pool.device_status() == 0
        return sel, view.k, view.v, view2.k, view2.v, out, lse, out2, lse2, out3, lse3

    base = run()
    set_option(name, value)
    try:
        got = run()
    finally:
        set_option(name, 1 if name == "pdl" else -1 if name == "attend_landed" else 0)
    for i, (a, b) in enumerate(zip(base, got)):
        if bit_exact or i < 5:
            assert torch.equal(a, b), (name, i)
        else:
            assert (a - b).abs().max().item() <= ATTN_ATOL, (name, i)


# ------------------------------------------------------------------ index in host memory, streamed in tiles

@pytest.mark.parametrize("n_blocks,tile_blocks,M,pinned", [(1000, 256, 4, True), (333, 128, 1, True), (700, 1024, 2, False),
                                                          (2100, 128, 3, True)])
def test_scoring_from_a_host_resident_index_in_tiles(n_blocks, tile_blocks, M, pinned):
    # several tiles with a ragged last one, one tile larger than the index, many tiles (statistics carried across 17)
    from paper_2609_04852_b200 import SelectParams
    spec = SMALL.with_(n_blocks=n_blocks, n_q_tokens=M, budget_blocks=40)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, qb = queries(spec)
    dev = torch.device("cuda", 0)
    idx_host = pool.index(0).cpu().contiguous()                 # [L][G][n_blocks][d]: the index, now in host memory
    assert np.array_equal(bits(idx_host), osess.idx[:, :, :n_blocks])
    if pinned:
        idx_host = idx_host.pin_memory()
    R, _ = orc.block_scores(qb[0], osess.idx, n_blocks)
    scores = torch.full((1, n_blocks), -1.0, dtype=torch.float32, device=dev)
    for _ in range(2):                                          # the second call reuses the staging buffers
        pool.score_host_index(idx_host, n_blocks, q[0].to(dev), scores[0], tile_blocks)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    got = scores.cpu().numpy()[0]
    assert abs(got.sum() - M) < 1e-3 * M
    check_scores(got, R, M)
    # selection from these scores, on the device
    sel = torch.zeros(1, 40, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    pool.topk(scores, _params(budget_blocks=40, n_sink_blocks=1, n_recent_blocks=2), sel, n_sel)
    torch.cuda.synchronize()
    ref_sel = orc.select(R, spec.block_tokens, 40, 1 << 30, 0, 1, 2)
    check_selection(sel.cpu().numpy()[0, : int(n_sel[0])], R, ref_sel, 1, 2)
    # and the same scores as the index in device memory gives, to rounding
    dev_scores = torch.zeros(1, n_blocks, dtype=torch.float32, device=dev)
    pool.score(q.to(dev), dev_scores)
    assert np.allclose(dev_scores.cpu().numpy()[0], got, rtol=1e-4, atol=1e-9)


def test_host_index_argument_errors():
    from paper_2609_04852_b200 import KvmemError
    spec = SMALL.with_(n_blocks=300)
    pool = fill_pool(spec)
    dev = torch.device("cuda", 0)
    idx_host = pool.index(0).cpu().contiguous()
    q, _ = queries(spec)
    scores = torch.zeros(300, dtype=torch.float32, device=dev)
    with pytest.raises(KvmemError):
        pool.score_host_index(idx_host, 300, q[0].to(dev), scores, 100)          # tile not a multiple of 128
    with pytest.raises(KvmemError):
        pool.score_host_index(idx_host, 400, q[0].to(dev), scores, 128)          # more blocks than the index holds
    with pytest.raises(ValueError):
        pool.score_host_index(idx_host.to(dev), 300, q[0].to(dev), scores, 128)  # not a host tensor


# ------------------------------------------------------------------ several sessions, permuted pages

def test_multi_session_ragged_lengths_and_permuted_pages():
    spec = CONFIGS["batch8"].with_(name="batch3", n_sessions=3, n_blocks=150, n_planted=5, budget_blocks=20)
    lens = [150, 97, 130]
    pool = fill_pool(spec, lens)
    osess = fill_oracle(spec, lens)
    q, qb = queries(spec)
    got = _run_step(pool, spec, q.cuda(), _params(budget_blocks=spec.budget_blocks), spec.budget_blocks)
    for s in range(3):
        ref = _oracle_step(spec, osess[s], qb, s, spec.budget_blocks)
        sel_gpu, _ = _compare_step(spec, got, s, ref)
        same = _oracle_step(spec, osess[s], qb, s, spec.budget_blocks, sel_override=sel_gpu)
        _compare_view_and_attention(spec, got, s, same)


def test_gather_in_isolation_with_oracle_ids():
    spec = SMALL
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    ids = np.array([0, 3, 4, 77, 128, 199], np.int32)
    dev = torch.device("cuda", 0)
    sel = torch.from_numpy(ids).to(dev).view(1, -1).contiguous()
    n_sel = torch.tensor([len(ids)], dtype=torch.int32, device=dev)
    view = pool.new_view(1, 8 * spec.block_tokens)
    view.k.fill_(7.0)
    pool.materialize(sel, n_sel, view)
    assert pool.device_status() == 0
    vK, vV = orc.gather(osess.repo, osess.table, ids, 8 * spec.block_tokens)
    T = len(ids) * spec.block_tokens
    assert np.array_equal(bits(view.k[0])[:, :, :T], vK[:, :, :T]) and np.array_equal(bits(view.v[0])[:, :, :T], vV[:, :, :T])
    assert torch.all(view.k[0][:, :, T:] == 7.0)                 # tokens past the view are untouched


def test_out_of_range_ids_are_flagged_not_dereferenced():
    from paper_2609_04852_b200.kvmem import E_DEVICE_RANGE
    spec = SMALL
    pool = fill_pool(spec)
    dev = torch.device("cuda", 0)
    sel = torch.tensor([[1, 5000, 7]], dtype=torch.int32, device=dev)
    n_sel = torch.tensor([3], dtype=torch.int32, device=dev)
    view = pool.new_view(1, 4 * spec.block_tokens)
    pool.materialize(sel, n_sel, view)
    assert pool.device_status() == E_DEVICE_RANGE
    assert pool.device_status() == 0                              # reading clears the word


# ------------------------------------------------------------------ host-side errors leave the pool unchanged

def test_argument_and_capacity_errors():
    from paper_2609_04852_b200 import KvmemError, Pool
    from paper_2609_04852_b200.kvmem import E_CAPACITY, E_INVALID, E_STATE, E_UNSUPPORTED
    spec = SMALL.with_(n_blocks=8)
    dev = torch.device("cuda", 0)
    pool = Pool(1, 32, 8, 128, 64, 1, 8, 8, 0)
    from kvmem_workloads import kv_blocks
    K, V = kv_blocks(spec, 0, 0, 4, dev)
    pool.append_blocks(0, K, V, [0, 1, 2, 3])
    with pytest.raises(KvmemError) as e:
        pool.append_blocks(0, K, V, [3, 4, 5, 6])                 # page 3 is taken
    assert e.value.status == E_STATE and pool.session_blocks(0) == 4
    with pytest.raises(KvmemError) as e:
        pool.append_blocks(0, K[:100], V[:100])                   # partial block
    assert e.value.status == E_INVALID
    pool.append_blocks(0, K, V)
    with pytest.raises(KvmemError) as e:
        pool.append_blocks(0, K, V)                               # session and pool are full
    assert e.value.status == E_CAPACITY and pool.session_blocks(0) == 8
    q, _ = queries(spec)
    sel = torch.zeros(1, 2, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(KvmemError) as e:
        pool.select(q.cuda(), _params(budget_blocks=4), sel, n_sel)   # sel_stride 2 < k = 4
    assert e.value.status == E_CAPACITY
    with pytest.raises(KvmemError) as e:
        Pool(1, 32, 5, 128, 64, 1, 8, 8, 0)                       # 32 % 5 != 0
    assert e.value.status == E_INVALID
    q17 = torch.zeros(1, 17, 1, 32, 128, dtype=torch.bfloat16, device=dev)
    view = pool.new_view(1, 8 * 64)
    out, lse = pool.new_outputs(1, 17)
    with pytest.raises(KvmemError) as e:
        pool.view_attend(q17, view, n_sel, out, lse)              # 17 tokens x 4 heads per KV head > 64 rows
    assert e.value.status == E_UNSUPPORTED
    pool.session_reset(0)
    assert pool.session_blocks(0) == 0
    pool.append_blocks(0, K, V)
    assert pool.session_blocks(0) == 4 and pool.device_status() == 0


# ------------------------------------------------------------------ the whole step with host buffers

@pytest.mark.parametrize("pinned", [True, False])
def test_recall_step_with_host_buffers_equals_the_device_calls(pinned):
    """kvmem_recall_step_host: query from host memory, O and LSE into host memory.  Pinned result buffers are written by
    the step's last kernel directly, pageable ones through the staging copies; both must give the bytes of
    kvmem_select + kvmem_materialize_attend on device buffers, and match the oracle."""
    spec = SMALL.with_(n_blocks=300, n_planted=12, budget_blocks=12, n_q_tokens=4)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    dev = torch.device("cuda", 0)
    q, qb = queries(spec)
    prm = _params(budget_blocks=12)
    sel = torch.zeros(1, 12, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    view = pool.new_view(1, 12 * 64)
    out, lse = pool.new_outputs(1, 4)
    pool.select(q.to(dev), prm, sel, n_sel)
    pool.materialize_attend(q.to(dev), sel, n_sel, view, out, lse)
    torch.cuda.synchronize()
    q_host = q.clone().pin_memory() if pinned else q.clone()
    out_host = torch.full(out.shape, float("nan"), dtype=torch.float32)
    lse_host = torch.full(lse.shape, float("nan"), dtype=torch.float32)
    if pinned:
        out_host, lse_host = out_host.pin_memory(), lse_host.pin_memory()
    sel2 = torch.zeros_like(sel)
    n_sel2 = torch.zeros_like(n_sel)
    view2 = pool.new_view(1, 12 * 64)
    for _ in range(2):                                          # the second call reuses the staging buffer
        pool.recall_step_host(q_host, prm, sel2, n_sel2, view2, out_host, lse_host)      # synchronous
    assert pool.device_status() == 0
    assert torch.equal(sel2, sel) and torch.equal(view2.k, view.k) and torch.equal(view2.v, view.v)
    assert torch.equal(out_host, out.cpu()) and torch.equal(lse_host, lse.cpu())
    ref = _oracle_step(spec, osess, qb, 0, 12)
    assert np.array_equal(sel2.cpu().numpy()[0], ref["sel"])     # budget = planted blocks: a resolvable gap
    assert np.abs(out_host.numpy()[0] - ref["out"]).max() <= ATTN_ATOL and np.abs(lse_host.numpy()[0] - ref["lse"]).max() <= ATTN_ATOL
