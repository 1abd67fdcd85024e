"""Whole-step parity cases beyond the five benchmark shapes: more than one scored layer (the mean over (l, h) of
Eq. "kvmem-block-score" on the GPU, and every later stage with L > 1), a session that is reset and refilled, ids
outside the session in both gather variants, and the in-block key layout against the raw-key definition of the
position-consistent view (Sec. 4.4)."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, Guards, bits, check_rotated_keys, fill_oracle, fill_pool, full_step, queries
from kvmem_workloads import CONFIGS, kv_blocks, page_table
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu

SMALL = CONFIGS["tiny"].with_(name="small", n_blocks=200, n_planted=6, budget_blocks=24)


# ------------------------------------------------------------------ more than one scored layer

@pytest.mark.parametrize("L,G,H,M,n_blocks,budget", [(2, 8, 32, 4, 200, 24), (4, 4, 16, 4, 333, 40), (2, 8, 32, 1, 130, 130)],
                         ids=["L2G8H32", "L4G4H16", "L2-everything-selected"])
def test_whole_step_with_several_scored_layers(L, G, H, M, n_blocks, budget):
    """select, materialize, view_attend, materialize_attend and paged_attend with L > 1: the score is the mean over
    layers and heads, every layer has its own pages, index rows, view rows and outputs."""
    spec = SMALL.with_(name=f"L{L}", n_layers=L, n_kv_heads=G, n_q_heads=H, n_q_tokens=M, n_blocks=n_blocks,
                       n_planted=6, budget_blocks=budget)
    modes = full_step(spec, qsets=(0, 1, 2))
    assert len(modes) == 3
    modes = full_step(spec, qsets=(0,), gap_forced_budget=min(spec.n_planted, budget), n_sink=1, n_recent=2)
    assert len(modes) == 1


def test_layers_are_not_mixed_up():
    """With L = 2, zeroing layer 1 of the query must leave layer 0's attention outputs unchanged and change the scores:
    a kernel that read the wrong layer's rows would not show that."""
    from paper_2609_04852_b200 import SelectParams
    spec = SMALL.with_(name="L2mix", n_layers=2, n_q_tokens=2, n_blocks=96, budget_blocks=96)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    q, _ = queries(spec)
    q2 = q.clone()
    q2[:, :, 1] = 0
    g = Guards(dev)
    outs = []
    for qq in (q, q2):
        sel, n_sel = g.empty((1, 96), torch.int32), g.empty((1,), torch.int32)
        scores = g.empty((1, 96), torch.float32)
        out, lse = g.outputs(pool, 1, 2)
        pool.select(qq.to(dev), SelectParams(96, 1 << 30, 0, 0, 0), sel, n_sel, scores)
        pool.paged_attend(qq.to(dev), sel, n_sel, out, lse)
        torch.cuda.synchronize()
        R, _ = orc.block_scores(bits(qq)[0], osess.idx, 96)
        assert np.abs(scores.cpu().numpy()[0] - R).max() <= 1e-3 * R.max()
        outs.append((out.clone(), lse.clone(), scores.clone()))
    g.check()
    assert torch.equal(outs[0][0][:, :, 0], outs[1][0][:, :, 0]) and torch.equal(outs[0][1][:, :, 0], outs[1][1][:, :, 0])
    assert not torch.equal(outs[0][2], outs[1][2])
    # layer 1 with a zero query: uniform attention, lse = ln T
    T = 96 * spec.block_tokens
    assert (outs[1][1][:, :, 1] - np.log(T)).abs().max().item() <= ATTN_ATOL
    assert pool.device_status() == 0


# ------------------------------------------------------------------ reset and refill

def test_reset_session_is_empty_on_the_device_and_its_pages_can_be_reused():
    """After kvmem_session_reset the device sees an empty session (select gives n_sel = 0, status clean, nothing read),
    and the freed pages can go to another session without the first one reaching them."""
    from paper_2609_04852_b200 import Pool, SelectParams
    spec = SMALL.with_(name="reset", n_sessions=2, n_blocks=40, n_planted=3, budget_blocks=8, n_q_tokens=2)
    dev = torch.device("cuda", 0)
    pool = Pool(1, 32, 8, 128, 64, 2, 40, 40, 0)                 # 40 pages in all: session 1 can only live in session 0's old pages
    K0, V0 = kv_blocks(spec, 0, 0, 40, dev)
    pool.append_blocks(0, K0, V0)
    q, qb = queries(spec)
    qd = q.to(dev)
    g = Guards(dev)
    sel, n_sel = g.empty((1, 8), torch.int32, fill=-1), g.empty((1,), torch.int32, fill=77)
    prm = SelectParams(8, 1 << 30, 0, 0, 0)
    pool.select(qd[0:1], prm, sel, n_sel)
    assert int(n_sel.item()) == 8
    pool.session_reset(0)
    assert pool.session_blocks(0) == 0
    sel.fill_(-1)
    pool.select(qd[0:1], prm, sel, n_sel)                        # empty session: nothing selected, nothing flagged
    out, lse = g.outputs(pool, 1, 2)
    pool.paged_attend(qd[0:1], sel, n_sel, out, lse)
    torch.cuda.synchronize()
    assert int(n_sel.item()) == 0 and bool((sel == -1).all())
    assert bool((out == 0).all()) and bool(torch.isneginf(lse).all())
    assert pool.device_status() == 0
    # session 1 takes over the pages; its step must match the oracle on session 1's bytes
    K1, V1 = kv_blocks(spec, 1, 0, 40, dev)
    pool.append_blocks(1, K1, V1)
    ospec = spec.with_(n_sessions=1)
    repo = orc.Repository.empty(40, 64, 1, 8, 128)
    table = np.arange(40, dtype=np.int32)
    repo.place(bits(K1), bits(V1), table)
    idx = orc.mean_k_index(bits(K1), 64)
    assert np.array_equal(bits(pool.index(1)), idx)
    scores = g.empty((1, 40), torch.float32)
    view = g.view(pool, 1, 8 * 64)
    pool.select(qd[1:2], prm, sel, n_sel, scores, session_first=1)
    pool.materialize(sel, n_sel, view, session_first=1)
    out1, lse1 = g.outputs(pool, 1, 2)
    pool.view_attend(qd[1:2], view, n_sel, out1, lse1)
    torch.cuda.synchronize()
    g.check()
    R, _ = orc.block_scores(qb[1], idx, 40)
    ref_sel = orc.select(R, 64, 8, 1 << 30)
    assert np.array_equal(sel.cpu().numpy()[0], ref_sel)
    vK, vV = orc.gather(repo, table, ref_sel, 8 * 64)
    assert np.array_equal(bits(view.k[0]), vK) and np.array_equal(bits(view.v[0]), vV)
    ro, rl = orc.attend(qb[1], vK, vV, 8 * 64)
    assert np.abs(out1.cpu().numpy()[0] - ro).max() <= ATTN_ATOL and np.abs(lse1.cpu().numpy()[0] - rl).max() <= ATTN_ATOL
    # session 0 is still empty on the device although the pages are live again
    pool.select(qd[0:1], prm, sel, n_sel)
    torch.cuda.synchronize()
    assert int(n_sel.item()) == 0 and pool.device_status() == 0 and ospec.n_sessions == 1


# ------------------------------------------------------------------ ids outside the session

@pytest.mark.parametrize("gather_mode", [1, 0])
def test_both_gather_variants_skip_an_id_outside_the_session(gather_mode):
    from paper_2609_04852_b200 import set_option
    from paper_2609_04852_b200.kvmem import E_DEVICE_RANGE
    spec = SMALL
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    dev = torch.device("cuda", 0)
    ids = [1, 5000, 7, -3, 150, 199, 200, 12, 13, 14]             # 5000, -3 and 200 are outside [0, 200)
    good = [j for j, b in enumerate(ids) if 0 <= b < spec.n_blocks]
    sel = torch.tensor([ids], dtype=torch.int32, device=dev)
    n_sel = torch.tensor([len(ids)], dtype=torch.int32, device=dev)
    g = Guards(dev)
    view = g.view(pool, 1, len(ids) * spec.block_tokens)
    view.k.fill_(7.0), view.v.fill_(9.0)
    set_option("gather_mode", gather_mode)
    try:
        pool.materialize(sel, n_sel, view)
        assert pool.device_status() == E_DEVICE_RANGE
    finally:
        set_option("gather_mode", 1)
    g.check()
    B = spec.block_tokens
    for j, b in enumerate(ids):
        kj, vj = view.k[0][:, :, j * B:(j + 1) * B], view.v[0][:, :, j * B:(j + 1) * B]
        if j in good:
            vK, vV = orc.gather(osess.repo, osess.table, np.array([b], np.int32), B)
            assert np.array_equal(bits(kj), vK) and np.array_equal(bits(vj), vV), f"slot {j}"
        else:
            assert bool((kj == 7.0).all()) and bool((vj == 9.0).all()), f"slot {j} of a flagged id was written"


# ------------------------------------------------------------------ in-block key layout against the raw-key definition

THETA, WINDOW = 1.0e6, 4096
# One bf16 rounding moves an element by at most 2^-9 of its size, sigma = 2^-9 / sqrt(3).  The definition (Sec. 4.4)
# rounds RoPE(k, p0 + t) once; the in-block formulations round the stored key RoPE(k, t) and then either the query
# rotated back by p0 or the stored key rotated on by p0: three roundings separate a logit of one formulation from the
# definition's.  With |q|^2 = 2 d and unit-variance keys the logit difference has
#   sigma_s = sqrt(3) * (2^-9 / sqrt(3)) * sqrt(sum_c q_c^2 k_c^2) / sqrt(d)  ~  2^-9 * sqrt(2 d) / sqrt(d) = 2.8e-3,
# lse moves by at most the largest logit difference and out by a probability-weighted mean of them, so
# 7 sigma_s = 2e-2 bounds both with room for the largest of a few thousand logits.
REFORMULATION_ATOL = 2e-2


def _fill_in_block_and_raw(spec):
    """A pool with rope_in_block_keys filled from raw keys, and the ORACLE repository of the raw keys themselves."""
    from paper_2609_04852_b200 import Pool
    dev = torch.device("cuda", 0)
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens, 1, spec.n_blocks,
                spec.n_blocks, 0, WINDOW, THETA, rope_in_block_keys=True)
    tab = orc.rope_table(WINDOW, spec.head_dim, THETA)
    table = page_table(spec)[0]
    raw_repo = orc.Repository.empty(spec.n_blocks, spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim)
    for b0 in range(0, spec.n_blocks, 64):
        b1 = min(spec.n_blocks, b0 + 64)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, table[b0:b1].tolist())
        raw_repo.place(bits(K), bits(V), np.ascontiguousarray(table[b0:b1].numpy()))
    torch.cuda.synchronize()
    return pool, raw_repo, tab, table.numpy()


@pytest.mark.parametrize("n_blocks,budget,M,first", [(150, 20, 4, 517), (700, 60, 4, 17), (90, 1, 1, 0), (64, 60, 2, 250)])
def test_in_block_layout_against_the_raw_key_definition(n_blocks, budget, M, first):
    """kvmem_paged_attend_rope (query rotated back per block) and kvmem_materialize_attend_rope (stored keys rotated on
    per block) on a rope_in_block_keys pool, compared with the definition: attention over the view whose keys are the
    RAW keys rotated to their compact positions, one rounding each."""
    spec = SMALL.with_(name="in_block_def", n_blocks=n_blocks, n_planted=5, budget_blocks=budget, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool, raw_repo, tab, table = _fill_in_block_and_raw(spec)
    B = spec.block_tokens
    ids = np.sort(np.random.default_rng(7 * n_blocks).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    qd = q.to(dev)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    T = budget * B
    dK, dV = orc.gather_rope(raw_repo, table, ids, T, first, tab, in_block=False)      # the definition's view
    ref_out, ref_lse = orc.attend(qb[0], dK, dV, T)
    g = Guards(dev)
    out_q, lse_q = g.outputs(pool, 1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out_q, lse_q, first)
    view = g.view(pool, 1, T)
    out_k, lse_k = g.outputs(pool, 1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view, out_k, lse_k, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    for name, o, l in (("query rotated back", out_q, lse_q), ("stored keys rotated on", out_k, lse_k)):
        eo, el = np.abs(o.cpu().numpy()[0] - ref_out).max(), np.abs(l.cpu().numpy()[0] - ref_lse).max()
        assert eo <= REFORMULATION_ATOL and el <= REFORMULATION_ATOL, f"{name}: out {eo:.2e}, lse {el:.2e}"
    # values are never re-encoded: the view's V equals the definition's bit for bit, its K within one bf16 step
    assert np.array_equal(bits(view.v[0]), dV)
    kf, df = view.k[0].float().cpu().numpy(), orc.bf16_bits_to_f32(dK)
    assert np.abs(kf - df).max() <= 2.0 ** -7 * max(np.abs(df).max(), 1.0)


# ------------------------------------------------------------------ a bounded wait that runs out

def test_a_bounded_wait_that_runs_out_sets_the_status_word_and_leaves_the_pool_usable():
    """The kernels' wait routine, given a barrier nobody arrives at and a 2 ms limit, gives up, reports
    KVMEM_E_TIMEOUT through the status word and returns; a normal step on the same pool then matches the oracle."""
    from paper_2609_04852_b200.kvmem import E_TIMEOUT
    spec = SMALL
    pool = fill_pool(spec)
    assert pool.device_status() == 0
    waited = pool.selftest_wait_timeout(2000)
    assert 2_000_000 <= waited < 500_000_000, f"the wait lasted {waited} ns"
    assert pool.device_status() == E_TIMEOUT
    assert pool.device_status() == 0                              # reading clears the word
    modes = full_step(spec, qsets=(0,))                           # a fresh pool in the same context ...
    assert len(modes) == 1
    from paper_2609_04852_b200 import SelectParams                # ... and the pool that saw the timeout still works
    dev = torch.device("cuda", 0)
    q, qb = queries(spec)
    sel = torch.zeros(1, 24, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    pool.select(q.to(dev), SelectParams(24, 1 << 30, 0, 0, 0), sel, n_sel)
    out, lse = pool.new_outputs(1, spec.n_q_tokens)
    pool.paged_attend(q.to(dev), sel, n_sel, out, lse)
    torch.cuda.synchronize()
    osess = fill_oracle(spec)[0]
    R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
    ids = sel.cpu().numpy()[0, : int(n_sel.item())]
    vK, vV = orc.gather(osess.repo, osess.table, np.ascontiguousarray(ids), 24 * spec.block_tokens)
    ro, rl = orc.attend(qb[0], vK, vV, len(ids) * spec.block_tokens)
    assert np.abs(out.cpu().numpy()[0] - ro).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - rl).max() <= ATTN_ATOL
    assert pool.device_status() == 0


# ------------------------------------------------------------------ decode scores at many shapes

@pytest.mark.parametrize("ns,L,G,H,M,n_blocks", [(1, 1, 8, 32, 4, 2048), (1, 1, 8, 32, 4, 5000), (1, 1, 8, 32, 1, 16384),
                                               (3, 1, 8, 32, 2, 700), (1, 2, 8, 32, 4, 333), (1, 4, 4, 16, 4, 150),
                                               (1, 1, 4, 32, 2, 97), (8, 1, 8, 32, 1, 4096), (1, 1, 8, 32, 4, 1)],
                         ids=["128k-shape", "ragged-5000", "1m-shape", "3-sessions", "L2", "L4G4", "GQA8", "batch8-shape", "one-block"])
def test_decode_scores_at_many_shapes(ns, L, G, H, M, n_blocks):
    """kvmem_score for sessions of different length in one call, several layers, other head groupings, one block:
    against the oracle within the score tolerance, nothing written past a session's blocks, and twice in a row with
    identical bits (fixed summation order)."""
    from kvmem_harness import check_scores
    spec = SMALL.with_(name="scores", n_sessions=ns, n_layers=L, n_kv_heads=G, n_q_heads=H, n_q_tokens=M, n_blocks=n_blocks,
                       n_planted=min(6, n_blocks), budget_blocks=1)
    dev = torch.device("cuda", 0)
    lens = [n_blocks if s == 0 else max(1, n_blocks - 37 * s) for s in range(ns)]        # ragged session lengths
    pool = fill_pool(spec, lens)
    osess = fill_oracle(spec, lens, gen_device=dev)
    q, qb = queries(spec)
    qd = q.to(dev)
    g = Guards(dev)
    runs = []
    for _ in range(2):
        sc = g.empty((ns, n_blocks), torch.float32, fill=-1.0)
        pool.score(qd, sc)
        torch.cuda.synchronize()
        assert pool.device_status() == 0
        runs.append(sc)
    g.check()
    assert torch.equal(runs[0], runs[1]), "two runs of the scorer differ"
    half = g.empty((ns, n_blocks), torch.float32, fill=-1.0)
    pool.score(qd, half, score_scale=0.5)                       # a rank's share of the head mean, scaled in the kernel
    torch.cuda.synchronize()
    for s in range(ns):
        R, _ = orc.block_scores(qb[s], osess[s].idx, lens[s])
        check_scores(runs[0].cpu().numpy()[s, : lens[s]], R, M)
        assert bool((runs[0][s, lens[s]:] == -1.0).all()), "scores past the session's blocks were written"
        assert torch.equal(half[s, : lens[s]] * 2.0, runs[0][s, : lens[s]]), "score_scale must be an exact power-of-two factor here"


# ------------------------------------------------------------------ other block sizes on the passes that read pages

@pytest.mark.parametrize("B,n_blocks,budget,M", [(32, 300, 21, 4), (32, 300, 64, 2), (16, 500, 37, 4), (16, 260, 260, 1),
                                                 (128, 90, 5, 4), (128, 40, 40, 2), (256, 30, 7, 4), (32, 2000, 999, 4)],
                         ids=["B32-ragged", "B32-even", "B16-ragged", "B16-all", "B128", "B128-all", "B256", "B32-long"])
def test_fused_and_copy_free_passes_with_other_block_sizes(B, n_blocks, budget, M):
    """The paper's default block is 32 tokens (Sec. 4.3).  kvmem_materialize_attend and kvmem_paged_attend walk the view in
    64-token tiles: a tile is 64 / B selected blocks (an odd count ends in a partly filled tile) or a slice of one block.
    Against the oracle, and bit for bit against the separate calls."""
    spec = SMALL.with_(name=f"B{B}", block_tokens=B, n_blocks=n_blocks, n_planted=4, budget_blocks=budget, n_q_tokens=M,
                       max_view_tokens=1 << 30)
    modes = full_step(spec, qsets=(0, 1))
    assert len(modes) == 2


@pytest.mark.parametrize("B,n_blocks,budget,first", [(32, 200, 21, 517), (16, 300, 37, 0), (128, 40, 9, 64)])
def test_copy_free_position_consistent_attention_with_other_block_sizes(B, n_blocks, budget, first):
    """kvmem_paged_attend_rope over raw keys (each key fragment rotated to its compact position on the way to the tensor
    cores) with 16-, 32- and 128-token blocks, against attention over the oracle's position-consistent view."""
    from test_gpu_rope import SPEC as RSPEC, _fill_both
    spec = RSPEC.with_(name=f"ropeB{B}", block_tokens=B, n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=4)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    ids = np.sort(np.random.default_rng(B + n_blocks).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    g = Guards(dev)
    out, lse = g.outputs(pool, 1, 4)
    pool.paged_attend_rope(q.to(dev), sel, n_sel, out, lse, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    vK, vV = orc.gather_rope(repo, table, ids, budget * B, first, tab)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, budget * B)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL


def test_execution_cache_with_32_token_blocks():
    """Cache update and attention over the cache's page table with the paper's default block size."""
    from test_gpu_rope import SPEC as RSPEC, THETA, WINDOW, _fill_both
    from test_gpu_view_cache import _compare, _working_sets
    spec = RSPEC.with_(name="cacheB32", block_tokens=32, n_blocks=120, budget_blocks=20, n_q_tokens=4)
    pool, repo, _, tab, table = _fill_both(spec)
    dev = torch.device("cuda", 0)
    cap = 23
    cache = pool.new_view_cache(cap, 2, 131)
    ocache = orc.ViewCache(repo, cap)
    sets = _working_sets(np.random.default_rng(5), spec.n_blocks, [20, 21, 23, 7, 20])
    q, qb = queries(spec)
    for step, sel in enumerate(sets):
        ids = torch.zeros(cap, dtype=torch.int32)
        ids[: len(sel)] = torch.from_numpy(sel)
        cache.update(0, ids.to(dev), torch.tensor([len(sel)], dtype=torch.int32, device=dev))
        stats_ref = ocache.update(repo, table, sel, 2, 131, tab)
        _compare(cache, ocache, stats_ref, step)
        out, lse = pool.new_outputs(1, 4)
        cache.attend(q[0].to(dev), out[0], lse[0])
        torch.cuda.synchronize()
        vK, vV = ocache.view(cap * 32)
        O, LSE = orc.attend(qb[0], vK, vV, len(sel) * 32)
        assert np.abs(out[0].cpu().numpy() - O).max() <= ATTN_ATOL and np.abs(lse[0].cpu().numpy() - LSE).max() <= ATTN_ATOL, step
    assert pool.device_status() == 0 and THETA > 0 and WINDOW > 0


# ------------------------------------------------------------------ more than 16 query rows per KV head

@pytest.mark.parametrize("M,G,H,n_blocks,budget", [(8, 8, 32, 300, 40), (4, 4, 32, 300, 40), (5, 8, 32, 200, 24), (16, 8, 32, 300, 40),
                                                  (13, 8, 32, 150, 150), (8, 4, 32, 700, 333), (2, 8, 32, 64, 1)],
                         ids=["M8-32rows", "GQA8-32rows", "M5-20rows", "M16-64rows", "M13-52rows-all", "GQA8-64rows-long", "M2-8rows"])
def test_attention_with_up_to_64_query_rows_per_kv_head(M, G, H, n_blocks, budget):
    """1 + 7 draft tokens with GQA 4, or 4 tokens with GQA 8, exceed one 16-row MMA tile.  The attention kernels then run
    two or four row tiles over the same K/V stream (a row count that does not fill the last tile included): every stage
    against the oracle, the fused and copy-free passes bit for bit against the separate calls."""
    spec = SMALL.with_(name=f"rows{M * H // G}", n_q_tokens=M, n_kv_heads=G, n_q_heads=H, n_blocks=n_blocks, n_planted=5,
                       budget_blocks=budget)
    modes = full_step(spec, qsets=(0, 1))
    assert len(modes) == 2


def test_thirty_two_rows_at_32_token_blocks_and_two_sessions():
    spec = SMALL.with_(name="rows32B32", n_sessions=2, block_tokens=32, n_q_tokens=8, n_blocks=260, n_planted=4, budget_blocks=37,
                       max_view_tokens=1 << 30)
    assert len(full_step(spec, qsets=(0,))) == 2


# ------------------------------------------------------------------ raw keys rotated inside the fused pass

@pytest.mark.parametrize("B,n_blocks,budget,M,first,L", [(64, 150, 20, 4, 517, 1), (64, 700, 60, 4, 17, 1), (64, 90, 1, 1, 0, 1), (64, 64, 63, 2, 64, 1),
                                                        (32, 200, 21, 4, 131, 1), (16, 300, 37, 2, 0, 1), (128, 40, 9, 4, 64, 1),
                                                        (64, 120, 33, 3, 200, 2), (32, 90, 50, 4, 7, 2)])
def test_position_consistent_view_and_attention_in_one_pass_over_raw_keys(B, n_blocks, budget, M, first, L):
    """kvmem_materialize_attend_rope on a pool of raw keys: the warps that attend over a tile rotate its keys to their
    compact positions (angles composed from the table rows of the warp's first position and of the offset inside its
    share) and hand them back for the store.  Values are copied bit for bit; a rotated key may differ from the defined code
    (oracle gather with RoPE) by one bf16 rounding step on a small fraction of the elements; the results are those of
    attention over the defined view within the attention tolerance, and they are the copy-free pass's bit for bit."""
    from test_gpu_rope import SPEC as RSPEC, _fill_both
    spec = RSPEC.with_(name=f"rawfusedB{B}L{L}", block_tokens=B, n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=M, n_layers=L)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    ids = np.sort(np.random.default_rng(3 * n_blocks + B).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    qd = q.to(dev)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    T = budget * B
    g = Guards(dev)
    view = g.view(pool, 1, T)
    out, lse = g.outputs(pool, 1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view, out, lse, first)
    view2 = g.view(pool, 1, T)
    out2, lse2 = g.outputs(pool, 1, M)
    pool.materialize_rope(sel, n_sel, view2, first)
    pool.view_attend(qd, view2, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    vK, vV = orc.gather_rope(repo, table, ids, T, first, tab)
    check_rotated_keys(bits(view.k[0]), vK)
    assert np.array_equal(bits(view.v[0]), vV)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, T)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    # the separate calls rotate by the table's own rows: their view IS the defined code
    assert np.array_equal(bits(view2.k[0]), vK) and torch.equal(view.v, view2.v)
    assert np.abs(out2.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse2.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    out3, lse3 = g.outputs(pool, 1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out3, lse3, first)
    torch.cuda.synchronize()
    g.check()
    assert torch.equal(out3, out) and torch.equal(lse3, lse), "copy-free and one-pass rotate the same fragments the same way"


# ------------------------------------------------------------------ incremental contiguous view

@pytest.mark.parametrize("gather_mode,B", [(1, 64), (0, 64), (1, 32)])
def test_incremental_view_over_a_sequence_of_working_sets(gather_mode, B):
    """kvmem_materialize_delta against the oracle's view_update over overlapping working sets: the view equals the plain
    gather of the newest set after every step, the counts are the oracle's, and a slot whose block stays is provably not
    written (it is overwritten with a marker before the call and keeps it)."""
    from paper_2609_04852_b200 import set_option
    spec = SMALL.with_(name="delta_view", block_tokens=B, n_blocks=150, n_planted=4, budget_blocks=24, max_view_tokens=1 << 30)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    cap = 24
    g = Guards(dev)
    view = g.view(pool, 1, cap * B)
    stats = g.empty((1, 3), torch.int32)
    oK = np.zeros((1, spec.n_kv_heads, cap * B, spec.head_dim), np.uint16)
    oV = np.zeros_like(oK)
    rng = np.random.default_rng(21)
    from test_gpu_view_cache import _working_sets
    sets = _working_sets(rng, spec.n_blocks, [20, 20, 24, 7, 20, 24, 24, 1])
    sets.insert(3, sets[2].copy())                        # an unchanged working set
    sets.append(np.concatenate([sets[-1], np.array([140, 141], np.int32)]))      # pure append behind an unchanged prefix
    prev = np.zeros(0, np.int32)
    set_option("gather_mode", gather_mode)
    try:
        for step, sel in enumerate(sets):
            def dev_ids(a):
                t = torch.zeros(1, cap, dtype=torch.int32)
                t[0, : len(a)] = torch.from_numpy(np.ascontiguousarray(a, np.int32))
                return t.to(dev), torch.tensor([len(a)], dtype=torch.int32, device=dev)
            p_ids, p_n = dev_ids(prev)
            s_ids, s_n = dev_ids(sel)
            action, _ = orc.view_delta_plan(prev, sel)
            stay = [j for j in range(len(sel)) if action[j] == 0]
            marker = torch.tensor(-7.0, dtype=torch.bfloat16)
            for j in stay[:2]:                             # a slot that stays must not be written: it keeps a marker
                view.k[0, :, :, j * B:(j + 1) * B] = marker
            pool.materialize_delta(p_ids, p_n, s_ids, s_n, view, stats)
            torch.cuda.synchronize()
            assert pool.device_status() == 0
            g.check()
            counts = orc.view_update(osess.repo, osess.table, oK, oV, prev, sel)
            assert stats.cpu().numpy()[0].tolist() == counts.tolist(), step
            T = len(sel) * B
            for j in stay[:2]:
                assert bool((view.k[0, :, :, j * B:(j + 1) * B] == marker).all()), f"step {step}: slot {j} stays but was written"
                view.k[0, :, :, j * B:(j + 1) * B] = torch.from_numpy(oK[:, :, j * B:(j + 1) * B].view(np.int16)).view(torch.bfloat16).to(dev)
            gK, gV = orc.gather(osess.repo, osess.table, sel, cap * B)
            assert np.array_equal(bits(view.k[0])[:, :, :T], gK[:, :, :T]) and np.array_equal(bits(view.v[0])[:, :, :T], gV[:, :, :T]), step
            assert np.array_equal(oK[:, :, :T], gK[:, :, :T])
            prev = sel
    finally:
        set_option("gather_mode", 1)


# ------------------------------------------------------------------ in-block key layout with other block sizes (copy-free pass)

@pytest.mark.parametrize("B,n_blocks,budget,M,first", [(32, 200, 21, 4, 131), (32, 300, 128, 2, 0), (16, 300, 37, 4, 17), (128, 40, 9, 4, 64),
                                                      (32, 64, 1, 1, 5)])
def test_query_rotating_copy_free_attention_with_other_block_sizes(B, n_blocks, budget, M, first):
    """kvmem_paged_attend_rope on a pool whose pages hold RoPE(k, offset in block), with 16-, 32- and 128-token blocks: every
    block of a 64-token tile has its own compact position, so the query is rotated back once per block.  Against the
    oracle's statement of the same formulation at the attention tolerance."""
    from test_gpu_rope_in_block import SPEC as ISPEC, _fill_both as fill_in_block
    spec = ISPEC.with_(name=f"inblockB{B}", block_tokens=B, n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = fill_in_block(spec, encoded=False)
    ids = np.sort(np.random.default_rng(11 * n_blocks + B).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    T = budget * B
    g = Guards(dev)
    out, lse = g.outputs(pool, 1, M)
    pool.paged_attend_rope(q.to(dev), sel, n_sel, out, lse, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    pK, pV = orc.gather(repo, table, ids, T)
    ro, rl = orc.attend_qrot(qb[0], pK, pV, T, B, first, tab)
    assert np.abs(out.cpu().numpy()[0] - ro).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - rl).max() <= ATTN_ATOL
    # and the position-consistent view of the same blocks (one rotation per block) gives the same attention within the
    # rounding that separates the two formulations
    vK, vV = orc.gather_rope(repo, table, ids, T, first, tab, in_block=True)
    do, dl = orc.attend(qb[0], vK, vV, T)
    assert np.abs(out.cpu().numpy()[0] - do).max() <= REFORMULATION_ATOL and np.abs(lse.cpu().numpy()[0] - dl).max() <= REFORMULATION_ATOL


# ------------------------------------------------------------------ position-consistent FP8 view

@pytest.mark.parametrize("in_block,k,M,first,k_scale,v_scale", [(False, 20, 4, 517, 1.0, 1.0), (False, 33, 1, 0, 0.5, 0.25),
                                                                (True, 20, 4, 131, 1.0, 1.0), (False, 1, 2, 64, 2.0, 1.0)])
def test_position_consistent_fp8_view(in_block, k, M, first, k_scale, v_scale):
    """kvmem_materialize_fp8_rope: the code of a key is the E4M3 code of the key rotated to its compact position (the
    oracle's position-consistent gather, then its quantiser: both pinned); values as in the plain FP8 view.  Codes byte
    for byte, then FP8 attention over the view against the oracle's."""
    if in_block:
        from test_gpu_rope_in_block import SPEC as RSPEC, _fill_both as fill
        spec = RSPEC.with_(name="fp8rope_ib", n_q_tokens=M)
        pool, repo, idx, tab, table = fill(spec, encoded=False)
    else:
        from test_gpu_rope import SPEC as RSPEC, _fill_both as fill
        spec = RSPEC.with_(name="fp8rope", n_q_tokens=M)
        pool, repo, idx, tab, table = fill(spec)
    dev = torch.device("cuda", 0)
    B = spec.block_tokens
    ids = np.sort(np.random.default_rng(5 + k).choice(spec.n_blocks, size=k, replace=False)).astype(np.int32)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([k], dtype=torch.int32, device=dev)
    cap = k * B
    g = Guards(dev)
    k8 = g.empty((1, spec.n_layers, spec.n_kv_heads, cap, spec.head_dim), torch.uint8)
    v8t = g.empty((1, spec.n_layers, spec.n_kv_heads, cap // 64, spec.head_dim, 64), torch.uint8)
    pool.materialize_fp8_rope(sel, n_sel, k8, v8t, first, k_scale, v_scale)
    q, qb = queries(spec)
    out, lse = g.outputs(pool, 1, M)
    pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out, lse, k_scale, v_scale)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    k_inv, v_inv = float(np.float32(1.0) / np.float32(k_scale)), float(np.float32(1.0) / np.float32(v_scale))
    vK, _ = orc.gather_rope(repo, table, ids, cap, first, tab, in_block=in_block)       # the position-consistent bf16 keys
    rK = orc.quantize_e4m3(vK, k_inv)
    _, rV = orc.gather_fp8(repo, table, ids, cap, k_inv, v_inv)                         # values: quantised and transposed per tile
    assert np.array_equal(k8.cpu().numpy()[0], rK), "FP8 codes of the rotated keys differ"
    assert np.array_equal(v8t.cpu().numpy()[0], rV), "FP8 value codes differ"
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, cap, k_scale, v_scale)
    err_o, err_l = np.abs(out.cpu().numpy()[0] - ref_out).max(), np.abs(lse.cpu().numpy()[0] - ref_lse).max()
    assert err_o <= ATTN_ATOL * max(1.0, v_scale) and err_l <= ATTN_ATOL, (err_o, err_l)
