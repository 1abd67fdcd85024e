"""Pools whose pages hold keys rotated by their in-block offset (k' = RoPE(k, t)) on the GPU against the oracle.
The stored keys, the index (built from the raw keys), the position-consistent view and the execution cache are
defined codes and compared bit for bit; the copy-free attention, which rotates the query back once per block
instead of every key forward, is compared with the oracle's attention of the same formulation within the
attention tolerance."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, bits, queries
from kvmem_workloads import CONFIGS, kv_blocks, page_table
from oracle import kvmem_oracle as orc
from test_gpu_view_cache import _compare, _working_sets

pytestmark = pytest.mark.gpu

THETA = 1.0e6
WINDOW = 4096
SPEC = CONFIGS["tiny"].with_(name="rope_in_block", n_blocks=150, n_planted=5, budget_blocks=20, n_q_tokens=4)


def _pool(spec, window=WINDOW):
    from paper_2609_04852_b200 import Pool
    return Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens, spec.n_sessions,
                spec.n_sessions * spec.n_blocks, spec.n_blocks, 0, window, THETA, rope_in_block_keys=True)


def _fill_both(spec, encoded=True, window=WINDOW):
    """encoded: the generator's keys are taken as RoPE-encoded at positions pos0[b] + t and appended as such;
    otherwise they are raw keys appended with kvmem_append_blocks.  Either way the oracle repository holds
    RoPE(raw, t) and the index comes from the raw keys."""
    dev = torch.device("cuda", 0)
    pool = _pool(spec, window)
    tab = orc.rope_table(window, spec.head_dim, THETA)
    B = spec.block_tokens
    pos0 = [(37 * b * B) % (window - B) for b in range(spec.n_blocks)]
    table = page_table(spec)[0]
    repo = orc.Repository.empty(spec.n_blocks, B, spec.n_layers, spec.n_kv_heads, spec.head_dim)
    idx = np.zeros((spec.n_layers, spec.n_kv_heads, spec.n_blocks, spec.head_dim), np.uint16)
    for b0 in range(0, spec.n_blocks, 64):
        b1 = min(spec.n_blocks, b0 + 64)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        Kb, Vb = bits(K), bits(V)
        n_tok = (b1 - b0) * B
        if encoded:
            pool.append_blocks_rope(0, K, V, pos0[b0:b1], table[b0:b1].tolist())
            tok_pos = np.concatenate([np.arange(pos0[b], pos0[b] + B) for b in range(b0, b1)]).astype(np.int32)
            raw = orc.rope_rotate(Kb.reshape(n_tok, -1, spec.head_dim), tok_pos, tab, inverse=True).reshape(Kb.shape)
        else:
            pool.append_blocks(0, K, V, table[b0:b1].tolist())
            raw = Kb
        t_in_block = (np.arange(n_tok) % B).astype(np.int32)
        stored = orc.rope_rotate(np.ascontiguousarray(raw.reshape(n_tok, -1, spec.head_dim)), t_in_block, tab).reshape(Kb.shape)
        repo.place(stored, Vb, np.ascontiguousarray(table[b0:b1].numpy()))
        orc.mean_k_index(raw, B, idx, b0)
    torch.cuda.synchronize()
    return pool, repo, idx, tab, table.numpy()


@pytest.mark.parametrize("encoded", [True, False])
def test_pages_hold_the_in_block_rotation_and_the_index_comes_from_raw_keys(encoded):
    pool, repo, idx, tab, table = _fill_both(SPEC, encoded)
    assert np.array_equal(bits(pool.index(0)), idx), "index must be built from the raw keys"
    dev = torch.device("cuda", 0)
    n = SPEC.n_blocks
    sel = torch.arange(n, dtype=torch.int32, device=dev).view(1, -1)
    n_sel = torch.tensor([n], dtype=torch.int32, device=dev)
    view = pool.new_view(1, n * SPEC.block_tokens)
    pool.materialize(sel, n_sel, view)                       # plain gather: the stored bytes
    vK, vV = orc.gather(repo, table, np.arange(n, dtype=np.int32), n * SPEC.block_tokens)
    assert np.array_equal(bits(view.k[0]), vK), "stored keys differ from RoPE(raw, in-block offset)"
    assert np.array_equal(bits(view.v[0]), vV)
    assert pool.device_status() == 0


@pytest.mark.parametrize("n_blocks,budget,M,first", [(150, 20, 4, 517), (700, 60, 4, 17), (90, 1, 1, 0), (64, 64, 2, 0)])
def test_view_by_block_rotation_and_attention_with_the_query_rotated_back(n_blocks, budget, M, first):
    spec = SPEC.with_(n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    B = spec.block_tokens
    ids = np.sort(np.random.default_rng(n_blocks).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    qd = q.to(dev)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    T = budget * B
    # the position-consistent view: one rotation per block, bit-exact
    view = pool.new_view(1, T)
    pool.materialize_rope(sel, n_sel, view, first)
    out, lse = pool.new_outputs(1, M)
    pool.view_attend(qd, view, n_sel, out, lse)
    torch.cuda.synchronize()
    vK, vV = orc.gather_rope(repo, table, ids, T, first, tab, in_block=True)
    assert np.array_equal(bits(view.k[0]), vK) and np.array_equal(bits(view.v[0]), vV)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, T)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    # copy-free: the stored keys as they are, the query rotated back by each block's compact position
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out2, lse2, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    pK, pV = orc.gather(repo, table, ids, T)
    q_out, q_lse = orc.attend_qrot(qb[0], pK, pV, T, B, first, tab)
    assert np.abs(out2.cpu().numpy()[0] - q_out).max() <= ATTN_ATOL and np.abs(lse2.cpu().numpy()[0] - q_lse).max() <= ATTN_ATOL
    # the two formulations are the same mathematics, one rounding of the keys or of the query apart
    assert (out2 - out).abs().max().item() <= 3e-2 and (lse2 - lse).abs().max().item() <= 3e-2


@pytest.mark.parametrize("n_blocks,budget,M,first", [(150, 20, 4, 517), (700, 60, 4, 17), (90, 1, 1, 0), (64, 64, 2, 0)])
def test_fused_position_consistent_materialise_and_attend(n_blocks, budget, M, first):
    # one pass: every K tile is rotated by its block position in shared memory, stored to the view and attended over
    spec = SPEC.with_(n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    B = spec.block_tokens
    ids = np.sort(np.random.default_rng(n_blocks + 1).choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    q, qb = queries(spec)
    qd = q.to(dev)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    T = budget * B
    view = pool.new_view(1, T)
    out, lse = pool.new_outputs(1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view, out, lse, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    vK, vV = orc.gather_rope(repo, table, ids, T, first, tab, in_block=True)
    assert np.array_equal(bits(view.k[0]), vK), "fused pass: rotated keys differ from the defined code"
    assert np.array_equal(bits(view.v[0]), vV)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, T)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    # the same bytes as the two separate calls
    view2 = pool.new_view(1, T)
    out2, lse2 = pool.new_outputs(1, M)
    pool.materialize_rope(sel, n_sel, view2, first)
    pool.view_attend(qd, view2, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert torch.equal(view2.k, view.k) and torch.equal(view2.v, view.v)
    assert torch.equal(out2, out) and torch.equal(lse2, lse)


def test_query_rotation_really_depends_on_the_compact_position():
    # the same selection at two different first positions must differ (a rotator that ignored p0 would pass the
    # tolerance test only by accident), and each must match its own oracle result
    spec = SPEC.with_(n_blocks=64, budget_blocks=12, n_q_tokens=2)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    ids = np.arange(3, 15, dtype=np.int32)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([12], dtype=torch.int32, device=dev)
    q, qb = queries(spec)
    pK, pV = orc.gather(repo, table, ids, 12 * 64)
    outs = []
    for first in (0, 1000):
        out, lse = pool.new_outputs(1, 2)
        pool.paged_attend_rope(q.to(dev), sel, n_sel, out, lse, first)
        torch.cuda.synchronize()
        ro, rl = orc.attend_qrot(qb[0], pK, pV, 12 * 64, 64, first, tab)
        assert np.abs(out.cpu().numpy()[0] - ro).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - rl).max() <= ATTN_ATOL
        outs.append(lse.clone())
    assert (outs[0] - outs[1]).abs().max().item() > 10 * ATTN_ATOL
    assert pool.device_status() == 0


@pytest.mark.parametrize("max_delta,first_position", [(0, 0), (2, 131)])
def test_execution_cache_loads_and_rebuilds_by_block_rotation(max_delta, first_position):
    pool, repo, _, tab, table = _fill_both(SPEC)
    dev = torch.device("cuda", 0)
    cap = 24
    cache = pool.new_view_cache(cap, max_delta, first_position)
    ocache = orc.ViewCache(repo, cap)
    sets = _working_sets(np.random.default_rng(12), SPEC.n_blocks, [20, 20, 24, 7, 20, 24])
    q, qb = queries(SPEC)
    for step, sel in enumerate(sets):
        ids = torch.zeros(cap, dtype=torch.int32)
        ids[: len(sel)] = torch.from_numpy(sel)
        cache.update(0, ids.to(dev), torch.tensor([len(sel)], dtype=torch.int32, device=dev))
        stats_ref = ocache.update(repo, table, sel, max_delta, first_position, tab, in_block=True)
        _compare(cache, ocache, stats_ref, step)
        out, lse = pool.new_outputs(1, SPEC.n_q_tokens)
        cache.attend(q[0].to(dev), out[0], lse[0])
        torch.cuda.synchronize()
        vK, vV = ocache.view(cap * SPEC.block_tokens)
        O, LSE = orc.attend(qb[0], vK, vV, len(sel) * SPEC.block_tokens)
        assert np.abs(out[0].cpu().numpy() - O).max() <= ATTN_ATOL and np.abs(lse[0].cpu().numpy() - LSE).max() <= ATTN_ATOL, step
    assert pool.device_status() == 0


def test_in_block_layout_needs_a_table_covering_one_block():
    from paper_2609_04852_b200 import KvmemError, Pool
    with pytest.raises(KvmemError):
        Pool(1, 32, 8, 128, 64, 1, 8, 8, 0, 0, 0.0, rope_in_block_keys=True)          # no rotary support at all
    with pytest.raises(KvmemError):
        Pool(1, 32, 8, 128, 64, 1, 8, 8, 0, 32, THETA, rope_in_block_keys=True)       # table shorter than a block
