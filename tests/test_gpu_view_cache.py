"""Execution cache on the GPU against the oracle: working-set reuse with bounded delta re-RoPE (Sec. 4.4).
Slot records, statistics and cache contents (keys are a defined code, values are copies) are compared bit
for bit after every update of a sequence of overlapping working sets; attention over the cache is compared
with the oracle's attention over its own cache within the attention tolerance."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, bits, queries
from kvmem_workloads import CONFIGS
from oracle import kvmem_oracle as orc
from test_gpu_rope import THETA, WINDOW, _fill_both

pytestmark = pytest.mark.gpu

SPEC = CONFIGS["tiny"].with_(name="cache", n_blocks=150, n_planted=5, budget_blocks=20, n_q_tokens=4)


def _working_sets(rng, n_blocks, sizes, keep_frac=0.7):
    """Ascending id lists; each keeps about keep_frac of the previous one."""
    prev = np.sort(rng.choice(n_blocks, size=sizes[0], replace=False))
    out = [prev.astype(np.int32)]
    for n in sizes[1:]:
        n_keep = min(int(round(keep_frac * len(prev))), n)
        keep = rng.choice(prev, size=n_keep, replace=False)
        rest = np.setdiff1d(np.arange(n_blocks), prev)
        new = rng.choice(rest, size=n - n_keep, replace=False)
        prev = np.sort(np.concatenate([keep, new]))
        out.append(prev.astype(np.int32))
    return out


def _cache_pages_token_major(cache):
    """GPU slots [cap][2][L][G][B][d] -> oracle layout ([cap][B][L][G][d] keys, values)."""
    pg = bits(cache.pages())
    return np.ascontiguousarray(pg[:, 0].transpose(0, 3, 1, 2, 4)), np.ascontiguousarray(pg[:, 1].transpose(0, 3, 1, 2, 4))


def _compare(cache, ocache, stats_ref, step):
    sb, sp, sc, vs, n = cache.records()
    assert n == ocache.n_view, step
    assert np.array_equal(cache.stats.cpu().numpy(), stats_ref), (step, cache.stats.cpu().numpy(), stats_ref)
    assert np.array_equal(vs.numpy()[:n], ocache.view_slots[:n]), step
    assert np.array_equal(sb.numpy(), ocache.slot_block), step
    live = ocache.slot_block >= 0
    assert np.array_equal(sp.numpy()[live], ocache.slot_pos[live]) and np.array_equal(sc.numpy()[live], ocache.slot_cnt[live]), step
    gK, gV = _cache_pages_token_major(cache)
    assert np.array_equal(gK[live], ocache.K[live]), f"step {step}: cached keys differ"
    assert np.array_equal(gV[live], ocache.V[live]), f"step {step}: cached values differ"


@pytest.mark.parametrize("max_delta,first_position", [(0, 0), (2, 0), (1000, 131)])
def test_sequence_of_overlapping_working_sets_matches_the_oracle(max_delta, first_position):
    pool, repo, _, tab, table = _fill_both(SPEC)
    dev = torch.device("cuda", 0)
    cap = 24
    cache = pool.new_view_cache(cap, max_delta, first_position)
    ocache = orc.ViewCache(repo, cap)
    rng = np.random.default_rng(11)
    sets = _working_sets(rng, SPEC.n_blocks, [20, 20, 24, 7, 20, 20, 1, 19, 24, 24])
    sets.insert(3, sets[2].copy())                                        # an unchanged working set
    q, qb = queries(SPEC)
    for step, sel in enumerate(sets):
        ids = torch.zeros(cap, dtype=torch.int32)
        ids[: len(sel)] = torch.from_numpy(sel)
        cache.update(0, ids.to(dev), torch.tensor([len(sel)], dtype=torch.int32, device=dev))
        stats_ref = ocache.update(repo, table, sel, max_delta, first_position, tab)
        _compare(cache, ocache, stats_ref, step)
        if max_delta == 0:                                                # always rebuilt: equals the position-consistent gather
            vK, vV = ocache.view(cap * SPEC.block_tokens)
            fK, fV = orc.gather_rope(repo, table, sel, cap * SPEC.block_tokens, first_position, tab)
            assert np.array_equal(vK, fK) and np.array_equal(vV, fV)
        # attention over the cache through its page table
        out, lse = pool.new_outputs(1, SPEC.n_q_tokens)
        cache.attend(q[0].to(dev), out[0], lse[0])
        torch.cuda.synchronize()
        vK, vV = ocache.view(cap * SPEC.block_tokens)
        O, LSE = orc.attend(qb[0], vK, vV, len(sel) * SPEC.block_tokens)
        assert np.abs(out[0].cpu().numpy() - O).max() <= ATTN_ATOL, step
        assert np.abs(lse[0].cpu().numpy() - LSE).max() <= ATTN_ATOL, step
    assert pool.device_status() == 0


def test_cache_fed_by_select_over_consecutive_queries():
    """The ids come from kvmem_select on the device (no host round trip) for a sequence of query sets."""
    from paper_2609_04852_b200 import SelectParams
    from kvmem_workloads import make_queries
    pool, repo, idx, tab, table = _fill_both(SPEC)
    dev = torch.device("cuda", 0)
    cap = SPEC.budget_blocks
    cache = pool.new_view_cache(cap, 3, 0)
    ocache = orc.ViewCache(repo, cap)
    prm = SelectParams(budget_blocks=cap, max_view_tokens=1 << 30, mandatory_tokens=0, n_sink_blocks=2, n_recent_blocks=3)
    sel = torch.zeros(1, cap, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    for step in range(5):
        qd = make_queries(SPEC, step).to(dev)
        pool.select(qd, prm, sel, n_sel)
        cache.update(0, sel[0], n_sel)
        torch.cuda.synchronize()
        # the oracle selects for itself; this workload has a resolvable gap at the boundary, so the ids agree
        R, _ = orc.block_scores(bits(qd.cpu())[0], idx, SPEC.n_blocks)
        ids = orc.select(R, SPEC.block_tokens, cap, 1 << 30, 0, 2, 3)
        assert np.array_equal(sel[0, : int(n_sel[0])].cpu().numpy(), ids), step
        stats_ref = ocache.update(repo, table, ids, 3, 0, tab)
        _compare(cache, ocache, stats_ref, step)
    assert pool.device_status() == 0


def test_too_long_selection_and_bad_arguments_are_reported():
    from paper_2609_04852_b200 import KvmemError
    pool, *_ = _fill_both(SPEC.with_(n_blocks=40))
    dev = torch.device("cuda", 0)
    cache = pool.new_view_cache(8, 1, 0)
    ids = torch.arange(16, dtype=torch.int32, device=dev)
    cache.update(0, ids, torch.tensor([12], dtype=torch.int32, device=dev))   # 12 > 8 slots: clamped and flagged
    assert pool.device_status() == -7
    _, _, _, _, n = cache.records()
    assert n == 8
    cache2 = pool.new_view_cache(8, 1, WINDOW)                                 # compact positions outside the rotary table
    with pytest.raises(KvmemError):
        cache2.update(0, ids, torch.tensor([4], dtype=torch.int32, device=dev))
    with pytest.raises(KvmemError):
        pool.new_view_cache(0, 1, 0)
