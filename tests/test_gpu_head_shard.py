"""Sharding one session by KV head, emulated on one GPU: the two ranks' pools (half of the heads each) run one after
the other, and the all-reduce of the block scores is replaced by adding the other rank's scaled scores (no rank
waits for another inside a kernel, so running them in sequence is the same computation).  The combined scores,
the selection and each rank's share of the attention output are compared with the oracle on the whole session."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, bits, check_scores, fill_oracle, queries
from kvmem_workloads import CONFIGS, kv_blocks, page_table, select_params
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu


def _shard_pool(spec, g0, g1):
    from paper_2609_04852_b200 import Pool
    dev = torch.device("cuda", 0)
    r = spec.n_q_heads // spec.n_kv_heads
    pool = Pool(spec.n_layers, (g1 - g0) * r, g1 - g0, spec.head_dim, spec.block_tokens, 1, spec.n_blocks, spec.n_blocks, 0)
    table = page_table(spec)[0]
    for b0 in range(0, spec.n_blocks, 256):
        b1 = min(spec.n_blocks, b0 + 256)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K[:, :, g0:g1].contiguous(), V[:, :, g0:g1].contiguous(), table[b0:b1].tolist())
    torch.cuda.synchronize()
    return pool


@pytest.mark.parametrize("world,n_blocks,budget,M", [(2, 300, 8, 4), (4, 150, 10, 1)])
def test_head_sharded_step_matches_the_oracle_on_the_whole_session(world, n_blocks, budget, M):
    from paper_2609_04852_b200 import SelectParams
    from paper_2609_04852_b200.sharding import combine_head_shard_scores, head_sharded_step, kv_heads_for_rank, query_heads_of
    spec = CONFIGS["tiny"].with_(name="headshard", n_blocks=n_blocks, n_planted=budget, budget_blocks=budget, n_q_tokens=M)      # budget = planted blocks: a resolvable gap at the boundary
    dev = torch.device("cuda", 0)
    r = spec.n_q_heads // spec.n_kv_heads
    prm = SelectParams(**select_params(spec))
    q, qb = queries(spec)
    ranks = []
    for rank in range(world):
        g0, g1 = kv_heads_for_rank(spec.n_kv_heads, rank, world)
        h0, h1 = query_heads_of((g0, g1), r)
        pool = _shard_pool(spec, g0, g1)
        q_local = q[:, :, :, h0:h1].contiguous().to(dev)
        scores = torch.zeros(1, n_blocks, dtype=torch.float32, device=dev)
        pool.score(q_local, scores, score_scale=1.0 / world)         # the rank's share of the head mean, scaled in the kernel
        ranks.append(dict(pool=pool, q=q_local, h=(h0, h1), own=scores.clone()))
    torch.cuda.synchronize()
    # the oracle on the unsharded session
    osess = fill_oracle(spec)[0]
    R_ref, _ = orc.block_scores(qb[0], osess.idx, n_blocks)
    sel_ref = orc.select(R_ref, spec.block_tokens, budget, spec.max_view_tokens)
    T = len(sel_ref) * spec.block_tokens
    vK, vV = orc.gather(osess.repo, osess.table, sel_ref, T)
    O_ref, lse_ref = orc.attend(qb[0], vK, vV, T)
    combined = []
    for rank, me in enumerate(ranks):
        others = sum(o["own"] for i, o in enumerate(ranks) if i != rank)
        scores = torch.zeros(1, n_blocks, dtype=torch.float32, device=dev)
        sel = torch.zeros(1, budget, dtype=torch.int32, device=dev)
        n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
        view = me["pool"].new_view(1, budget * spec.block_tokens)
        out, lse = me["pool"].new_outputs(1, M)
        head_sharded_step(me["pool"], me["q"], prm, scores, sel, n_sel, view, out, lse, world,
                          all_reduce=lambda t: t.add_(others))
        torch.cuda.synchronize()
        assert me["pool"].device_status() == 0
        check_scores(scores.cpu().numpy()[0], R_ref, M)
        assert np.array_equal(sel.cpu().numpy()[0, : int(n_sel.item())], sel_ref), "planted gap is resolvable: ids must agree"
        h0, h1 = me["h"]
        assert np.abs(out.cpu().numpy()[0] - O_ref[:, :, h0:h1]).max() <= ATTN_ATOL
        assert np.abs(lse.cpu().numpy()[0] - lse_ref[:, :, h0:h1]).max() <= ATTN_ATOL
        # the view holds the rank's own heads of the selected blocks, bit for bit
        g0, g1 = h0 // r, h1 // r
        assert np.array_equal(bits(view.k[0]), vK[:, g0:g1]) and np.array_equal(bits(view.v[0]), vV[:, g0:g1])
        combined.append(scores.cpu().numpy().copy())
    # with two ranks the sum a + b is the same bits in either order: every rank holds identical scores
    if world == 2:
        assert np.array_equal(combined[0], combined[1])
    assert combine_head_shard_scores(torch.ones(2), 1).tolist() == [1.0, 1.0]
