"""The N > 1 plumbing on CPU: two gloo ranks own disjoint sessions, run the oracle on their own
shard with no exchange, and agree on the slowest rank's time."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_04852_b200.sharding import max_over_ranks, owner_of, sessions_for_rank, whole_job_rate


def test_partition_is_disjoint_balanced_and_complete():
    for n in (0, 1, 7, 8, 9, 64):
        for world in (1, 2, 3, 8):
            parts = [sessions_for_rank(n, r, world) for r in range(world)]
            flat = [s for p in parts for s in p]
            assert flat == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
            for s in range(n):
                assert s in parts[owner_of(s, n, world)]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from kvmem_workloads import CONFIGS, kv_blocks, make_queries
        from oracle import kvmem_oracle as orc
        spec = CONFIGS["batch8"].with_(n_sessions=4, n_blocks=24, n_planted=2, budget_blocks=4, permute_pages=False)
        mine = sessions_for_rank(spec.n_sessions, rank, world)
        q_all = make_queries(spec, 0)
        picked = {}
        for s in mine:                                    # the shard's own sessions only, no exchange
            K, _ = kv_blocks(spec, s, 0, spec.n_blocks)
            Kb = K.view(torch.int16).numpy().view(np.uint16)
            idx = orc.mean_k_index(Kb, spec.block_tokens)
            qb = q_all[s].contiguous().view(torch.int16).numpy().view(np.uint16)
            R, _ = orc.block_scores(qb, idx, spec.n_blocks)
            picked[s] = orc.select(R, spec.block_tokens, spec.budget_blocks, spec.max_view_tokens).tolist()
        local_ms = 10.0 + 5.0 * rank
        dist.barrier()
        slowest, = max_over_ranks([local_ms])
        gathered = [None] * world
        dist.all_gather_object(gathered, picked)          # test bookkeeping only
        if rank == 0:
            ret["slowest"] = slowest
            ret["picked"] = {k: v for d in gathered for k, v in d.items()}
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_sessions_and_take_the_max_time():
    world = 2
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        assert ret["slowest"] == 15.0
        picked = dict(ret["picked"])
    assert sorted(picked) == [0, 1, 2, 3] and all(len(v) == 4 for v in picked.values())
    assert whole_job_rate(100, world, 15.0) == 2 * 100 / 0.015


def test_max_over_ranks_without_a_process_group_is_identity():
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


# ---- sharding by KV head inside one session: one all-reduce of the block scores --------------------

def test_head_partition_and_query_head_mapping():
    from paper_2609_04852_b200.sharding import kv_heads_for_rank, query_heads_of
    assert [kv_heads_for_rank(8, r, 4) for r in range(4)] == [(0, 2), (2, 4), (4, 6), (6, 8)]
    assert query_heads_of((2, 4), 4) == (8, 16)
    for bad in ((8, 3), (6, 4)):
        try:
            kv_heads_for_rank(bad[0], 0, bad[1])
        except ValueError:
            continue
        raise AssertionError("uneven head split must be refused")


def _head_worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from kvmem_workloads import CONFIGS, kv_blocks, make_queries
        from oracle import kvmem_oracle as orc
        from paper_2609_04852_b200.sharding import combine_head_shard_scores, kv_heads_for_rank, query_heads_of
        spec = CONFIGS["tiny"].with_(n_blocks=96, n_planted=6, budget_blocks=12, n_q_tokens=2)
        r = spec.n_q_heads // spec.n_kv_heads
        g0, g1 = kv_heads_for_rank(spec.n_kv_heads, rank, world)
        h0, h1 = query_heads_of((g0, g1), r)
        K, V = kv_blocks(spec, 0, 0, spec.n_blocks)
        Kb = K.view(torch.int16).numpy().view(np.uint16)
        Vb = V.view(torch.int16).numpy().view(np.uint16)
        qb = make_queries(spec, 0)[0].contiguous().view(torch.int16).numpy().view(np.uint16)      # [M][L][H][d]
        # this rank's shard: its KV heads of the keys, its query heads of the query
        idx_local = orc.mean_k_index(np.ascontiguousarray(Kb[:, :, g0:g1]), spec.block_tokens)
        q_local = np.ascontiguousarray(qb[:, :, h0:h1])
        R_local, _ = orc.block_scores(q_local, idx_local, spec.n_blocks)
        # the library's scoring kernel applies the 1/world share itself (score_scale); the oracle's R_local is scaled here
        R = combine_head_shard_scores(torch.from_numpy(R_local.astype(np.float32)) * (1.0 / world), world).numpy()
        sel = orc.select(R, spec.block_tokens, spec.budget_blocks, spec.max_view_tokens)
        # attention over the own heads only
        table = np.arange(spec.n_blocks, dtype=np.int32)
        repo = orc.Repository.empty(spec.n_blocks, spec.block_tokens, spec.n_layers, g1 - g0, spec.head_dim)
        repo.place(np.ascontiguousarray(Kb[:, :, g0:g1]), np.ascontiguousarray(Vb[:, :, g0:g1]), table)
        T = len(sel) * spec.block_tokens
        vK, vV = orc.gather(repo, table, sel, T)
        O_local, lse_local = orc.attend(q_local, vK, vV, T)
        # the unsharded computation, for comparison (every rank can afford it at this size)
        idx = orc.mean_k_index(Kb, spec.block_tokens)
        R_full, _ = orc.block_scores(qb, idx, spec.n_blocks)
        sel_full = orc.select(R_full, spec.block_tokens, spec.budget_blocks, spec.max_view_tokens)
        full = orc.Repository.empty(spec.n_blocks, spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim)
        full.place(Kb, Vb, table)
        fK, fV = orc.gather(full, table, sel_full, T)
        O_full, lse_full = orc.attend(qb, fK, fV, T)
        gathered = [None] * world
        dist.all_gather_object(gathered, (R.tobytes(), sel.tolist()))      # test bookkeeping only
        ret[rank] = dict(
            r_close=bool(np.allclose(R, R_full, rtol=1e-5, atol=1e-9)), sel_same=sel.tolist() == sel_full.tolist(),
            out_same=bool(np.array_equal(O_local, O_full[:, :, h0:h1]) and np.array_equal(lse_local, lse_full[:, :, h0:h1])),
            ranks_agree=all(g == gathered[0] for g in gathered), r_sum=float(R.sum()))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_kv_heads_with_one_all_reduce_of_the_scores():
    world = 2
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_head_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        res = {k: dict(v) for k, v in ret.items()}
    assert sorted(res) == [0, 1]
    for r in res.values():
        assert r["r_close"] and r["sel_same"] and r["out_same"] and r["ranks_agree"]
        assert abs(r["r_sum"] - 2.0) < 1e-4                 # sum_b R_b = M query tokens


def test_combining_scores_without_ranks_is_the_identity_and_an_injected_reduce_is_used():
    from paper_2609_04852_b200.sharding import combine_head_shard_scores
    x = torch.tensor([0.25, 0.75])
    assert combine_head_shard_scores(x.clone(), 1).tolist() == [0.25, 0.75]
    other = torch.tensor([0.5, 0.5])
    y = combine_head_shard_scores(x.clone() * 0.5, 2, all_reduce=lambda t: t.add_(other * 0.5))
    assert y.tolist() == [0.375, 0.625]


# ---- the benchmark launches its own ranks -----------------------------------------------------------

def _bench(*argv, env=None):
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    e = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(root, "bench.py"), *argv], env=e, capture_output=True, text=True,
                          timeout=300)


def test_bench_with_gpus_2_launches_two_ranks_and_prints_one_line():
    """`bench.py --gpus 2` from a plain command line becomes two ranks (gloo here: the launch and timing plumbing
    without a GPU); rank 0 prints exactly one JSON line with n_gpus = 2 and the slowest rank's time."""
    import json
    res = _bench("--gpus", "2", "--launch-selfcheck", "--steps", "5")
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_slowest_rank"] == 15.0
    assert line["value"] == whole_job_rate(5, 2, 15.0)


def test_bench_refuses_a_rank_count_that_differs_from_gpus():
    res = _bench("--gpus", "2", "--launch-selfcheck", env={"WORLD_SIZE": "1", "RANK": "0"})
    assert res.returncode != 0 and "WORLD_SIZE=1" in (res.stderr + res.stdout)
    assert not [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
