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
