"""Parity at the full benchmark sizes (128K, 1M, 8 x 256K), in the launch configuration the
benchmark times.  The oracle gets the same bytes: the generator is bit-identical on CPU and GPU
(checked below), so the history is generated on the device and copied to the host for the oracle.
"""
import numpy as np
import pytest
import torch

from kvmem_harness import bits, check_scores, check_selection, fill_oracle, fill_pool, full_step, queries
from kvmem_workloads import CONFIGS, kv_blocks, planted_blocks, select_params
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu


def test_generator_is_bit_identical_on_cpu_and_gpu():
    spec = CONFIGS["128k"]
    Kc, Vc = kv_blocks(spec, 0, 100, 108, "cpu")
    Kg, Vg = kv_blocks(spec, 0, 100, 108, torch.device("cuda", 0))
    assert torch.equal(Kc, Kg.cpu()) and torch.equal(Vc, Vg.cpu())
    spec = CONFIGS["1m"]
    ids = planted_blocks(spec, 0)[0][:2].tolist()
    for b in ids:
        Kc, _ = kv_blocks(spec, 0, b, b + 1, "cpu")
        Kg, _ = kv_blocks(spec, 0, b, b + 1, torch.device("cuda", 0))
        assert torch.equal(Kc, Kg.cpu())


def _full_step(spec, qsets=(0,), gap_forced_budget=None):
    return full_step(spec, qsets, gap_forced_budget)


def test_config_tiny_full():
    """The small configuration exactly as stated (256 blocks of 64 tokens, one query token, 8 planted blocks, budget 32,
    seed 0), every query set; with the budget at the planted count the boundary gap is wide and the ids must be equal."""
    spec = CONFIGS["tiny"]
    assert (spec.n_blocks, spec.block_tokens, spec.n_q_tokens, spec.n_planted, spec.budget_blocks, spec.seed) == (256, 64, 1, 8, 32, 0)
    _full_step(spec, qsets=tuple(range(spec.n_query_sets)))
    modes = _full_step(spec, qsets=tuple(range(spec.n_query_sets)), gap_forced_budget=spec.n_planted)
    assert modes == ["exact"] * spec.n_query_sets


def test_config_128k_full():
    spec = CONFIGS["128k"]
    _full_step(spec, qsets=(0, 1))
    modes = _full_step(spec, gap_forced_budget=spec.n_planted)       # k = planted count: the boundary gap is wide
    assert modes == ["exact"]


def test_config_1m_full():
    _full_step(CONFIGS["1m"], qsets=(0, 5, 10, 15))


def test_config_batch8_full():
    _full_step(CONFIGS["batch8"], qsets=(0, 5, 10, 15))


def test_config_chunk512_full():
    """512-token chunk against the 1M index: score (tensor cores) -> select -> materialize."""
    from paper_2609_04852_b200 import SelectParams, budget_blocks
    spec = CONFIGS["chunk512"]
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec, gen_device=dev)[0]
    prm_d = select_params(spec)
    prm = SelectParams(**prm_d)
    B = spec.block_tokens
    k = budget_blocks(prm, B, spec.n_blocks)
    sel = torch.zeros(1, k, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    scores = torch.zeros(1, spec.n_blocks, dtype=torch.float32, device=dev)
    view = pool.new_view(1, k * B)
    q, qb = queries(spec, 0)
    pool.select(q.to(dev), prm, sel, n_sel, scores)
    pool.materialize(sel, n_sel, view)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
    check_scores(scores.cpu().numpy()[0], R, spec.n_q_tokens)
    ref_sel = orc.select(R, B, prm_d["budget_blocks"], prm_d["max_view_tokens"])
    sel_gpu = sel.cpu().numpy()[0, : int(n_sel.item())]
    assert len(sel_gpu) == k
    check_selection(sel_gpu, R, ref_sel)
    assert set(planted_blocks(spec, 0)[0].tolist()) <= set(sel_gpu.tolist())
    vK, vV = orc.gather(osess.repo, osess.table, np.ascontiguousarray(sel_gpu), k * B)
    assert np.array_equal(bits(view.k[0]), vK) and np.array_equal(bits(view.v[0]), vV)


def test_workspace_scaling_recipe_at_reduced_size():
    """The workspace-scaling recipe (32-token blocks, 128-token query, 64K view) with a 20K-block history: the
    general top-k path (more than 16,384 blocks) fed by tensor-core scoring, then the gather of 32-token blocks."""
    from paper_2609_04852_b200 import SelectParams, budget_blocks
    spec = CONFIGS["table4"].with_(name="table4-small", n_blocks=20000, n_planted=64, budget_blocks=300)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec, gen_device=dev)[0]
    prm_d = select_params(spec)
    prm = SelectParams(**prm_d)
    B = spec.block_tokens
    k = budget_blocks(prm, B, spec.n_blocks)
    assert B == 32 and k == 300
    sel = torch.zeros(1, k, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    scores = torch.zeros(1, spec.n_blocks, dtype=torch.float32, device=dev)
    view = pool.new_view(1, k * B)
    q, qb = queries(spec, 0)
    pool.select(q.to(dev), prm, sel, n_sel, scores)
    pool.materialize(sel, n_sel, view)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert np.array_equal(bits(pool.index(0)), osess.idx)
    R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
    check_scores(scores.cpu().numpy()[0], R, spec.n_q_tokens)
    ref_sel = orc.select(R, B, prm_d["budget_blocks"], prm_d["max_view_tokens"])
    sel_gpu = sel.cpu().numpy()[0, : int(n_sel.item())]
    assert len(sel_gpu) == k
    check_selection(sel_gpu, R, ref_sel)
    assert set(planted_blocks(spec, 0)[0].tolist()) <= set(sel_gpu.tolist())
    vK, vV = orc.gather(osess.repo, osess.table, np.ascontiguousarray(sel_gpu), k * B)
    assert np.array_equal(bits(view.k[0]), vK) and np.array_equal(bits(view.v[0]), vV)
