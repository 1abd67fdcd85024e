"""The synthetic generator: deterministic, chunk-independent, shaped as the recipe says."""
import numpy as np
import torch

from kvmem_workloads import CONFIGS, kv_blocks, make_queries, page_table, planted_blocks, planted_directions


def test_chunks_are_independent_and_deterministic():
    spec = CONFIGS["tiny"].with_(n_blocks=24)
    K, V = kv_blocks(spec, 0, 0, 24)
    K2, V2 = kv_blocks(spec, 0, 5, 11)
    B = spec.block_tokens
    assert torch.equal(K[5 * B:11 * B], K2) and torch.equal(V[5 * B:11 * B], V2)
    assert K.dtype == torch.bfloat16 and K.shape == (24 * B, 1, 8, 128)
    K3, _ = kv_blocks(spec, 1, 0, 4)
    assert not torch.equal(K3, K[:4 * B])                       # sessions differ


def test_values_look_standard_normal_and_planted_blocks_are_shifted():
    spec = CONFIGS["tiny"].with_(n_blocks=64, n_planted=4)
    K, V = kv_blocks(spec, 0, 0, 64)
    assert abs(V.float().mean()) < 5e-3 and abs(V.float().std() - 1) < 5e-3
    ids, a = planted_blocks(spec, 0)
    assert len(set(ids.tolist())) == 4 and torch.all(a == 3.0)
    u = planted_directions(spec, 0)
    assert torch.allclose(u.norm(dim=-1), torch.ones(1, 8), atol=1e-6)
    proj = torch.einsum("tlgd,lgd->tlg", K.float(), u).view(64, spec.block_tokens, 1, 8).mean(dim=1)
    mask = torch.zeros(64, dtype=torch.bool)
    mask[ids] = True
    assert (proj[mask] > 2.5).all() and (proj[~mask].abs() < 0.7).all()


def test_zipf_shift_decays_with_rank():
    spec = CONFIGS["1m"]
    ids, a = planted_blocks(spec, 0)
    assert len(ids) == 1024 and abs(a[0] - 8.0) < 1e-6 and abs(a[-1] - (8 - 1.1 * np.log(1024))) < 1e-5
    assert torch.all(a[1:] < a[:-1])


def test_queries_and_page_tables():
    spec = CONFIGS["batch8"]
    q = make_queries(spec, 3)
    assert q.shape == (8, 1, 1, 32, 128) and q.dtype == torch.bfloat16
    assert not torch.equal(q, make_queries(spec, 4)) and torch.equal(q, make_queries(spec, 3))
    t = page_table(spec)
    assert t.shape == (8, 4096) and sorted(t.flatten().tolist()) == list(range(8 * 4096))
    assert not torch.equal(t[0], torch.arange(4096, dtype=torch.int32))
    assert torch.equal(page_table(CONFIGS["128k"])[0], torch.arange(2048, dtype=torch.int32))
