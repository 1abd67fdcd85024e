"""The allocation-free attention entry point (kvmem_view_attend_static).

It exists for hosts that cannot obtain device memory while running (all of HBM already given to a
KV pool, a frozen allocator, a plug-in that only sees one request's buffers).  Its split-K scratch
is a fixed array inside the library that every call shares and that keeps the previous call's
contents, so the check runs two calls in a row, with different queries and view lengths, and
compares each with the ordinary entry point that takes a caller workspace.  Collected last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

from kvmem_harness import ATTN_ATOL, fill_pool, queries
from kvmem_workloads import CONFIGS

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    from paper_2609_04852_b200 import KvmemError, SelectParams
    from paper_2609_04852_b200.kvmem import E_CAPACITY, E_INVALID
    spec = CONFIGS["tiny"].with_(name="noalloc", n_blocks=300, n_planted=6, budget_blocks=150, n_q_tokens=4)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    k = spec.budget_blocks
    sel = torch.zeros(1, k, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    view = pool.new_view(1, k * spec.block_tokens)
    for call, (qset, budget) in enumerate([(0, 150), (1, 37)]):          # second call: other query, shorter view
        q = queries(spec, qset)[0].to(dev)
        pool.select(q, SelectParams(budget, 1 << 30, 0, 0, 0), sel, n_sel)
        pool.materialize(sel, n_sel, view)
        ref_out, ref_lse = pool.new_outputs(1, spec.n_q_tokens)
        pool.view_attend(q, view, n_sel, ref_out, ref_lse)
        out, lse = pool.new_outputs(1, spec.n_q_tokens)
        out.fill_(float("nan"))
        lse.fill_(float("nan"))
        pool.view_attend_static(q, view, n_sel, out, lse)
        torch.cuda.synchronize()
        assert pool.device_status() == 0
        assert int(n_sel.item()) == budget
        assert torch.isfinite(out).all() and torch.isfinite(lse).all(), f"call {call}: output not written"
        assert (out - ref_out).abs().max().item() <= ATTN_ATOL, f"call {call}: outputs differ"
        assert (lse - ref_lse).abs().max().item() <= ATTN_ATOL, f"call {call}: log-sum-exp differs"
        # the same kernels with the same split boundaries ran on both sides: not a bit may differ
        assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse), f"call {call}: results are not bit-identical"

    # more (session, layer, KV head) triples than the built-in scratch covers: refused with a message
    big = CONFIGS["batch8"].with_(name="noalloc2", n_sessions=2, n_blocks=8, n_planted=1, budget_blocks=4)
    pool2 = fill_pool(big)
    q2 = queries(big, 0)[0].to(dev)
    view2 = pool2.new_view(2, 4 * big.block_tokens)
    out2, lse2 = pool2.new_outputs(2, big.n_q_tokens)
    n2 = torch.zeros(2, dtype=torch.int32, device=dev)
    with pytest.raises(KvmemError) as e:
        pool2.view_attend_static(q2, view2, n2, out2, lse2)
    assert e.value.status == E_CAPACITY and "at most 8" in str(e.value)
    # no session at all is an argument error, as it is for the entry point with a caller workspace
    empty = torch.zeros(0, big.n_q_tokens, 1, big.n_q_heads, big.head_dim, dtype=torch.bfloat16, device=dev)
    with pytest.raises(KvmemError) as e:
        pool2.view_attend_static(empty, view2, n2, out2, lse2)
    assert e.value.status == E_INVALID
