"""FP8 (E4M3) execution view on the GPU against the oracle: the codes written by kvmem_materialize_fp8 are
compared byte for byte (a quantised code: both sides round the same fp32 product), attention over the FP8 view
within the attention tolerance of the oracle's attention over the same codes."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, fill_oracle, fill_pool, queries
from kvmem_workloads import CONFIGS
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu

SPEC = CONFIGS["tiny"].with_(name="fp8", n_blocks=150, n_planted=5, budget_blocks=20, n_q_tokens=4)


def _ids(rng, n_blocks, k):
    return np.sort(rng.choice(n_blocks, size=k, replace=False)).astype(np.int32)


@pytest.mark.parametrize("k,cap_blocks,M,k_scale,v_scale", [(20, 20, 4, 1.0, 1.0), (33, 40, 1, 0.5, 0.25), (1, 1, 2, 2.0, 1.0),
                                                           (150, 150, 3, 1.0, 0.0625)])
def test_fp8_view_bytes_and_attention(k, cap_blocks, M, k_scale, v_scale):
    spec = SPEC.with_(n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)[0]
    rng = np.random.default_rng(k)
    ids = _ids(rng, spec.n_blocks, k)
    B, cap = spec.block_tokens, cap_blocks * spec.block_tokens
    sel = torch.full((1, cap_blocks), -1, dtype=torch.int32)
    sel[0, :k] = torch.from_numpy(ids)
    sel = sel.to(dev)
    n_sel = torch.tensor([k], dtype=torch.int32, device=dev)
    k8, v8t = pool.new_view_fp8(1, cap)
    pool.materialize_fp8(sel, n_sel, k8, v8t, k_scale, v_scale)
    q, qb = queries(spec)
    out, lse = pool.new_outputs(1, M)
    pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out, lse, k_scale, v_scale)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    k_inv, v_inv = np.float32(1.0) / np.float32(k_scale), np.float32(1.0) / np.float32(v_scale)
    rK, rV = orc.gather_fp8(osess.repo, osess.table, ids, cap, float(k_inv), float(v_inv))
    T = k * B
    assert np.array_equal(k8.cpu().numpy()[0][:, :, :T], rK[:, :, :T]), "FP8 key codes differ"
    assert np.array_equal(v8t.cpu().numpy()[0][:, :, :k], rV[:, :, :k]), "FP8 value codes differ"
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, T, k_scale, v_scale)
    err_o = np.abs(out.cpu().numpy()[0] - ref_out).max()
    err_l = np.abs(lse.cpu().numpy()[0] - ref_lse).max()
    assert err_o <= ATTN_ATOL * max(1.0, v_scale) and err_l <= ATTN_ATOL, (err_o, err_l)
    assert err_o <= 5e-2 * np.abs(ref_out).max()


def test_fp8_attention_stays_close_to_the_bf16_view():
    # quantisation moves the result, but only by the few per cent E4M3's three mantissa bits allow
    spec = SPEC
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    ids = _ids(np.random.default_rng(5), spec.n_blocks, 20)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([20], dtype=torch.int32, device=dev)
    q, _ = queries(spec)
    view = pool.new_view(1, 20 * 64)
    pool.materialize(sel, n_sel, view)
    out, lse = pool.new_outputs(1, spec.n_q_tokens)
    pool.view_attend(q.to(dev), view, n_sel, out, lse)
    k8, v8t = pool.new_view_fp8(1, 20 * 64)
    pool.materialize_fp8(sel, n_sel, k8, v8t)
    out8, lse8 = pool.new_outputs(1, spec.n_q_tokens)
    pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out8, lse8)
    torch.cuda.synchronize()
    assert (out8 - out).abs().max().item() < 0.05 and (lse8 - lse).abs().max().item() < 0.1


def test_fp8_empty_view_and_argument_errors():
    from paper_2609_04852_b200 import KvmemError
    spec = SPEC.with_(n_blocks=16)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    sel = torch.zeros(1, 4, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    k8, v8t = pool.new_view_fp8(1, 4 * 64)
    q, _ = queries(spec)
    out, lse = pool.new_outputs(1, spec.n_q_tokens)
    pool.materialize_fp8(sel, n_sel, k8, v8t)
    pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out, lse)
    torch.cuda.synchronize()
    assert torch.all(out == 0) and torch.all(torch.isinf(lse) & (lse < 0))
    with pytest.raises(KvmemError):
        pool.materialize_fp8(sel, n_sel, k8, v8t, k_scale=0.0)
    with pytest.raises(KvmemError):
        pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out, lse, v_scale=-1.0)
    assert pool.device_status() == 0
