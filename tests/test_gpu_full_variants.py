"""The step's variants at the 1M configuration, in the launch configuration `bench.py` times (18 splits of 228 tiles,
bounded producer lookahead): copy-free attention and the host-buffer step against the materialised path, the
position-consistent passes on the in-block key layout and the FP8 repository against the oracle at full size."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, bits, check_rotated_keys, fill_oracle, fill_pool, queries
from kvmem_workloads import CONFIGS, kv_blocks, page_table, select_params
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu

SPEC = CONFIGS["1m"]


def _select(pool, spec, qd):
    from paper_2609_04852_b200 import SelectParams, budget_blocks
    dev = qd.device
    prm = SelectParams(**select_params(spec))
    k = budget_blocks(prm, spec.block_tokens, spec.n_blocks)
    sel = torch.zeros(1, k, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    pool.select(qd, prm, sel, n_sel)
    torch.cuda.synchronize()
    assert int(n_sel.item()) == k
    return prm, k, sel, n_sel


def _oracle_selection(spec, osess, qb, dev):
    prm = select_params(spec)
    R, _ = orc.block_scores(qb[0], osess.idx, spec.n_blocks)
    ids = orc.select(R, spec.block_tokens, prm["budget_blocks"], prm["max_view_tokens"])
    sel = torch.from_numpy(ids.astype(np.int32)).view(1, -1).to(dev)
    n_sel = torch.tensor([len(ids)], dtype=torch.int32, device=dev)
    return sel, n_sel, np.ascontiguousarray(ids.astype(np.int32)), len(ids)


def test_1m_copy_free_and_host_buffer_steps_equal_the_materialised_path():
    spec = SPEC
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    q, _ = queries(spec)
    qd = q.to(dev)
    prm, k, sel, n_sel = _select(pool, spec, qd)
    M, B = spec.n_q_tokens, spec.block_tokens
    view = pool.new_view(1, k * B)
    out, lse = pool.new_outputs(1, M)
    pool.materialize(sel, n_sel, view)
    pool.view_attend(qd, view, n_sel, out, lse)             # compared with the oracle at this size in test_gpu_full_configs
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend(qd, sel, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert torch.equal(out2, out) and torch.equal(lse2, lse)
    view3 = pool.new_view(1, k * B)
    sel3, n_sel3 = torch.zeros_like(sel), torch.zeros_like(n_sel)
    out_h = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    pool.recall_step_host(q.pin_memory(), prm, sel3, n_sel3, view3, out_h, lse_h)
    assert torch.equal(sel3, sel) and torch.equal(view3.k, view.k) and torch.equal(view3.v, view.v)
    assert torch.equal(out_h, out.cpu()) and torch.equal(lse_h, lse.cpu())
    # the same step with its arguments marshalled once
    sel4, n_sel4 = torch.zeros_like(sel), torch.zeros_like(n_sel)
    out_h2, lse_h2 = torch.zeros_like(out_h).pin_memory(), torch.zeros_like(lse_h).pin_memory()
    step = pool.host_step(q.shape, prm, sel4, n_sel4, view3, out_h2, lse_h2)
    step(q.pin_memory())
    assert torch.equal(sel4, sel) and torch.equal(out_h2, out_h) and torch.equal(lse_h2, lse_h)
    with pytest.raises(ValueError):
        step(q[:, :1].contiguous())
    assert pool.device_status() == 0


def test_1m_position_consistent_passes_on_the_in_block_layout():
    from paper_2609_04852_b200 import Pool
    spec = SPEC
    dev = torch.device("cuda", 0)
    theta, B = 1.0e6, spec.block_tokens
    window = spec.max_view_tokens + 64
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, B, 1, spec.n_blocks, spec.n_blocks, 0,
                window, theta, rope_in_block_keys=True)
    tab = orc.rope_table(window, spec.head_dim, theta)
    table = page_table(spec)[0]
    for b0 in range(0, spec.n_blocks, 1024):                 # raw keys in: the append rotates each by its offset in the block
        b1 = min(spec.n_blocks, b0 + 1024)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, table[b0:b1].tolist())
    q, qb = queries(spec)
    qd = q.to(dev)
    osess = fill_oracle(spec, gen_device=dev)[0]
    sel, n_sel, ids, k = _oracle_selection(spec, osess, qb, dev)             # the oracle's own selection drives both sides
    M, T = spec.n_q_tokens, k * B
    view = pool.new_view(1, T)
    out, lse = pool.new_outputs(1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view, out, lse, 0)          # one pass, K rotated in shared memory
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out2, lse2, 0)                    # copy-free, query rotated back per block
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    # oracle: the selected blocks only (their stored keys are RoPE(raw, offset in block)), at their compact positions
    assert np.array_equal(bits(pool.index(0)), osess.idx), "the index comes from the raw keys"
    rawK, rawV = orc.gather(osess.repo, osess.table, np.ascontiguousarray(ids), T)        # [L][G][T][d] raw keys of the selection
    L, G, _, d = rawK.shape
    t_in_block = np.tile((np.arange(T) % B).astype(np.int32), L * G)
    storedK = orc.rope_rotate(np.ascontiguousarray(rawK.reshape(L * G * T, 1, d)), t_in_block, tab).reshape(rawK.shape)
    p0 = np.tile(((np.arange(T) // B) * B).astype(np.int32), L * G)
    viewK = orc.rope_rotate(np.ascontiguousarray(storedK.reshape(L * G * T, 1, d)), p0, tab).reshape(rawK.shape)
    assert np.array_equal(bits(view.k[0]), viewK), "fused pass: rotated keys differ from the defined code"
    assert np.array_equal(bits(view.v[0]), rawV)
    ref_out, ref_lse = orc.attend(qb[0], viewK, rawV, T)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    q_out, q_lse = orc.attend_qrot(qb[0], storedK, rawV, T, B, 0, tab)
    assert np.abs(out2.cpu().numpy()[0] - q_out).max() <= ATTN_ATOL and np.abs(lse2.cpu().numpy()[0] - q_lse).max() <= ATTN_ATOL


def test_1m_fp8_repository_passes():
    from paper_2609_04852_b200 import Pool
    spec = SPEC
    dev = torch.device("cuda", 0)
    B = spec.block_tokens
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, B, 1, spec.n_blocks, spec.n_blocks, 0,
                fp8_pages=True, fp8_k_scale=0.5, fp8_v_scale=0.25)
    table = page_table(spec)[0]
    for b0 in range(0, spec.n_blocks, 1024):
        b1 = min(spec.n_blocks, b0 + 1024)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, table[b0:b1].tolist())
    q, qb = queries(spec)
    qd = q.to(dev)
    osess = fill_oracle(spec, gen_device=dev)[0]
    sel, n_sel, ids, k = _oracle_selection(spec, osess, qb, dev)
    M, T = spec.n_q_tokens, k * B
    k8, v8t = pool.new_view_fp8(1, T)
    out, lse = pool.new_outputs(1, M)
    pool.materialize_attend_fp8(qd, sel, n_sel, k8, v8t, out, lse)
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_fp8(qd, sel, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert torch.equal(out2, out) and torch.equal(lse2, lse)
    assert np.array_equal(bits(pool.index(0)), osess.idx)
    rK, rV = orc.gather_fp8(osess.repo, osess.table, np.ascontiguousarray(ids), T, 2.0, 4.0)
    assert np.array_equal(k8.cpu().numpy()[0], rK) and np.array_equal(v8t.cpu().numpy()[0], rV)
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, T, 0.5, 0.25)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL


def test_1m_fp8_view_written_while_attended_over_bf16_pages():
    """kvmem_materialize_attend_fp8 on the bf16 repository at full size, in the launch configuration bench.py --fp8 times:
    codes byte for byte against the oracle's quantising gather, results within tolerance of the oracle's FP8 attention and
    equal to the two separate calls bit for bit."""
    spec = SPEC
    dev = torch.device("cuda", 0)
    B = spec.block_tokens
    pool = fill_pool(spec)
    q, qb = queries(spec)
    qd = q.to(dev)
    osess = fill_oracle(spec, gen_device=dev)[0]
    sel, n_sel, ids, k = _oracle_selection(spec, osess, qb, dev)
    M, T = spec.n_q_tokens, k * B
    k8, v8t = pool.new_view_fp8(1, T)
    out, lse = pool.new_outputs(1, M)
    pool.materialize_attend_fp8(qd, sel, n_sel, k8, v8t, out, lse)
    k8s, v8s = pool.new_view_fp8(1, T)
    out2, lse2 = pool.new_outputs(1, M)
    pool.materialize_fp8(sel, n_sel, k8s, v8s)
    pool.view_attend_fp8(qd, k8s, v8s, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert torch.equal(k8, k8s) and torch.equal(v8t, v8s) and torch.equal(out, out2) and torch.equal(lse, lse2)
    rK, rV = orc.gather_fp8(osess.repo, osess.table, np.ascontiguousarray(ids), T, 1.0, 1.0)
    assert np.array_equal(k8.cpu().numpy()[0], rK) and np.array_equal(v8t.cpu().numpy()[0], rV)
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, T, 1.0, 1.0)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL


def test_1m_position_consistent_passes_on_raw_keys():
    """Raw keys in the pages (the paper's layout, Sec. 4.3/4.4): the rotating gather against the oracle at full size,
    attention over it, and the copy-free pass that rotates key fragments in registers, which must give the same bits."""
    from paper_2609_04852_b200 import Pool
    spec = SPEC
    dev = torch.device("cuda", 0)
    theta, B = 1.0e6, spec.block_tokens
    window = spec.max_view_tokens + 64
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, B, 1, spec.n_blocks, spec.n_blocks, 0,
                window, theta)
    tab = orc.rope_table(window, spec.head_dim, theta)
    table = page_table(spec)[0]
    for b0 in range(0, spec.n_blocks, 1024):
        b1 = min(spec.n_blocks, b0 + 1024)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, table[b0:b1].tolist())
    q, qb = queries(spec)
    qd = q.to(dev)
    osess = fill_oracle(spec, gen_device=dev)[0]
    sel, n_sel, ids, k = _oracle_selection(spec, osess, qb, dev)
    M, T, first = spec.n_q_tokens, k * B, 37
    view = pool.new_view(1, T)
    out, lse = pool.new_outputs(1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view, out, lse, first)      # one pass on a raw-key pool
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out2, lse2, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    vK, vV = orc.gather_rope(osess.repo, osess.table, ids, T, first, tab)
    check_rotated_keys(bits(view.k[0]), vK)
    assert np.array_equal(bits(view.v[0]), vV)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, T)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    assert torch.equal(out2, out) and torch.equal(lse2, lse)
