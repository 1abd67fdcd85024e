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


# ---- one pass over a bf16 repository: tiles quantised on the way to the view and to the tensor cores ----

@pytest.mark.parametrize("n_blocks,k,cap_blocks,M,k_scale,v_scale,L", [(150, 20, 20, 4, 1.0, 1.0, 1), (700, 333, 340, 4, 0.5, 0.25, 1),
                                                                      (90, 1, 1, 1, 2.0, 1.0, 1), (64, 64, 64, 2, 1.0, 0.0625, 1),
                                                                      (300, 7, 7, 3, 1.0, 1.0, 1), (120, 37, 40, 2, 1.0, 0.5, 2)])
def test_fp8_view_written_while_attended_over_bf16_pages(n_blocks, k, cap_blocks, M, k_scale, v_scale, L):
    """kvmem_materialize_attend_fp8 on a bf16 repository: the view must hold the oracle's codes byte for byte, the results
    must be the oracle's attention over those codes within tolerance, and both must equal the two separate calls bit
    for bit; nothing outside the view and the outputs is written."""
    from kvmem_harness import Guards
    from kvmem_workloads import kv_blocks, page_table
    from paper_2609_04852_b200 import Pool
    spec = SPEC.with_(n_blocks=n_blocks, n_planted=min(8, n_blocks // 4), budget_blocks=k, n_q_tokens=M, n_layers=L)
    dev = torch.device("cuda", 0)
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens, 1, n_blocks, n_blocks, 0,
                fp8_k_scale=k_scale, fp8_v_scale=v_scale)
    table = page_table(spec)[0]
    for b0 in range(0, n_blocks, 256):
        b1 = min(n_blocks, b0 + 256)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, table[b0:b1].tolist())
    osess = fill_oracle(spec)[0]
    ids = _ids(np.random.default_rng(n_blocks + k), n_blocks, k)
    cap = cap_blocks * 64
    sel = torch.full((1, cap_blocks), -1, dtype=torch.int32)
    sel[0, :k] = torch.from_numpy(ids)
    sel = sel.to(dev)
    n_sel = torch.tensor([k], dtype=torch.int32, device=dev)
    q, qb = queries(spec)
    qd = q.to(dev)
    g = Guards(dev)
    k8 = g.empty((1, spec.n_layers, spec.n_kv_heads, cap, 128), torch.uint8)
    v8t = g.empty((1, spec.n_layers, spec.n_kv_heads, cap_blocks, 128, 64), torch.uint8)
    out, lse = g.outputs(pool, 1, M)
    pool.materialize_attend_fp8(qd, sel, n_sel, k8, v8t, out, lse)
    k8s, v8s = pool.new_view_fp8(1, cap)
    out2, lse2 = pool.new_outputs(1, M)
    pool.materialize_fp8(sel, n_sel, k8s, v8s, k_scale, v_scale)
    pool.view_attend_fp8(qd, k8s, v8s, n_sel, out2, lse2, k_scale, v_scale)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    g.check()
    k_inv, v_inv = np.float32(1.0) / np.float32(k_scale), np.float32(1.0) / np.float32(v_scale)
    rK, rV = orc.gather_fp8(osess.repo, osess.table, ids, cap, float(k_inv), float(v_inv))
    T = k * 64
    assert np.array_equal(k8.cpu().numpy()[0][:, :, :T], rK[:, :, :T]), "FP8 key codes differ"
    assert np.array_equal(v8t.cpu().numpy()[0][:, :, :k], rV[:, :, :k]), "FP8 value codes differ"
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, T, k_scale, v_scale)
    err_o = np.abs(out.cpu().numpy()[0] - ref_out).max()
    err_l = np.abs(lse.cpu().numpy()[0] - ref_lse).max()
    assert err_o <= ATTN_ATOL * max(1.0, v_scale) and err_l <= ATTN_ATOL, (err_o, err_l)
    assert torch.equal(k8[0, :, :, :T], k8s[0, :, :, :T]) and torch.equal(v8t[0, :, :, :k], v8s[0, :, :, :k])
    assert torch.equal(out, out2) and torch.equal(lse, lse2), "one pass and separate calls must be the same bits"


def test_fp8_one_pass_over_bf16_pages_with_two_sessions_of_different_lengths():
    """Sessions are independent: each gets its own selection length (one of them shorter than the row, one empty in a
    second call) and its own slice of the view; what lies beyond a session's selection is not written."""
    spec = SPEC.with_(name="fp8two", n_sessions=2, n_blocks=96, n_planted=4, n_q_tokens=2)
    dev = torch.device("cuda", 0)
    pool = fill_pool(spec)
    osess = fill_oracle(spec)
    M, cap_blocks = 2, 24
    cap = cap_blocks * 64
    rng = np.random.default_rng(5)
    for ks in ((24, 7), (0, 13)):
        ids = [_ids(rng, spec.n_blocks, k) for k in ks]
        sel = torch.full((2, cap_blocks), -1, dtype=torch.int32)
        for s_, idv in enumerate(ids):
            sel[s_, :len(idv)] = torch.from_numpy(idv)
        sel = sel.to(dev)
        n_sel = torch.tensor(list(ks), dtype=torch.int32, device=dev)
        q, qb = queries(spec)
        k8, v8t = pool.new_view_fp8(2, cap)
        k8.fill_(0x5A); v8t.fill_(0x5A)
        out, lse = pool.new_outputs(2, M)
        pool.materialize_attend_fp8(q.to(dev), sel, n_sel, k8, v8t, out, lse)
        torch.cuda.synchronize()
        assert pool.device_status() == 0
        for s_, k in enumerate(ks):
            rK, rV = orc.gather_fp8(osess[s_].repo, osess[s_].table, ids[s_], cap, 1.0, 1.0)
            T = k * 64
            assert np.array_equal(k8.cpu().numpy()[s_][:, :, :T], rK[:, :, :T]) and np.array_equal(v8t.cpu().numpy()[s_][:, :, :k], rV[:, :, :k])
            assert bool((k8[s_][:, :, T:] == 0x5A).all()) and bool((v8t[s_][:, :, k:] == 0x5A).all()), "wrote past the selection"
            if k == 0:
                assert bool((out[s_] == 0).all()) and bool(torch.isinf(lse[s_]).all())
                continue
            ref_out, ref_lse = orc.attend_fp8(qb[s_], rK, rV, T, 1.0, 1.0)
            assert np.abs(out.cpu().numpy()[s_] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[s_] - ref_lse).max() <= ATTN_ATOL


# ---- FP8 repository: the pages themselves hold the E4M3 tiles ---------------------------------------

def _fp8_pool(spec, k_scale, v_scale):
    from kvmem_workloads import kv_blocks, page_table
    from paper_2609_04852_b200 import Pool
    dev = torch.device("cuda", 0)
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens, spec.n_sessions,
                spec.n_sessions * spec.n_blocks, spec.n_blocks, 0, fp8_pages=True, fp8_k_scale=k_scale, fp8_v_scale=v_scale)
    tables = page_table(spec)
    for b0 in range(0, spec.n_blocks, 64):
        b1 = min(spec.n_blocks, b0 + 64)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks(0, K, V, tables[0, b0:b1].tolist())
    torch.cuda.synchronize()
    return pool


@pytest.mark.parametrize("n_blocks,k,M,k_scale,v_scale", [(150, 20, 4, 1.0, 1.0), (700, 333, 4, 0.5, 0.25), (90, 1, 1, 2.0, 1.0),
                                                         (64, 64, 2, 1.0, 0.0625)])
def test_fp8_repository_pages_view_and_copy_free_attention(n_blocks, k, M, k_scale, v_scale):
    """Quantised once at append: the gathered view must hold the codes the oracle gets by quantising its bf16 gather,
    the index must be the bf16 Mean-K of the keys that were appended, and attention straight over the pages must equal
    attention over the gathered view bit for bit and the oracle's attention over the codes within tolerance."""
    from kvmem_harness import bits
    from paper_2609_04852_b200 import SelectParams
    spec = SPEC.with_(n_blocks=n_blocks, n_planted=min(8, n_blocks // 4), budget_blocks=k, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool = _fp8_pool(spec, k_scale, v_scale)
    osess = fill_oracle(spec)[0]
    assert np.array_equal(bits(pool.index(0)), osess.idx), "the index comes from the bf16 keys"
    ids = _ids(np.random.default_rng(n_blocks), n_blocks, k)
    cap = k * 64
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([k], dtype=torch.int32, device=dev)
    k8, v8t = pool.new_view_fp8(1, cap)
    pool.materialize_fp8(sel, n_sel, k8, v8t, k_scale, v_scale)
    q, qb = queries(spec)
    out, lse = pool.new_outputs(1, M)
    pool.view_attend_fp8(q.to(dev), k8, v8t, n_sel, out, lse, k_scale, v_scale)
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_fp8(q.to(dev), sel, n_sel, out2, lse2)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    k_inv, v_inv = np.float32(1.0) / np.float32(k_scale), np.float32(1.0) / np.float32(v_scale)
    rK, rV = orc.gather_fp8(osess.repo, osess.table, ids, cap, float(k_inv), float(v_inv))
    assert np.array_equal(k8.cpu().numpy()[0], rK), "FP8 key codes differ"
    assert np.array_equal(v8t.cpu().numpy()[0], rV), "FP8 value codes differ"
    ref_out, ref_lse = orc.attend_fp8(qb[0], rK, rV, cap, k_scale, v_scale)
    for o, l in ((out, lse), (out2, lse2)):
        err_o = np.abs(o.cpu().numpy()[0] - ref_out).max()
        err_l = np.abs(l.cpu().numpy()[0] - ref_lse).max()
        assert err_o <= ATTN_ATOL * max(1.0, v_scale) and err_l <= ATTN_ATOL, (err_o, err_l)
    assert torch.equal(out2, out) and torch.equal(lse2, lse), "copy-free and gathered attention must be the same bits"
    # one pass: tiles stored to the view while attended over
    k8f, v8f = pool.new_view_fp8(1, cap)
    out3, lse3 = pool.new_outputs(1, M)
    pool.materialize_attend_fp8(q.to(dev), sel, n_sel, k8f, v8f, out3, lse3)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert torch.equal(k8f, k8) and torch.equal(v8f, v8t) and torch.equal(out3, out) and torch.equal(lse3, lse)
    # selection works off the bf16 index as on any pool: the planted blocks win
    R, _ = orc.block_scores(qb[0], osess.idx, n_blocks)
    n_pl = spec.n_planted
    ref_sel = orc.select(R, 64, n_pl, 1 << 30)
    sel2 = torch.zeros(1, n_pl, dtype=torch.int32, device=dev)
    n_sel2 = torch.zeros(1, dtype=torch.int32, device=dev)
    pool.select(q.to(dev), SelectParams(n_pl, 1 << 30, 0, 0, 0), sel2, n_sel2)
    assert np.array_equal(sel2.cpu().numpy()[0, : int(n_sel2.item())], ref_sel)


def test_page_formats_are_not_mixed_up():
    from paper_2609_04852_b200 import KvmemError, Pool
    from paper_2609_04852_b200.kvmem import E_INVALID, E_STATE
    spec = SPEC.with_(n_blocks=16, n_planted=2)
    dev = torch.device("cuda", 0)
    f8 = _fp8_pool(spec, 1.0, 0.5)
    bf = fill_pool(spec)
    sel = torch.arange(4, dtype=torch.int32, device=dev).view(1, -1)
    n_sel = torch.tensor([4], dtype=torch.int32, device=dev)
    q, _ = queries(spec)
    qd = q.to(dev)
    out, lse = f8.new_outputs(1, spec.n_q_tokens)
    view = f8.new_view(1, 4 * 64)
    for call in (lambda: f8.materialize(sel, n_sel, view), lambda: f8.materialize_attend(qd, sel, n_sel, view, out, lse),
                 lambda: f8.paged_attend(qd, sel, n_sel, out, lse), lambda: bf.paged_attend_fp8(qd, sel, n_sel, out, lse)):
        with pytest.raises(KvmemError) as e:
            call()
        assert e.value.status == E_STATE
    k8, v8t = f8.new_view_fp8(1, 4 * 64)
    with pytest.raises(KvmemError) as e:
        f8.materialize_fp8(sel, n_sel, k8, v8t, 1.0, 1.0)            # not the scales the pages were written with
    assert e.value.status == E_INVALID
    with pytest.raises(KvmemError):
        Pool(1, 32, 8, 128, 32, 1, 8, 8, 0, fp8_pages=True)          # 32-token blocks
    with pytest.raises(KvmemError):
        Pool(1, 32, 8, 128, 64, 1, 8, 8, 0, 4096, 1.0e6, fp8_pages=True)      # rotary support
    with pytest.raises(KvmemError):
        Pool(1, 32, 8, 128, 64, 1, 8, 8, 0, fp8_pages=True, fp8_k_scale=0.0)
    assert f8.device_status() == 0 and bf.device_status() == 0
    # half the memory: pages of 1 byte per element
    assert f8.storage.numel() < 0.6 * bf.storage.numel()


# ---- FP8 repository of in-block-rotated keys: position-consistent, copy-free, one byte per element ----

@pytest.mark.parametrize("encoded,n_blocks,k,M,first", [(False, 150, 20, 4, 517), (True, 700, 60, 4, 17), (False, 90, 1, 1, 0),
                                                       (True, 64, 64, 2, 0)])
def test_fp8_repository_of_in_block_rotated_keys(encoded, n_blocks, k, M, first):
    """The paper's three mechanisms together (FP8 KV cache, keys encoded at their compact positions, copy-free view):
    pages hold the codes of bf16(RoPE(k, offset in block)); attention rotates the query back once per block."""
    from kvmem_harness import bits
    from kvmem_workloads import kv_blocks, page_table
    from paper_2609_04852_b200 import Pool
    spec = SPEC.with_(n_blocks=n_blocks, n_planted=min(8, n_blocks // 4), budget_blocks=k, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    theta, window, B, d = 1.0e6, 4096, 64, spec.head_dim
    k_scale, v_scale = 0.5, 0.25
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, d, B, 1, n_blocks, n_blocks, 0, window, theta,
                rope_in_block_keys=True, fp8_pages=True, fp8_k_scale=k_scale, fp8_v_scale=v_scale)
    tab = orc.rope_table(window, d, theta)
    table = page_table(spec)[0]
    pos0 = [(37 * b * B) % (window - B) for b in range(n_blocks)]
    repo = orc.Repository.empty(n_blocks, B, spec.n_layers, spec.n_kv_heads, d)
    idx = np.zeros((spec.n_layers, spec.n_kv_heads, n_blocks, d), np.uint16)
    for b0 in range(0, n_blocks, 64):
        b1 = min(n_blocks, b0 + 64)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        Kb, Vb = bits(K), bits(V)
        n_tok = (b1 - b0) * B
        if encoded:      # the generator's keys taken as RoPE-encoded at pos0[b] + t: the append removes that first
            pool.append_blocks_rope(0, K, V, pos0[b0:b1], table[b0:b1].tolist())
            tok_pos = np.concatenate([np.arange(pos0[b], pos0[b] + B) for b in range(b0, b1)]).astype(np.int32)
            raw = orc.rope_rotate(Kb.reshape(n_tok, -1, d), tok_pos, tab, inverse=True).reshape(Kb.shape)
        else:
            pool.append_blocks(0, K, V, table[b0:b1].tolist())
            raw = Kb
        t_in = (np.arange(n_tok) % B).astype(np.int32)
        stored = orc.rope_rotate(np.ascontiguousarray(raw.reshape(n_tok, -1, d)), t_in, tab).reshape(Kb.shape)
        repo.place(stored, Vb, np.ascontiguousarray(table[b0:b1].numpy()))
        orc.mean_k_index(raw, B, idx, b0)
    torch.cuda.synchronize()
    assert np.array_equal(bits(pool.index(0)), idx), "the index comes from the raw bf16 keys"
    ids = _ids(np.random.default_rng(n_blocks + 3), n_blocks, k)
    cap = k * B
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([k], dtype=torch.int32, device=dev)
    k8, v8t = pool.new_view_fp8(1, cap)
    pool.materialize_fp8(sel, n_sel, k8, v8t, k_scale, v_scale)                 # the stored codes, gathered
    q, qb = queries(spec)
    out, lse = pool.new_outputs(1, M)
    pool.paged_attend_fp8_rope(q.to(dev), sel, n_sel, out, lse, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    k_inv, v_inv = np.float32(1.0) / np.float32(k_scale), np.float32(1.0) / np.float32(v_scale)
    rK, rV = orc.gather_fp8(repo, table.numpy(), ids, cap, float(k_inv), float(v_inv))
    assert np.array_equal(k8.cpu().numpy()[0], rK), "codes of the in-block-rotated keys differ"
    assert np.array_equal(v8t.cpu().numpy()[0], rV)
    ref_out, ref_lse = orc.attend_fp8_qrot(qb[0], rK, rV, cap, B, first, tab, k_scale, v_scale)
    err_o, err_l = np.abs(out.cpu().numpy()[0] - ref_out).max(), np.abs(lse.cpu().numpy()[0] - ref_lse).max()
    assert err_o <= ATTN_ATOL and err_l <= ATTN_ATOL, (err_o, err_l)
    if k > 1 and first + 200 + cap <= window:       # the rotation really follows the compact position
        out2, lse2 = pool.new_outputs(1, M)
        pool.paged_attend_fp8_rope(q.to(dev), sel, n_sel, out2, lse2, first + 200)
        torch.cuda.synchronize()
        ref2, ref_lse2 = orc.attend_fp8_qrot(qb[0], rK, rV, cap, B, first + 200, tab, k_scale, v_scale)
        assert np.abs(out2.cpu().numpy()[0] - ref2).max() <= ATTN_ATOL and np.abs(lse2.cpu().numpy()[0] - ref_lse2).max() <= ATTN_ATOL
        assert (lse2 - lse).abs().max().item() > 10 * ATTN_ATOL


def test_fp8_rope_reader_needs_both_options():
    from paper_2609_04852_b200 import KvmemError
    from paper_2609_04852_b200.kvmem import E_STATE
    spec = SPEC.with_(n_blocks=16, n_planted=2)
    dev = torch.device("cuda", 0)
    f8 = _fp8_pool(spec, 1.0, 1.0)
    sel = torch.arange(4, dtype=torch.int32, device=dev).view(1, -1)
    n_sel = torch.tensor([4], dtype=torch.int32, device=dev)
    q, _ = queries(spec)
    out, lse = f8.new_outputs(1, spec.n_q_tokens)
    with pytest.raises(KvmemError) as e:
        f8.paged_attend_fp8_rope(q.to(dev), sel, n_sel, out, lse, 0)
    assert e.value.status == E_STATE
