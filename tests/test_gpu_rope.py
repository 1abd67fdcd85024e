"""Position-consistent keys on the GPU against the oracle: de-RoPE at append, rotation of queries,
RoPE at compact positions during view assembly.  Rotated keys are a defined code (fp32 products and
sums, one rounding to bf16), so everything here is compared bit for bit; values are copied unchanged."""
import numpy as np
import pytest
import torch

from kvmem_harness import ATTN_ATOL, bits, check_rotated_keys, queries
from kvmem_workloads import CONFIGS, kv_blocks, page_table
from oracle import kvmem_oracle as orc

pytestmark = pytest.mark.gpu

THETA = 1.0e6
WINDOW = 4096                                   # native window of this toy model: positions [0, 4096)
SPEC = CONFIGS["tiny"].with_(name="rope", n_blocks=150, n_planted=5, budget_blocks=20, n_q_tokens=4)


def _pool(spec, rope=True):
    from paper_2609_04852_b200 import Pool
    return Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens, spec.n_sessions,
                spec.n_sessions * spec.n_blocks, spec.n_blocks, 0, WINDOW if rope else 0, THETA if rope else 0.0)


def _fill_both(spec):
    """The generator's keys are taken as RoPE-encoded at positions pos0[b] + t; both sides remove the encoding."""
    dev = torch.device("cuda", 0)
    pool = _pool(spec)
    tab = orc.rope_table(WINDOW, spec.head_dim, THETA)
    B = spec.block_tokens
    pos0 = [(37 * b * B) % (WINDOW - B) for b in range(spec.n_blocks)]
    table = page_table(spec)[0]
    repo = orc.Repository.empty(spec.n_blocks, B, spec.n_layers, spec.n_kv_heads, spec.head_dim)
    idx = np.zeros((spec.n_layers, spec.n_kv_heads, spec.n_blocks, spec.head_dim), np.uint16)
    for b0 in range(0, spec.n_blocks, 64):
        b1 = min(spec.n_blocks, b0 + 64)
        K, V = kv_blocks(spec, 0, b0, b1, dev)
        pool.append_blocks_rope(0, K, V, pos0[b0:b1], table[b0:b1].tolist())
        Kb, Vb = bits(K), bits(V)
        tok_pos = np.concatenate([np.arange(pos0[b], pos0[b] + B) for b in range(b0, b1)]).astype(np.int32)
        raw = orc.rope_rotate(Kb.reshape(len(tok_pos), -1, spec.head_dim), tok_pos, tab, inverse=True).reshape(Kb.shape)
        repo.place(raw, Vb, np.ascontiguousarray(table[b0:b1].numpy()))
        orc.mean_k_index(raw, B, idx, b0)
    torch.cuda.synchronize()
    return pool, repo, idx, tab, table.numpy()


def test_rotate_forward_and_inverse_bit_exact():
    dev = torch.device("cuda", 0)
    pool = _pool(SPEC.with_(n_blocks=4))
    tab = orc.rope_table(WINDOW, 128, THETA)
    g = torch.Generator().manual_seed(3)
    x = torch.randn(333, 5, 128, generator=g).to(torch.bfloat16)
    pos = torch.randint(0, WINDOW, (333,), generator=g, dtype=torch.int32)
    for inverse in (False, True):
        y = pool.rope_rotate(x.to(dev), pos.to(dev), inverse=inverse)
        ref = orc.rope_rotate(bits(x), pos.numpy(), tab, inverse=inverse)
        assert np.array_equal(bits(y), ref)
    assert pool.device_status() == 0


def test_append_removes_the_encoding_and_indexes_raw_keys():
    pool, repo, idx, tab, table = _fill_both(SPEC)
    assert np.array_equal(bits(pool.index(0)), idx), "index of de-rotated keys differs"
    # the pages hold the raw keys: gather everything without rotation and compare
    dev = torch.device("cuda", 0)
    sel = torch.arange(SPEC.n_blocks, dtype=torch.int32, device=dev).view(1, -1)
    n_sel = torch.tensor([SPEC.n_blocks], dtype=torch.int32, device=dev)
    view = pool.new_view(1, SPEC.n_blocks * SPEC.block_tokens)
    pool.materialize(sel, n_sel, view)
    vK, vV = orc.gather(repo, table, np.arange(SPEC.n_blocks, dtype=np.int32), SPEC.n_blocks * SPEC.block_tokens)
    assert np.array_equal(bits(view.k[0]), vK) and np.array_equal(bits(view.v[0]), vV)
    assert pool.device_status() == 0


@pytest.mark.parametrize("first_position", [0, 517])
def test_step_with_position_consistent_view(first_position):
    """de-RoPE the query, select, materialise with RoPE at compact positions, attend with the encoded query."""
    from paper_2609_04852_b200 import SelectParams
    spec = SPEC
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    k, B, M, H, d = spec.budget_blocks, spec.block_tokens, spec.n_q_tokens, spec.n_q_heads, spec.head_dim
    q, qb = queries(spec)                                     # encoded queries at positions just after the view
    q_pos = torch.arange(first_position + k * B, first_position + k * B + M, dtype=torch.int32)
    qd = q.to(dev)
    q_raw = pool.rope_rotate(qd.view(M, H, d), q_pos.to(dev), inverse=True).view(1, M, 1, H, d)
    q_raw_ref = orc.rope_rotate(qb[0].reshape(M, H, d), q_pos.numpy(), tab, inverse=True).reshape(M, 1, H, d)
    assert np.array_equal(bits(q_raw)[0], q_raw_ref)
    sel = torch.zeros(1, k, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    scores = torch.zeros(1, spec.n_blocks, dtype=torch.float32, device=dev)
    pool.select(q_raw, SelectParams(k, 1 << 30, 0, 0, 0), sel, n_sel, scores)
    view = pool.new_view(1, k * B)
    pool.materialize_rope(sel, n_sel, view, first_position)
    out, lse = pool.new_outputs(1, M)
    pool.view_attend(qd, view, n_sel, out, lse)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    R, _ = orc.block_scores(q_raw_ref, idx, spec.n_blocks)
    assert np.all(np.abs(scores.cpu().numpy()[0] - R) <= 1e-3 * np.abs(R) + 1e-9)
    ids = sel.cpu().numpy()[0, : int(n_sel.item())]
    assert len(ids) == k
    vK, vV = orc.gather_rope(repo, table, np.ascontiguousarray(ids), k * B, first_position, tab)
    assert np.array_equal(bits(view.v[0]), vV), "values must be copied unchanged"
    assert np.array_equal(bits(view.k[0]), vK), "rotated keys differ from the defined code"
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, k * B)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    # one call for both steps (one pass on a raw-key pool, angles composed from two table rows): values bit for bit, keys
    # within one bf16 rounding step of the defined code
    view3 = pool.new_view(1, k * B)
    out3, lse3 = pool.new_outputs(1, M)
    pool.materialize_attend_rope(qd, sel, n_sel, view3, out3, lse3, first_position)
    torch.cuda.synchronize()
    check_rotated_keys(bits(view3.k[0]), vK)
    assert torch.equal(view3.v, view.v)
    assert np.abs(out3.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse3.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    # the copy-free variant rotates the same raw tiles the same way: same keys, same tile order, same results bit for bit
    out2, lse2 = pool.new_outputs(1, M)
    pool.paged_attend_rope(qd, sel, n_sel, out2, lse2, first_position)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    assert np.abs(out2.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse2.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL
    assert torch.equal(out2, out3) and torch.equal(lse2, lse3)


@pytest.mark.parametrize("n_blocks,budget,M", [(700, 60, 4), (90, 1, 1), (64, 64, 2)])
def test_position_consistent_paged_attention_over_long_and_short_views(n_blocks, budget, M):
    # several tiles per split and a ragged split range; a single tile; every block selected
    spec = SPEC.with_(n_blocks=n_blocks, budget_blocks=budget, n_q_tokens=M)
    dev = torch.device("cuda", 0)
    pool, repo, idx, tab, table = _fill_both(spec)
    B = spec.block_tokens
    rng = np.random.default_rng(n_blocks)
    ids = np.sort(rng.choice(n_blocks, size=budget, replace=False)).astype(np.int32)
    first = 17 if (17 + budget * B) <= WINDOW else 0
    q, qb = queries(spec)
    sel = torch.from_numpy(ids).view(1, -1).to(dev)
    n_sel = torch.tensor([budget], dtype=torch.int32, device=dev)
    out, lse = pool.new_outputs(1, M)
    pool.paged_attend_rope(q.to(dev), sel, n_sel, out, lse, first)
    torch.cuda.synchronize()
    assert pool.device_status() == 0
    vK, vV = orc.gather_rope(repo, table, ids, budget * B, first, tab)
    ref_out, ref_lse = orc.attend(qb[0], vK, vV, budget * B)
    assert np.abs(out.cpu().numpy()[0] - ref_out).max() <= ATTN_ATOL and np.abs(lse.cpu().numpy()[0] - ref_lse).max() <= ATTN_ATOL


def test_rotary_errors():
    from paper_2609_04852_b200 import KvmemError
    from paper_2609_04852_b200.kvmem import E_INVALID, E_STATE
    spec = SPEC.with_(n_blocks=8)
    dev = torch.device("cuda", 0)
    K, V = kv_blocks(spec, 0, 0, 2, dev)
    plain = _pool(spec, rope=False)
    with pytest.raises(KvmemError) as e:
        plain.append_blocks_rope(0, K, V, [0, 64])
    assert e.value.status == E_STATE and plain.session_blocks(0) == 0
    pool = _pool(spec)
    with pytest.raises(KvmemError) as e:
        pool.append_blocks_rope(0, K, V, [0, WINDOW - 10])          # second block would run past the table
    assert e.value.status == E_INVALID and pool.session_blocks(0) == 0
    pool.append_blocks_rope(0, K, V, [0, 64])
    sel = torch.tensor([[0, 1]], dtype=torch.int32, device=dev)
    n_sel = torch.tensor([2], dtype=torch.int32, device=dev)
    view = pool.new_view(1, 2 * spec.block_tokens)
    with pytest.raises(KvmemError) as e:
        pool.materialize_rope(sel, n_sel, view, WINDOW - 64)         # compact positions would leave the table
    assert e.value.status == E_INVALID
    out, lse = pool.new_outputs(1, 1)
    q = torch.zeros(1, 1, 1, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device=dev)
    with pytest.raises(KvmemError) as e:
        pool.paged_attend_rope(q, sel, n_sel, out, lse, WINDOW - 64)
    assert e.value.status == E_INVALID
    with pytest.raises(KvmemError) as e:
        plain.paged_attend_rope(q, sel, n_sel, out, lse, 0)
    assert e.value.status == E_STATE
    with pytest.raises(KvmemError) as e:
        pool.materialize_attend_rope(q, sel, n_sel, view, out, lse, WINDOW - 64)
    assert e.value.status == E_INVALID
    with pytest.raises(KvmemError) as e:
        plain.materialize_attend_rope(q, sel, n_sel, plain.new_view(1, 2 * spec.block_tokens), out, lse, 0)
    assert e.value.status == E_STATE
    assert pool.device_status() == 0
