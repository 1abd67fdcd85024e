"""Pins for the CPU oracle: what the equations and plain mathematics fix, independent of
the oracle's own code.  Closed forms, invariants, special cases that reduce to textbook
softmax attention, brute force on tiny inputs, planted-block recovery.
"""
import math

import numpy as np
import pytest
from conftest import bits_of, from_bits, to_bits
from scipy.special import logsumexp, softmax

from kvmem_workloads import CONFIGS, kv_blocks, make_queries, page_table, planted_blocks
from oracle import kvmem_oracle as orc

rng = np.random.default_rng(20260425)


def rand_bits(*shape, scale=1.0):
    return to_bits(rng.standard_normal(shape).astype(np.float32) * scale)


# ------------------------------------------------------------------ Mean-K index (Eq. mean_k_index)

def test_index_identical_keys_give_that_key():
    B, L, G, d = 8, 2, 3, 16
    key = rand_bits(1, L, G, d)
    K = np.repeat(key, 5 * B, axis=0)
    idx = orc.mean_k_index(K, B)
    for b in range(5):
        assert np.array_equal(idx[:, :, b, :], key[0])


def test_index_plus_minus_pairs_cancel():
    B, L, G, d = 16, 1, 2, 8
    half = from_bits(rand_bits(B // 2, L, G, d))
    blk = np.empty((B, L, G, d), np.float32)
    blk[0::2], blk[1::2] = half, -half                    # +x, -x, +y, -y ...: fp32 partial sums hit 0 exactly
    idx = orc.mean_k_index(to_bits(blk), B)
    assert np.all(from_bits(idx) == 0.0)


def test_index_hand_example():
    # one block of 4 tokens, d = 2: mean of (1,2,3,6) = 3 ; mean of (0.5,-0.5,0.25,0.75) = 0.25
    K = to_bits(np.array([[1, .5], [2, -.5], [3, .25], [6, .75]], np.float32).reshape(4, 1, 1, 2))
    idx = orc.mean_k_index(K, 4)
    assert from_bits(idx).reshape(-1).tolist() == [3.0, 0.25]


def test_index_within_one_ulp_of_fp64_mean_and_layout():
    B, L, G, d, nb = 64, 2, 4, 32, 7
    K = rand_bits(nb * B, L, G, d)
    idx = orc.mean_k_index(K, B)
    exact = from_bits(K).astype(np.float64).reshape(nb, B, L, G, d).mean(axis=1)        # [nb][L][G][d]
    exact = np.transpose(exact, (1, 2, 0, 3))                                             # [L][G][nb][d]
    got = from_bits(idx).astype(np.float64)
    ulp = np.maximum(np.abs(exact), 2.0 ** -126) * 2.0 ** -8                              # bf16: 8 bits of significand
    assert np.all(np.abs(got - exact) <= ulp)


def test_index_incremental_append_equals_one_shot():
    B, L, G, d = 32, 1, 2, 16
    K = rand_bits(6 * B, L, G, d)
    one = orc.mean_k_index(K, B)
    inc = np.zeros_like(one)
    orc.mean_k_index(K[: 2 * B].copy(), B, inc, 0)
    orc.mean_k_index(K[2 * B:].copy(), B, inc, 2)
    assert np.array_equal(one, inc)


def test_index_footprint_matches_paper_growth():
    # Sec. 6.5 (values in tests/golden/index_footprint.txt): ~0.25 GiB at 256K tokens and ~9.5 GiB at 10M tokens with
    # 32-token blocks.  One vector per (block, layer, KV head) means bytes grow linearly in blocks: both figures give
    # the same per-block size, and that size is what the oracle's index layout occupies for a model whose scored
    # layers x KV heads x head_dim x 2 bytes come to 32 KiB per block.
    import os
    rows = [ln.split() for ln in open(os.path.join(os.path.dirname(__file__), "golden", "index_footprint.txt"))
            if ln.strip() and not ln.startswith("#")]
    (t0, b0, g0), (t1, b1, g1) = [(int(r[0]), int(r[1]), float(r[2])) for r in rows]
    per_block_small = g0 * 2 ** 30 / (t0 / b0)
    per_block_large = g1 * 2 ** 30 / (t1 / b1)
    assert abs(per_block_small - 32 * 1024) < 1
    assert abs(per_block_large / per_block_small - 1) < 0.03
    # the oracle's index of a geometry with 32 KiB per block (e.g. 16 scored layers x 8 KV heads x 128 dims, bf16)
    L, G, d, NB, B = 16, 8, 128, 3, b0
    idx = orc.mean_k_index(rand_bits(NB * B, L, G, d), B)
    assert idx.nbytes == NB * int(per_block_small) and idx.shape == (L, G, NB, d)


# ------------------------------------------------------------------ block scores (Eq. kvmem-block-score)

def _scores(q, idx, NB=None):
    return orc.block_scores(q, idx, idx.shape[2] if NB is None else NB)


def test_scores_sum_to_number_of_query_tokens_and_bounds():
    M, L, H, G, d, NB = 3, 2, 8, 2, 32, 50
    q, idx = rand_bits(M, L, H, d), rand_bits(L, G, NB, d)
    R, Rg = _scores(q, idx)
    assert abs(R.sum() - M) < 1e-5
    assert np.all(R >= 0) and np.all(R <= M)
    assert np.allclose(Rg.mean(axis=0), R, rtol=1e-6, atol=1e-9)
    assert np.allclose(Rg.sum(axis=1), M, atol=1e-5)


def test_scores_all_equal_index_is_uniform():
    M, L, H, G, d, NB = 2, 1, 4, 2, 16, 37
    q = rand_bits(M, L, H, d)
    idx = np.repeat(rand_bits(L, G, 1, d), NB, axis=2)
    R, _ = _scores(q, idx)
    assert np.allclose(R, M / NB, rtol=1e-6)


def test_scores_permutation_equivariance():
    M, L, H, G, d, NB = 2, 2, 4, 2, 16, 23
    q, idx = rand_bits(M, L, H, d), rand_bits(L, G, NB, d)
    perm = rng.permutation(NB)
    R, Rg = _scores(q, idx)
    Rp, Rgp = _scores(q, np.ascontiguousarray(idx[:, :, perm, :]))
    assert np.array_equal(Rp, R[perm]) and np.array_equal(Rgp, Rg[:, perm])


def test_scores_softmax_shift_invariance():
    # adding one vector c to every Mean-K of a head adds the constant q.c to all of its logits.
    # values on a coarse dyadic grid so that kbar + c is exactly representable in bf16
    M, L, H, G, d, NB = 1, 1, 4, 2, 8, 11
    q = to_bits(rng.integers(-4, 5, (M, L, H, d)) / 4.0)
    base = rng.integers(-8, 9, (L, G, NB, d)) / 8.0
    c = rng.integers(-8, 9, (L, G, 1, d)) / 8.0
    R0, _ = _scores(q, to_bits(base))
    R1, _ = _scores(q, to_bits(base + c))
    assert np.allclose(R0, R1, rtol=1e-6, atol=1e-9)


def test_scores_two_blocks_logistic_closed_form():
    d = 16
    qv = rng.integers(-4, 5, d) / 2.0
    k0, k1 = rng.integers(-4, 5, d) / 4.0, rng.integers(-4, 5, d) / 4.0
    idx = to_bits(np.stack([k0, k1]).reshape(1, 1, 2, d))
    R, _ = _scores(to_bits(qv.reshape(1, 1, 1, d)), idx)
    delta = float(qv @ (k0 - k1)) / math.sqrt(d)
    assert abs(R[0] - 1 / (1 + math.exp(-delta))) < 1e-6 and abs(R[0] + R[1] - 1) < 1e-6


def test_scores_single_token_blocks_are_textbook_attention_probabilities():
    # B = 1, L = H = G = M = 1: the Mean-K of a block is its only key, so R_b is the
    # softmax attention probability of token b.
    d, NB = 32, 40
    K = rand_bits(NB, 1, 1, d)
    q = rand_bits(1, 1, 1, d)
    idx = orc.mean_k_index(K, 1)
    R, _ = _scores(q, idx)
    p = softmax(from_bits(K).reshape(NB, d).astype(np.float64) @ from_bits(q).reshape(d).astype(np.float64)
                / math.sqrt(d))
    assert np.allclose(R, p, rtol=1e-6, atol=1e-10)


def test_scores_query_head_uses_kv_head_h_div_r():
    # H = 4, G = 2 (r = 2).  Only query head 1 is non-zero; under g(h) = h / r it reads KV head 0.
    # KV head 0 marks block 2, KV head 1 marks block 5; a modulo mapping would reward block 5.
    H, G, d, NB, s = 4, 2, 4, 8, 6.0
    q = np.zeros((1, 1, H, d), np.float32)
    q[0, 0, 1, 0] = 2.0
    idx = np.zeros((1, G, NB, d), np.float32)
    idx[0, 0, 2, 0] = s                       # logit = 2 * s / sqrt(4) = s
    idx[0, 1, 5, 0] = s
    R, Rg = _scores(to_bits(q), to_bits(idx))
    hot = math.exp(s) / (math.exp(s) + NB - 1)
    cold = 1.0 / (math.exp(s) + NB - 1)
    exp_R = np.full(NB, (3 * (1 / NB) + cold) / H)
    exp_R[2] = (3 * (1 / NB) + hot) / H
    assert np.allclose(R, exp_R, rtol=1e-6)
    assert np.allclose(Rg[1], 1 / NB, rtol=1e-6)           # KV head 1 saw only zero queries
    assert abs(Rg[0][2] - (1 / NB + hot) / 2) < 1e-6


def test_scores_sum_over_tokens_mean_over_layers_and_heads():
    # two layers, two tokens: with one-hot-ish logits the outer operations are visible in closed form
    M, L, H, G, d, NB, s = 2, 2, 1, 1, 4, 4, 8.0   # sqrt(d) = 2 is exact in bf16
    q = np.zeros((M, L, H, d), np.float32)
    q[0, 0, 0, 0] = math.sqrt(d)              # token 0, layer 0 looks along dim 0
    q[1, 1, 0, 1] = math.sqrt(d)              # token 1, layer 1 looks along dim 1
    idx = np.zeros((L, G, NB, d), np.float32)
    idx[0, 0, 1, 0] = s                       # layer 0: block 1 lights up on dim 0
    idx[1, 0, 3, 1] = s                       # layer 1: block 3 lights up on dim 1
    R, _ = _scores(to_bits(q), to_bits(idx))
    hot = math.exp(s) / (math.exp(s) + NB - 1)
    cold = 1.0 / (math.exp(s) + NB - 1)
    # each (m, l) pair contributes weight 1/(L*H) = 1/2; two of the four pairs are uniform (zero query)
    want = np.array([cold + 1 / NB, (hot + cold) / 2 + 1 / NB, cold + 1 / NB, (hot + cold) / 2 + 1 / NB])
    assert np.allclose(R, want, rtol=1e-6)
    assert abs(R.sum() - M) < 1e-6


def test_scores_union_of_two_tiles_combines_with_normaliser_weights():
    # global softmax across tiles (Sec. 5.2): for one (l, m, h) row, the score over A u B equals
    # the per-tile softmax re-weighted by Z_tile / (Z_A + Z_B)
    d, nA, nB_ = 16, 9, 14
    q = rand_bits(1, 1, 1, d)
    idx = rand_bits(1, 1, nA + nB_, d)
    R, _ = _scores(q, idx)
    RA, _ = _scores(q, np.ascontiguousarray(idx[:, :, :nA]))
    RB, _ = _scores(q, np.ascontiguousarray(idx[:, :, nA:]))
    logits = from_bits(idx).reshape(-1, d).astype(np.float64) @ from_bits(q).reshape(d).astype(np.float64) / math.sqrt(d)
    zA, zB = np.exp(logits[:nA]).sum(), np.exp(logits[nA:]).sum()
    assert np.allclose(R[:nA], RA * zA / (zA + zB), rtol=1e-5)
    assert np.allclose(R[nA:], RB * zB / (zA + zB), rtol=1e-5)


def test_scores_candidate_set_is_first_NB_rows_of_a_larger_index():
    M, L, H, G, d = 1, 1, 2, 1, 8
    q, idx = rand_bits(M, L, H, d), rand_bits(L, G, 20, d)
    R_a, _ = _scores(q, idx, NB=12)
    R_b, _ = _scores(q, np.ascontiguousarray(idx[:, :, :12]))
    assert np.array_equal(R_a, R_b)


# ------------------------------------------------------------------ budget and selector

def test_budget_clamp_follows_capacity_inequality():
    # N(Q) + B * k <= B_a
    assert orc.budget_blocks(NB=1000, B=64, budget_blocks=512, max_view_tokens=262144) == 512
    assert orc.budget_blocks(16384, 64, 4096, 262144) == 4096              # exactly window-bound
    assert orc.budget_blocks(16384, 64, 5000, 262144) == 4096
    assert orc.budget_blocks(16384, 64, 4096, 262144, mandatory_tokens=1) == 4095
    assert orc.budget_blocks(10, 64, 4096, 262144) == 10
    assert orc.budget_blocks(10, 64, 4, 100, mandatory_tokens=200) == 0
    assert orc.budget_blocks(10, 64, -3, 1000) == 0
    for NB, B, k, Ba, nq in rng.integers(1, 5000, (50, 5)):
        got = orc.budget_blocks(int(NB), int(B), int(k), int(Ba), int(nq))
        assert got <= k and got <= NB and (got == 0 or nq + B * got <= Ba)
        assert got == min(k, NB) or nq + B * (got + 1) > Ba                # and it is the largest such k


def _brute_select(R, k, n_sink, n_recent):
    NB = len(R)
    k = min(k, NB)
    chosen = list(range(min(n_sink, k)))
    for b in range(NB - 1, NB - 1 - n_recent, -1):
        if len(chosen) < k and b >= 0 and b not in chosen:
            chosen.append(b)
    rest = sorted((b for b in range(NB) if b not in chosen), key=lambda b: (-float(R[b]), b))
    chosen += rest[: k - len(chosen)]
    return sorted(chosen)


@pytest.mark.parametrize("NB,k,sink,recent", [(1, 1, 0, 0), (7, 3, 0, 0), (50, 10, 1, 2), (50, 50, 3, 3),
                                              (50, 60, 0, 0), (20, 4, 3, 3), (20, 2, 5, 5), (6, 5, 4, 4),
                                              (33, 0, 1, 1), (40, 17, 0, 40)])
def test_select_matches_exhaustive_sort(NB, k, sink, recent):
    R = rng.random(NB).astype(np.float32)
    R[rng.integers(0, NB, NB // 3)] = R[0]                 # force ties
    got = orc.select(R, 64, k, 1 << 30, 0, sink, recent)
    assert got.tolist() == _brute_select(R, k, sink, recent)
    assert np.all(np.diff(got) > 0)


def test_select_ties_go_to_the_lower_id_and_output_is_chronological():
    R = np.array([.1, .5, .5, .5, .2, .5], np.float32)
    assert orc.select(R, 64, 2, 1 << 30).tolist() == [1, 2]
    assert orc.select(R, 64, 3, 1 << 30).tolist() == [1, 2, 3]
    assert orc.select(R, 64, 5, 1 << 30).tolist() == [1, 2, 3, 4, 5]
    R = np.array([.9, .1, .8, .2, .7], np.float32)
    assert orc.select(R, 64, 3, 1 << 30).tolist() == [0, 2, 4]


def test_select_sink_and_recent_are_always_kept_and_budget_respected():
    R = np.zeros(100, np.float32)
    R[40:50] = 1.0
    got = orc.select(R, 64, 8, 1 << 30, 0, n_sink_blocks=2, n_recent_blocks=3).tolist()
    assert got == [0, 1, 40, 41, 42, 97, 98, 99]
    got = orc.select(R, 64, 8, 64 * 4, 0, 2, 3).tolist()   # capacity of 4 blocks: sinks first, then newest
    assert got == [0, 1, 98, 99]


# ------------------------------------------------------------------ gather

def test_gather_is_a_copy_through_the_block_table():
    B, L, G, d, NB = 4, 2, 3, 8, 10
    K, V = rand_bits(NB * B, L, G, d), rand_bits(NB * B, L, G, d)
    ident = np.arange(NB, dtype=np.int32)
    perm = rng.permutation(NB + 5)[:NB].astype(np.int32)
    sel = np.array([1, 4, 5, 9], np.int32)
    views = []
    for table in (ident, perm):
        repo = orc.Repository.empty(NB + 5, B, L, G, d)
        repo.place(K, V, table)
        views.append(orc.gather(repo, table, sel, cap_tokens=6 * B))
    assert np.array_equal(views[0][0], views[1][0]) and np.array_equal(views[0][1], views[1][1])
    vK, vV = views[1]
    for j, b in enumerate(sel):
        for t in range(B):
            assert np.array_equal(vK[:, :, j * B + t, :], K[b * B + t])
            assert np.array_equal(vV[:, :, j * B + t, :], V[b * B + t])
    assert not vK[:, :, len(sel) * B:, :].any()             # beyond the view: untouched


# ------------------------------------------------------------------ attention

def _view_from_tokens(K, V):
    """token-major [T][L][G][d] -> view layout [L][G][T][d]"""
    return np.ascontiguousarray(np.transpose(K, (1, 2, 0, 3))), np.ascontiguousarray(np.transpose(V, (1, 2, 0, 3)))


def test_attend_constant_values_and_zero_query():
    M, L, H, G, d, T = 2, 1, 4, 2, 16, 33
    vK, vV = rand_bits(L, G, T, d), rand_bits(L, G, T, d)
    const = to_bits(np.full((L, G, T, d), 0.75, np.float32))
    out, _ = orc.attend(rand_bits(M, L, H, d), vK, const, T)
    assert np.allclose(out, 0.75, atol=1e-6)
    out, lse = orc.attend(to_bits(np.zeros((M, L, H, d))), vK, vV, T)
    assert np.allclose(lse, math.log(T), atol=1e-6)
    meanV = from_bits(vV).astype(np.float64).mean(axis=2)                     # [L][G][d]
    for h in range(H):
        assert np.allclose(out[:, 0, h, :], meanV[0, h // (H // G)], atol=1e-6)


def test_attend_one_and_two_token_closed_forms():
    d = 8
    qv = rng.integers(-4, 5, d) / 2.0
    k = rng.integers(-4, 5, (2, d)) / 2.0
    v = rng.integers(-4, 5, (2, d)) / 2.0
    q = to_bits(qv.reshape(1, 1, 1, d))
    vK, vV = to_bits(k.reshape(1, 1, 2, d)), to_bits(v.reshape(1, 1, 2, d))
    out, lse = orc.attend(q, vK, vV, 1)
    assert np.allclose(out.reshape(d), v[0]) and abs(lse.item() - qv @ k[0] / math.sqrt(d)) < 1e-5
    out, lse = orc.attend(q, vK, vV, 2, scale=0.5)
    s = 0.5 * (k @ qv)
    w = 1 / (1 + math.exp(s[1] - s[0]))
    assert np.allclose(out.reshape(d), w * v[0] + (1 - w) * v[1], atol=1e-6)
    assert abs(lse.item() - (max(s) + math.log1p(math.exp(-abs(s[0] - s[1]))))) < 1e-5


def test_attend_equals_textbook_gqa_attention():
    M, L, H, G, d, T = 3, 2, 8, 2, 32, 77
    q = rand_bits(M, L, H, d)
    K, V = rand_bits(T, L, G, d), rand_bits(T, L, G, d)
    vK, vV = _view_from_tokens(K, V)
    out, lse = orc.attend(q, vK, vV, T)
    qf, Kf, Vf = (from_bits(a).astype(np.float64) for a in (q, K, V))
    for m in range(M):
        for l in range(L):
            for h in range(H):
                g = h // (H // G)
                s = Kf[:, l, g, :] @ qf[m, l, h] / math.sqrt(d)
                assert np.allclose(out[m, l, h], softmax(s) @ Vf[:, l, g, :], atol=1e-6)
                assert abs(lse[m, l, h] - logsumexp(s)) < 1e-5


def test_attend_split_merge_identity():
    # attention over a concatenation = LSE-weighted merge of attention over the parts
    M, L, H, G, d, T = 1, 1, 2, 1, 16, 40
    q, vK, vV = rand_bits(M, L, H, d), rand_bits(L, G, T, d), rand_bits(L, G, T, d)
    o, l = orc.attend(q, vK, vV, T)
    oa, la = orc.attend(q, np.ascontiguousarray(vK[:, :, :15]), np.ascontiguousarray(vV[:, :, :15]), 15)
    ob, lb = orc.attend(q, np.ascontiguousarray(vK[:, :, 15:]), np.ascontiguousarray(vV[:, :, 15:]), T - 15)
    wa = 1 / (1 + np.exp(lb - la))
    assert np.allclose(o, wa[..., None] * oa + (1 - wa[..., None]) * ob, atol=1e-6)
    assert np.allclose(l, np.logaddexp(la, lb), atol=1e-5)


def test_attend_empty_view():
    out, lse = orc.attend(rand_bits(1, 1, 2, 8), rand_bits(1, 1, 4, 8), rand_bits(1, 1, 4, 8), 0)
    assert not out.any() and np.all(np.isneginf(lse))


# ------------------------------------------------------------------ whole path on small workspaces

def _pipeline(spec, qset=0, **sel_kw):
    K, V = kv_blocks(spec, 0, 0, spec.n_blocks)
    Kb, Vb = bits_of(K), bits_of(V)
    q = bits_of(make_queries(spec, qset))[0]
    table = page_table(spec)[0].numpy()
    repo = orc.Repository.empty(int(table.max()) + 1, spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim)
    repo.place(Kb, Vb, table)
    idx = orc.mean_k_index(Kb, spec.block_tokens)
    R, _ = orc.block_scores(q, idx, spec.n_blocks)
    kw = dict(budget_blocks=spec.budget_blocks, max_view_tokens=spec.max_view_tokens)
    kw.update(sel_kw)
    sel = orc.select(R, spec.block_tokens, **kw)
    vK, vV = orc.gather(repo, table, sel, max(len(sel), 1) * spec.block_tokens)
    out, lse = orc.attend(q, vK, vV, len(sel) * spec.block_tokens)
    return dict(K=Kb, V=Vb, q=q, R=R, sel=sel, out=out, lse=lse, vK=vK, vV=vV)


SMALL = CONFIGS["tiny"].with_(name="small", n_blocks=48, n_planted=4, budget_blocks=12, n_q_tokens=2)


def test_path_selecting_everything_equals_full_attention_over_the_raw_history():
    spec = SMALL
    res = _pipeline(spec, budget_blocks=10 ** 6, max_view_tokens=10 ** 9)
    assert res["sel"].tolist() == list(range(spec.n_blocks))
    qf, Kf, Vf = (from_bits(res[n]).astype(np.float64) for n in ("q", "K", "V"))
    r = spec.group
    for m in range(spec.n_q_tokens):
        for h in range(spec.n_q_heads):
            s = Kf[:, 0, h // r, :] @ qf[m, 0, h] / math.sqrt(spec.head_dim)
            assert np.allclose(res["out"][m, 0, h], softmax(s) @ Vf[:, 0, h // r, :], atol=1e-6)
            assert abs(res["lse"][m, 0, h] - logsumexp(s)) < 1e-5


def test_path_recovers_planted_blocks_within_budget_and_in_order():
    spec = SMALL
    res = _pipeline(spec)
    planted = set(planted_blocks(spec, 0)[0].tolist())
    assert planted <= set(res["sel"].tolist())
    assert len(res["sel"]) == spec.budget_blocks and np.all(np.diff(res["sel"]) > 0)
    assert len(res["sel"]) * spec.block_tokens <= spec.max_view_tokens
    gap = _pipeline(spec, budget_blocks=spec.n_planted)          # gap-forced variant: exactly the planted set
    assert set(gap["sel"].tolist()) == planted


def test_path_sparse_view_is_close_to_full_attention_by_the_mass_bound():
    # |O_sel - O_full|_inf <= 2 * (1 - covered mass) * max|V| for each (m, h)
    spec = SMALL
    res = _pipeline(spec)
    qf, Kf, Vf = (from_bits(res[n]).astype(np.float64) for n in ("q", "K", "V"))
    B, r = spec.block_tokens, spec.group
    tok = np.concatenate([np.arange(b * B, (b + 1) * B) for b in res["sel"]])
    for m in range(spec.n_q_tokens):
        for h in range(0, spec.n_q_heads, 5):
            g = h // r
            p = softmax(Kf[:, 0, g, :] @ qf[m, 0, h] / math.sqrt(spec.head_dim))
            full = p @ Vf[:, 0, g, :]
            miss = 1.0 - p[tok].sum()
            bound = 2 * miss * np.abs(Vf[:, 0, g, :]).max() + 1e-6
            assert np.abs(res["out"][m, 0, h] - full).max() <= bound


@pytest.mark.slow
def test_tiny_config_planted_recovery():
    spec = CONFIGS["tiny"]
    res = _pipeline(spec)
    planted = set(planted_blocks(spec, 0)[0].tolist())
    assert planted <= set(res["sel"].tolist()) and len(res["sel"]) == 32
    assert abs(res["R"].sum() - spec.n_q_tokens) < 1e-5


# ------------------------------------------------------------------ working-set delta (Eq. kvmem-working-set-delta)

def test_working_set_delta_matches_set_algebra():
    for n_prev, n_next, universe in [(0, 5, 20), (7, 0, 20), (12, 12, 15), (40, 33, 60), (9, 9, 9)]:
        prev = np.sort(rng.choice(universe, n_prev, replace=False)).astype(np.int32)
        nxt = np.sort(rng.choice(universe, n_next, replace=False)).astype(np.int32)
        ret, inc, out = orc.working_set_delta(prev, nxt)
        P, N = set(prev.tolist()), set(nxt.tolist())
        assert ret[:, 0].tolist() == sorted(P & N) and inc[:, 0].tolist() == sorted(N - P) and out.tolist() == sorted(P - N)
        assert len(ret) + len(inc) == n_next and len(ret) + len(out) == n_prev
        for bid, old, new in ret.tolist():
            assert prev[old] == bid and nxt[new] == bid           # slots index the chronological lists
        for bid, new in inc.tolist():
            assert nxt[new] == bid
    ret, inc, out = orc.working_set_delta(np.array([1, 4, 6], np.int32), np.array([2, 4, 6, 9], np.int32))
    assert ret.tolist() == [[4, 1, 1], [6, 2, 2]] and inc.tolist() == [[2, 0], [9, 3]] and out.tolist() == [1]
