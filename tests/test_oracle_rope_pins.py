"""Pins for the oracle's RoPE functions: what rotary position embedding fixes mathematically."""
import math

import numpy as np
from conftest import from_bits, to_bits

from oracle import kvmem_oracle as orc

rng = np.random.default_rng(77)
THETA = 1.0e6


def _textbook_rope(x, pos, d, theta):
    """fp64 rotate-half RoPE written the usual way: x * cos + rotate_half(x) * sin."""
    half = d // 2
    freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = np.asarray(pos, np.float64)[:, None] * freq[None, :]
    cos = np.concatenate([np.cos(ang), np.cos(ang)], axis=-1)[:, None, :]
    sin = np.concatenate([np.sin(ang), np.sin(ang)], axis=-1)[:, None, :]
    rot = np.concatenate([-x[..., half:], x[..., :half]], axis=-1)
    return x * cos + rot * sin


def test_table_entries_are_cos_sin_of_position_times_frequency():
    d, n = 16, 300
    tab = orc.rope_table(n, d, THETA)
    assert np.all(tab[0, :, 0] == 1.0) and np.all(tab[0, :, 1] == 0.0)            # position 0: no rotation
    assert np.allclose(tab[:, 0, 0], np.cos(np.arange(n)), atol=1e-7)             # pair 0 has frequency 1
    assert np.allclose(tab[:, 0, 1], np.sin(np.arange(n)), atol=1e-7)
    f5 = THETA ** (-10.0 / d)
    assert abs(tab[123, 5, 0] - math.cos(123 * f5)) < 1e-7 and abs(tab[123, 5, 1] - math.sin(123 * f5)) < 1e-7
    assert np.allclose(tab[..., 0] ** 2 + tab[..., 1] ** 2, 1.0, atol=1e-6)


def test_rotation_matches_textbook_rope_within_one_bf16_ulp():
    d, rows, vec = 64, 40, 3
    x = to_bits(rng.standard_normal((rows, vec, d)).astype(np.float32))
    pos = rng.integers(0, 5000, rows).astype(np.int32)
    tab = orc.rope_table(5000, d, THETA)
    y = from_bits(orc.rope_rotate(x, pos, tab)).astype(np.float64)
    ref = _textbook_rope(from_bits(x).astype(np.float64), pos, d, THETA)
    ulp = np.maximum(np.abs(ref), 2.0 ** -126) * 2.0 ** -8
    assert np.all(np.abs(y - ref) <= ulp + 1e-6)


def test_position_zero_is_identity_and_quarter_turn_swaps_halves():
    d = 8
    x = to_bits(rng.standard_normal((2, 1, d)).astype(np.float32))
    tab = orc.rope_table(4, d, THETA)
    assert np.array_equal(orc.rope_rotate(x, np.zeros(2, np.int32), tab), x)
    # a hand-made table row with angle pi/2 for every pair: (a, b) -> (-b, a)
    quarter = np.zeros((1, d // 2, 2), np.float32)
    quarter[0, :, 1] = 1.0
    y = from_bits(orc.rope_rotate(x, np.zeros(2, np.int32), quarter))
    xf = from_bits(x)
    assert np.array_equal(y[..., : d // 2], -xf[..., d // 2:]) and np.array_equal(y[..., d // 2:], xf[..., : d // 2])


def test_inverse_undoes_forward_up_to_bf16_rounding_and_norms_are_kept():
    d, rows = 128, 64
    x = to_bits(rng.standard_normal((rows, 2, d)).astype(np.float32))
    pos = rng.integers(0, 100000, rows).astype(np.int32)
    tab = orc.rope_table(100000, d, THETA)
    y = orc.rope_rotate(x, pos, tab)
    back = from_bits(orc.rope_rotate(y, pos, tab, inverse=True))
    xf, yf = from_bits(x), from_bits(y)
    assert np.abs(back - xf).max() <= 2.0 ** -6                                      # two bf16 roundings of values ~ N(0,1)
    assert np.allclose(np.linalg.norm(yf, axis=-1), np.linalg.norm(xf, axis=-1), rtol=5e-3)


def test_attention_logit_depends_only_on_relative_position():
    # <RoPE(q, m), RoPE(k, n)> is a function of m - n
    d = 64
    q = to_bits(rng.standard_normal((1, 1, d)).astype(np.float32))
    k = to_bits(rng.standard_normal((1, 1, d)).astype(np.float32))
    tab = orc.rope_table(3000, d, THETA)

    def logit(m, n):
        qm = from_bits(orc.rope_rotate(q, np.array([m], np.int32), tab)).reshape(d).astype(np.float64)
        kn = from_bits(orc.rope_rotate(k, np.array([n], np.int32), tab)).reshape(d).astype(np.float64)
        return float(qm @ kn)
    base = logit(17, 5)
    for shift in (1, 100, 2500):
        assert abs(logit(17 + shift, 5 + shift) - base) < 0.15                        # bf16 rounding of 64 terms
    assert abs(logit(17, 5) - logit(400, 5)) > 1e-3                                   # and it does depend on m - n


def test_rotating_twice_adds_positions():
    # delta re-RoPE identity (Sec. 4.4): RoPE(RoPE(x, a), b) = RoPE(x, a + b) up to rounding
    d = 32
    x = to_bits(rng.standard_normal((5, 1, d)).astype(np.float32))
    tab = orc.rope_table(1000, d, THETA)
    a, b = np.full(5, 300, np.int32), np.full(5, 45, np.int32)
    two = from_bits(orc.rope_rotate(orc.rope_rotate(x, a, tab), b, tab))
    one = from_bits(orc.rope_rotate(x, a + b, tab))
    assert np.abs(two - one).max() <= 2.0 ** -5


def test_gather_rope_rotates_keys_to_compact_positions_and_copies_values():
    B, L, G, d, NB = 4, 1, 2, 16, 9
    K, V = to_bits(rng.standard_normal((NB * B, L, G, d)).astype(np.float32)), to_bits(rng.standard_normal((NB * B, L, G, d)).astype(np.float32))
    table = rng.permutation(NB).astype(np.int32)
    repo = orc.Repository.empty(NB, B, L, G, d)
    repo.place(K, V, table)
    sel = np.array([2, 3, 7], np.int32)
    tab = orc.rope_table(64, d, THETA)
    first = 5
    vK, vV = orc.gather_rope(repo, table, sel, 4 * B, first, tab)
    plainK, plainV = orc.gather(repo, table, sel, 4 * B)
    assert np.array_equal(vV, plainV)                                                 # V is copied unchanged
    for j, b in enumerate(sel):
        for t in range(B):
            want = orc.rope_rotate(np.ascontiguousarray(K[b * B + t].reshape(1, L * G, d)),
                                   np.array([first + j * B + t], np.int32), tab).reshape(L, G, d)
            assert np.array_equal(vK[:, :, j * B + t, :], want)
    # with an all-zero position table offset (first_pos = 0, single block at j = 0, t = 0) the first token is unrotated
    vK0, _ = orc.gather_rope(repo, table, sel[:1], B, 0, tab)
    assert np.array_equal(vK0[:, :, 0, :], K[sel[0] * B])


# ---- keys stored with the rotation of their offset inside the block ("in-block" layout) -------------------

def _in_block_repo(B=8, L=1, G=2, d=32, NB=10, seed=21, n_pos=512):
    r = np.random.default_rng(seed)
    K = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    V = to_bits(r.standard_normal((NB * B, L, G, d)).astype(np.float32))
    tab = orc.rope_table(n_pos, d, THETA)
    t_in_block = (np.arange(NB * B) % B).astype(np.int32)
    Kp = orc.rope_rotate(K.reshape(NB * B, L * G, d), t_in_block, tab).reshape(K.shape)      # k' = R(t) k
    table = r.permutation(NB).astype(np.int32)
    raw, stored = orc.Repository.empty(NB, B, L, G, d), orc.Repository.empty(NB, B, L, G, d)
    raw.place(K, V, table)
    stored.place(Kp, V, table)
    return r, K, V, Kp, table, raw, stored, tab


def test_in_block_view_rotates_stored_keys_by_the_block_position_only():
    _, _, _, Kp, table, raw, stored, tab = _in_block_repo()
    B, L, G, d = 8, 1, 2, 32
    sel = np.array([1, 4, 7, 8], np.int32)
    first = 19
    vK, vV = orc.gather_rope(stored, table, sel, 5 * B, first, tab, in_block=True)
    for j, b in enumerate(sel):
        rows = np.ascontiguousarray(Kp[b * B:(b + 1) * B].reshape(B, L * G, d))
        want = orc.rope_rotate(rows, np.full(B, first + j * B, np.int32), tab).reshape(B, L, G, d)   # one angle per block
        assert np.array_equal(vK[:, :, j * B:(j + 1) * B].transpose(2, 0, 1, 3), want)
    # the same keys, to two bf16 roundings, as rotating the raw keys to first + j*B + t (rotations add)
    rK, rV = orc.gather_rope(raw, table, sel, 5 * B, first, tab)
    assert np.array_equal(vV, rV)
    assert np.abs(from_bits(vK) - from_bits(rK)).max() <= 2.0 ** -5


def test_query_rotation_gives_the_logits_of_rotated_keys():
    r, _, _, _, table, raw, stored, tab = _in_block_repo(seed=33)
    B, L, G, d, H, M = 8, 1, 2, 32, 4, 2
    sel = np.array([0, 2, 3, 6, 9], np.int32)
    T, cap, first = len(sel) * B, 6 * B, 40
    q = to_bits(r.standard_normal((M, L, H, d)).astype(np.float32))
    sK, sV = orc.gather(stored, table, sel, cap)                         # the stored keys, not rotated further
    O1, lse1 = orc.attend_qrot(q, sK, sV, T, B, first, tab)
    # (R(-p0) q) . k' = q . R(p0) k': attention over the view that kvo_gather_rope builds from the same pages
    vK, vV = orc.gather_rope(stored, table, sel, cap, first, tab, in_block=True)
    O2, lse2 = orc.attend(q, vK, vV, T)
    assert np.abs(O1 - O2).max() < 2e-2 and np.abs(lse1 - lse2).max() < 2e-2
    # and over the view of raw keys rotated to their compact positions
    rK, rV = orc.gather_rope(raw, table, sel, cap, first, tab)
    O3, lse3 = orc.attend(q, rK, rV, T)
    assert np.abs(O1 - O3).max() < 3e-2 and np.abs(lse1 - lse3).max() < 3e-2


def test_query_rotation_at_position_zero_is_plain_attention_over_the_stored_keys():
    r, _, _, _, table, _, stored, tab = _in_block_repo(seed=5)
    B, d = 8, 32
    q = to_bits(r.standard_normal((1, 1, 4, d)).astype(np.float32))
    sel = np.array([3], np.int32)
    sK, sV = orc.gather(stored, table, sel, B)
    O1, lse1 = orc.attend_qrot(q, sK, sV, B, B, 0, tab)                   # one tile at position 0: R(0) = identity
    O2, lse2 = orc.attend(q, sK, sV, B)
    assert np.array_equal(O1, O2) and np.array_equal(lse1, lse2)
    # the rotated query itself: each tile uses the bf16 query of kvo_rope_rotate(inverse) at its position
    sel2 = np.array([3, 5], np.int32)
    sK2, sV2 = orc.gather(stored, table, sel2, 2 * B)
    q_rot = orc.rope_rotate(np.ascontiguousarray(q.reshape(1, 4, d)), np.array([B], np.int32), tab, inverse=True).reshape(q.shape)
    # logits of the second tile alone, from LSEs: lse(both) = log(exp(lse(tile 0 with q)) + exp(lse(tile 1 with q_rot)))
    _, l_both = orc.attend_qrot(q, sK2, sV2, 2 * B, B, 0, tab)
    _, l0 = orc.attend(q, sK2[:, :, :B].copy(), sV2[:, :, :B].copy(), B)
    _, l1 = orc.attend(q_rot, sK2[:, :, B:].copy(), sV2[:, :, B:].copy(), B)
    assert np.allclose(l_both, np.logaddexp(l0, l1), atol=1e-5)


def test_composed_angles_stay_within_three_fp32_steps_of_the_table():
    """The bound behind the tolerance on keys rotated with composed angles: (cos, sin)(p1 + b) formed in fp32 from the
    table rows of p1 and b (two products, two fused multiply-adds) is within 3 * 2^-24 of the table's own row of p1 + b,
    for every warp share (b < 16) of a long window."""
    d, n = 128, 1 << 15
    tab = orc.rope_table(n, d, THETA)
    p1 = np.arange(0, n - 16, 16, dtype=np.int64)
    worst = 0.0
    for b in range(16):
        cb, sb = tab[p1, :, 0], tab[p1, :, 1]
        co, so = tab[b, :, 0][None, :], tab[b, :, 1][None, :]
        # fp32 products rounded once, then a fused multiply-add (exact product, one rounding): emulated in fp64
        c = (cb.astype(np.float64) * co.astype(np.float64) - (sb * so).astype(np.float64)).astype(np.float32)
        s = (sb.astype(np.float64) * co.astype(np.float64) + (cb * so).astype(np.float64)).astype(np.float32)
        worst = max(worst, float(np.abs(c - tab[p1 + b, :, 0]).max()), float(np.abs(s - tab[p1 + b, :, 1]).max()))
    assert worst <= 3 * 2.0 ** -24, worst
