"""Pins for the oracle's execution cache (working-set reuse with bounded delta re-RoPE, Sec. 4.4):
what the paper and rotary arithmetic fix, checked without reference to the oracle's own formulas."""
import numpy as np
from conftest import from_bits, to_bits

from oracle import kvmem_oracle as orc

THETA = 1.0e6
B, L, G, d, NB = 4, 1, 2, 16, 24


def _setup(seed=5, cap=8, n_pos=256):
    rng = np.random.default_rng(seed)
    K = to_bits(rng.standard_normal((NB * B, L, G, d)).astype(np.float32))
    V = to_bits(rng.standard_normal((NB * B, L, G, d)).astype(np.float32))
    table = rng.permutation(NB).astype(np.int32)
    repo = orc.Repository.empty(NB, B, L, G, d)
    repo.place(K, V, table)
    tab = orc.rope_table(n_pos, d, THETA)
    return rng, K, V, table, repo, tab, orc.ViewCache(repo, cap)


def _ids(*xs):
    return np.array(xs, np.int32)


def test_first_fill_equals_the_position_consistent_gather():
    _, _, _, table, repo, tab, cache = _setup()
    sel = _ids(1, 4, 5, 9, 17)
    stats = cache.update(repo, table, sel, max_delta=3, first_pos=7, tab=tab)
    assert list(stats) == [0, 0, 0, 5]                                   # everything is incoming
    vK, vV = cache.view(8 * B)
    gK, gV = orc.gather_rope(repo, table, sel, 8 * B, 7, tab)
    assert np.array_equal(vK, gK) and np.array_equal(vV, gV)
    assert list(cache.view_slots[:5]) == [0, 1, 2, 3, 4]                 # lowest free slots in ascending id order
    assert list(cache.slot_block[:5]) == list(sel) and np.all(cache.slot_block[5:] == -1)


def test_same_selection_again_touches_nothing():
    _, _, _, table, repo, tab, cache = _setup()
    sel = _ids(0, 3, 8, 20)
    cache.update(repo, table, sel, 2, 0, tab)
    K0, V0, slots0 = cache.K.copy(), cache.V.copy(), cache.view_slots.copy()
    stats = cache.update(repo, table, sel, 2, 0, tab)
    assert list(stats) == [4, 0, 0, 0]
    assert np.array_equal(cache.K, K0) and np.array_equal(cache.V, V0) and np.array_equal(cache.view_slots, slots0)
    assert np.all(cache.slot_cnt == 0)


def test_with_no_delta_budget_every_update_is_a_fresh_position_consistent_view():
    rng, _, _, table, repo, tab, cache = _setup(cap=10)
    for step in range(6):
        sel = np.sort(rng.choice(NB, size=int(rng.integers(3, 11)), replace=False)).astype(np.int32)
        cache.update(repo, table, sel, max_delta=0, first_pos=3, tab=tab)
        vK, vV = cache.view(10 * B)
        gK, gV = orc.gather_rope(repo, table, sel, 10 * B, 3, tab)
        assert np.array_equal(vK, gK) and np.array_equal(vV, gV), step
        assert np.all(cache.slot_cnt == 0)


def test_retained_blocks_keep_their_slot_and_incoming_take_the_lowest_free_ones():
    _, _, _, table, repo, tab, cache = _setup(cap=6)
    cache.update(repo, table, _ids(2, 5, 7, 11, 13), 4, 0, tab)          # slots 0..4
    slot_of = {int(b): int(s) for b, s in zip([2, 5, 7, 11, 13], cache.view_slots[:5])}
    stats = cache.update(repo, table, _ids(1, 5, 6, 11, 19, 21), 4, 0, tab)
    # retained: 5 (j 1 -> 1, unmoved), 11 (j 3 -> 3, unmoved); incoming 1, 6, 19, 21; outgoing 2, 7, 13 free slots 0, 2, 4; slot 5 was empty
    assert list(stats) == [2, 0, 0, 4]
    assert cache.view_slots[1] == slot_of[5] and cache.view_slots[3] == slot_of[11]
    assert [int(cache.view_slots[j]) for j in (0, 2, 4, 5)] == [0, 2, 4, 5]
    assert sorted(cache.view_slots[:6]) == list(range(6))                # a permutation of the slots
    for j, b in enumerate([1, 5, 6, 11, 19, 21]):
        s = cache.view_slots[j]
        assert cache.slot_block[s] == b and cache.slot_pos[s] == j
    # every block, moved or not, has bit-exact values
    vK, vV = cache.view(6 * B)
    _, gV = orc.gather_rope(repo, table, _ids(1, 5, 6, 11, 19, 21), 6 * B, 0, tab)
    assert np.array_equal(vV, gV)


def test_delta_rotation_is_the_textbook_rotation_of_the_cached_keys_by_the_position_change():
    _, _, _, table, repo, tab, cache = _setup(cap=8, n_pos=512)
    cache.update(repo, table, _ids(3, 6, 9, 12), 5, 10, tab)
    before = {int(b): from_bits(cache.K[cache.view_slots[j]]).astype(np.float64) for j, b in enumerate([3, 6, 9, 12])}
    # block 3 leaves, block 20 joins at the end: 6, 9, 12 move one block towards the front (delta = -B positions)
    stats = cache.update(repo, table, _ids(6, 9, 12, 20), 5, 10, tab)
    assert list(stats) == [0, 3, 0, 1]
    half = d // 2
    freq = THETA ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = -B * freq                                                      # rotation by -B positions
    c, s = np.cos(ang), np.sin(ang)
    for j, b in enumerate([6, 9, 12]):
        x = before[b]                                                    # [B][L][G][d], the bf16 values that were cached
        want = np.concatenate([x[..., :half] * c - x[..., half:] * s, x[..., half:] * c + x[..., :half] * s], axis=-1)
        got = from_bits(cache.K[cache.view_slots[j]]).astype(np.float64)
        assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-6)
        assert cache.slot_cnt[cache.view_slots[j]] == 1
    # and they stay close to keys rebuilt from raw K at the new positions: two bf16 roundings apart
    gK, _ = orc.gather_rope(repo, table, _ids(6, 9, 12, 20), 8 * B, 10, tab)
    vK, _ = cache.view(8 * B)
    assert np.abs(from_bits(vK) - from_bits(gK)).max() <= 2.0 ** -5
    assert np.array_equal(vK[:, :, 3 * B:4 * B], gK[:, :, 3 * B:4 * B])  # the incoming block is exact


def test_counter_bounds_the_delta_operations_between_reconstructions():
    _, _, _, table, repo, tab, cache = _setup(cap=8, n_pos=512)
    # block 10 is always selected; one block before it joins or leaves every step, so it moves every step
    sels = [_ids(10), _ids(2, 10), _ids(2, 4, 10), _ids(4, 10), _ids(10), _ids(1, 10), _ids(1, 3, 10)]
    cnts, kinds = [], []
    for sel in sels:
        stats = cache.update(repo, table, sel, max_delta=2, first_pos=0, tab=tab)
        s = cache.view_slots[len(sel) - 1]
        assert cache.slot_block[s] == 10
        cnts.append(int(cache.slot_cnt[s]))
        kinds.append((int(stats[1]), int(stats[2])))
        if cnts[-1] == 0:                                                # freshly built: bit-exact against the gather
            gK, _ = orc.gather_rope(repo, table, sel, 8 * B, 0, tab)
            vK, _ = cache.view(8 * B)
            j = len(sel) - 1
            assert np.array_equal(vK[:, :, j * B:(j + 1) * B], gK[:, :, j * B:(j + 1) * B])
    assert cnts == [0, 1, 2, 0, 1, 2, 0]                                 # delta, delta, rebuild, delta, delta, rebuild
    # block 10's own operation each step: steps 1, 2 delta; 3 rebuild; 4, 5 delta; 6 rebuild
    assert [k[1] >= 1 for k in kinds] == [False, False, False, True, False, False, True]


def test_attention_over_the_cache_matches_attention_over_a_fresh_view_within_rounding():
    rng, _, _, table, repo, tab, cache = _setup(seed=9, cap=10, n_pos=512)
    H = 4
    q = to_bits(rng.standard_normal((2, L, H, d)).astype(np.float32))
    prev = np.sort(rng.choice(NB, size=8, replace=False)).astype(np.int32)
    cache.update(repo, table, prev, 3, 0, tab)
    for _ in range(3):                                                   # three overlapping working sets
        keep = rng.choice(prev, size=5, replace=False)
        new = rng.choice(np.setdiff1d(np.arange(NB), prev), size=3, replace=False)
        prev = np.sort(np.concatenate([keep, new])).astype(np.int32)
        cache.update(repo, table, prev, 3, 0, tab)
    vK, vV = cache.view(10 * B)
    gK, gV = orc.gather_rope(repo, table, prev, 10 * B, 0, tab)
    T = len(prev) * B
    O1, lse1 = orc.attend(q, vK, vV, T)
    O2, lse2 = orc.attend(q, gK, gV, T)
    assert np.abs(O1 - O2).max() < 3e-2 and np.abs(lse1 - lse2).max() < 3e-2
    assert np.array_equal(vV, gV)


def test_selection_larger_than_the_cache_is_refused():
    _, _, _, table, repo, tab, cache = _setup(cap=3)
    try:
        cache.update(repo, table, _ids(1, 2, 3, 4), 1, 0, tab)
    except ValueError:
        return
    raise AssertionError("expected a refusal")


def test_in_block_layout_loads_and_rebuilds_with_the_block_position_only():
    rng, K, V, table, repo, tab, cache = _setup(cap=8, n_pos=512)
    # store k' = R(t) k instead of the raw keys
    t_in_block = (np.arange(NB * B) % B).astype(np.int32)
    Kp = orc.rope_rotate(np.ascontiguousarray(K.reshape(NB * B, L * G, d)), t_in_block, tab).reshape(K.shape)
    stored = orc.Repository.empty(NB, B, L, G, d)
    stored.place(Kp, V, table)
    for step, sel in enumerate([_ids(3, 6, 9, 12), _ids(6, 9, 12, 20), _ids(1, 6, 12, 20, 22)]):
        cache.update(stored, table, sel, max_delta=0, first_pos=10, tab=tab, in_block=True)     # always rebuilt
        vK, vV = cache.view(8 * B)
        gK, gV = orc.gather_rope(stored, table, sel, 8 * B, 10, tab, in_block=True)
        assert np.array_equal(vK, gK) and np.array_equal(vV, gV), step
