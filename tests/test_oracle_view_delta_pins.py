"""Pins of the oracle's incremental contiguous view (Eq. "kvmem-working-set-delta", Sec. 4.4): after any sequence of
working sets the updated view must equal the plain gather of the last one (its definition, a pinned function), a
slot whose block stays must not be read again, and the counts must be those of the pinned working-set delta."""
import numpy as np

from oracle import kvmem_oracle as orc


def _repo(rng, n_blocks=40, B=16, L=2, G=2, d=8):
    repo = orc.Repository.empty(n_blocks, B, L, G, d)
    K = rng.integers(0, 1 << 16, size=(n_blocks * B, L, G, d), dtype=np.uint16)
    V = rng.integers(0, 1 << 16, size=(n_blocks * B, L, G, d), dtype=np.uint16)
    table = rng.permutation(n_blocks).astype(np.int32)
    repo.place(K, V, table)
    return repo, table


def _sets(rng, n_blocks, sizes, keep=0.7):
    prev = np.sort(rng.choice(n_blocks, size=sizes[0], replace=False)).astype(np.int32)
    out = [prev]
    for n in sizes[1:]:
        n_keep = min(int(round(keep * len(prev))), n)
        kept = rng.choice(prev, size=n_keep, replace=False)
        rest = np.setdiff1d(np.arange(n_blocks), prev)
        prev = np.sort(np.concatenate([kept, rng.choice(rest, size=n - n_keep, replace=False)])).astype(np.int32)
        out.append(prev)
    return out


def test_updated_view_equals_the_gather_of_the_new_working_set():
    rng = np.random.default_rng(0)
    repo, table = _repo(rng)
    cap = 20 * 16
    vK, vV = np.zeros((2, 2, cap, 8), np.uint16), np.zeros((2, 2, cap, 8), np.uint16)
    prev = np.zeros(0, np.int32)
    for sel in _sets(rng, 40, [12, 12, 20, 5, 12, 1, 19, 20]):
        orc.view_update(repo, table, vK, vV, prev, sel)
        gK, gV = orc.gather(repo, table, sel, cap)
        T = len(sel) * 16
        assert np.array_equal(vK[:, :, :T], gK[:, :, :T]) and np.array_equal(vV[:, :, :T], gV[:, :, :T])
        prev = sel


def test_counts_are_those_of_the_working_set_delta():
    rng = np.random.default_rng(1)
    for sizes in ([10, 10], [10, 14], [14, 3], [1, 1], [8, 8]):
        prev, nxt = _sets(rng, 30, sizes)
        action, counts = orc.view_delta_plan(prev, nxt)
        ret, inc, out = orc.working_set_delta(prev, nxt)
        unmoved = int(sum(1 for (_, a, b) in ret if a == b))
        assert counts.tolist() == [unmoved, len(ret) - unmoved, len(inc)]
        assert sorted(nxt[action == 2].tolist()) == sorted(inc[:, 0].tolist())
        assert len(action) == len(nxt) and counts.sum() == len(nxt)


def test_hand_example():
    # prev = [2 5 7 9], next = [2 5 8 9 11]: slots 0, 1 stay; 8 is incoming at slot 2; 9 moves from slot 3 to slot 3 (stays);
    # 11 is incoming at slot 4
    action, counts = orc.view_delta_plan(np.array([2, 5, 7, 9], np.int32), np.array([2, 5, 8, 9, 11], np.int32))
    assert action.tolist() == [0, 0, 2, 0, 2] and counts.tolist() == [3, 0, 2]
    # one insertion in front shifts every retained block by one slot
    action, counts = orc.view_delta_plan(np.array([2, 5, 7, 9], np.int32), np.array([1, 2, 5, 7], np.int32))
    assert action.tolist() == [2, 1, 1, 1] and counts.tolist() == [0, 3, 1]


def test_a_slot_whose_block_stays_is_not_read_again():
    rng = np.random.default_rng(2)
    repo, table = _repo(rng)
    cap = 8 * 16
    vK, vV = np.zeros((2, 2, cap, 8), np.uint16), np.zeros((2, 2, cap, 8), np.uint16)
    prev = np.array([3, 4, 10, 20], np.int32)
    orc.view_update(repo, table, vK, vV, np.zeros(0, np.int32), prev)
    before = vK.copy()
    repo.pagesK[table[4]] ^= 0xFFFF                      # the repository copy of a block that stays in its slot changes ...
    nxt = np.array([3, 4, 11, 20, 30], np.int32)
    counts = orc.view_update(repo, table, vK, vV, prev, nxt)
    assert counts.tolist() == [3, 0, 2]
    assert np.array_equal(vK[:, :, 16:32], before[:, :, 16:32])      # ... and the view does not notice: slot 1 was not touched
    gK, _ = orc.gather(repo, table, nxt, cap)
    assert np.array_equal(vK[:, :, 32:80], gK[:, :, 32:80])          # the incoming blocks and the other retained one are right


def test_same_working_set_again_moves_nothing_and_an_empty_one_is_a_plain_gather():
    rng = np.random.default_rng(3)
    repo, table = _repo(rng)
    cap = 10 * 16
    sel = np.array([0, 7, 8, 33], np.int32)
    vK, vV = np.zeros((2, 2, cap, 8), np.uint16), np.zeros((2, 2, cap, 8), np.uint16)
    c0 = orc.view_update(repo, table, vK, vV, np.zeros(0, np.int32), sel)
    assert c0.tolist() == [0, 0, 4]
    gK, gV = orc.gather(repo, table, sel, cap)
    assert np.array_equal(vK, gK) and np.array_equal(vV, gV)
    c1 = orc.view_update(repo, table, vK, vV, sel, sel)
    assert c1.tolist() == [4, 0, 0] and np.array_equal(vK, gK)
    vK[:, :, 64:] = 0xABCD                                # tokens past the new view are left as they were
    orc.view_update(repo, table, vK, vV, sel, sel[:2])
    assert np.all(vK[:, :, 64:] == 0xABCD)
