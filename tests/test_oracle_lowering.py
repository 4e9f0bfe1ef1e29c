"""Pins of the metadata-lowering oracle (Sec. 3.4 / App. B.3; structured path of Sec. 3.2): its
boundaries and flags against a derivation that never sees ranges (numpy on the dense per-pair
mode vector), its table rows against the input lists, and its tag cross-check against a known
number of planted disagreements. CPU only."""
import numpy as np
import pytest

from oracle import lowering


def _random_state(rs, B=6, max_blocks=40, num_blocks=400, irregular=True):
    """A consistent scheduler state: per request a block list whose BASE pairs name one block twice,
    tags to match, dense pair modes."""
    free = list(rs.permutation(num_blocks))
    tags = np.zeros(num_blocks, np.uint8)
    lens, lists, modes = [], [], []
    for _ in range(B):
        nb = int(rs.integers(1, max_blocks + 1))
        L = nb * 16 - int(rs.integers(0, 16))
        npairs_full = nb // 2
        m = np.zeros((nb + 1) // 2, bool)
        if npairs_full:
            if irregular:
                m[:npairs_full] = rs.random(npairs_full) < 0.4
            else:
                a = int(rs.integers(0, npairs_full + 1)); b = int(rs.integers(a, npairs_full + 1))
                m[a:b] = True
        ids = []
        for p in range(len(m)):
            if m[p]:
                k = free.pop(); tags[k] = 1; ids += [k, k]
            else:
                ids.append(free.pop())
                if 2 * p + 1 < nb:
                    ids.append(free.pop())
        lens.append(L); lists.append(ids); modes.append(m)
    return tags, lens, lists, modes


@pytest.mark.parametrize("seed", range(6))
def test_boundaries_and_flags_match_the_dense_mode_vector(seed):
    rs = np.random.default_rng(seed)
    tags, lens, lists, modes = _random_state(rs, irregular=seed % 2 == 0)
    B = len(lens)
    rows = rs.permutation(B + 3)[:B]
    table = np.full((B + 3, 40), -7, np.int32)
    sl = np.full(B + 3, -7, np.int32)
    ranges = [lowering.ranges_of_modes(m) for m in modes]
    bounds, flags = lowering.lower_sparse(table, sl, tags, rows, lens, lists, ranges)
    for i in range(B):
        m = modes[i]
        idx = np.flatnonzero(m)
        exp = (idx[0], idx[-1] + 1) if len(idx) else (0, 0)
        assert tuple(bounds[rows[i]]) == exp
        assert list(table[rows[i], :len(lists[i])]) == lists[i]
        assert np.all(table[rows[i], len(lists[i]):] == -7)          # entries past the list are untouched
        assert sl[rows[i]] == lens[i]
    untouched = sorted(set(range(B + 3)) - set(rows.tolist()))
    assert np.all(table[untouched] == -7) and np.all(sl[untouched] == -7) and np.all(bounds[untouched] == 0)
    any_base = int(any(m.any() for m in modes))
    irregular = int(any(m.any() and m.sum() != np.flatnonzero(m)[-1] + 1 - np.flatnonzero(m)[0] for m in modes))
    assert list(flags) == [any_base, irregular, 0, 0]


def test_planted_disagreements_are_counted():
    rs = np.random.default_rng(42)
    tags, lens, lists, modes = _random_state(rs, B=5, irregular=True)
    ranges = [lowering.ranges_of_modes(m) for m in modes]
    rows = np.arange(5)
    planted = 0
    first = None
    for i in (1, 3):
        m = modes[i]
        if len(m) < 2:
            continue
        p = int(rs.integers(0, len(m) - 1))                # a full pair: flip its tag
        tags[lists[i][2 * p]] ^= 1
        planted += 1
        first = i if first is None else first
    table = np.zeros((5, 40), np.int32); sl = np.zeros(5, np.int32)
    _, flags = lowering.lower_sparse(table, sl, tags, rows, lens, lists, ranges)
    assert flags[2] == planted and flags[3] == (5 - first if planted else 0)


def test_touching_ranges_count_as_one_run():
    tags = np.zeros(20, np.uint8); tags[[1, 2, 3]] = 1
    ids = [0, 9, 1, 1, 2, 2, 3, 3, 4]                      # pairs: T B B B, then an unpaired block
    table = np.zeros((1, 16), np.int32); sl = np.zeros(1, np.int32)
    b, f = lowering.lower_sparse(table, sl, tags, [0], [9 * 16], [ids], [[(1, 2), (2, 4)]])
    assert tuple(b[0]) == (1, 4) and list(f) == [1, 0, 0, 0]
    b, f = lowering.lower_sparse(table, sl, tags, [0], [9 * 16], [ids], [[(1, 2), (3, 4)]])
    assert tuple(b[0]) == (1, 4) and f[0] == 1 and f[1] == 1 and f[2] == 1     # pair 2 is tagged BASE but outside every range


def test_ranges_of_modes_round_trip():
    rs = np.random.default_rng(3)
    for _ in range(50):
        m = rs.random(int(rs.integers(0, 30))) < 0.5
        back = np.zeros(len(m), bool)
        for a, b in lowering.ranges_of_modes(m):
            assert a < b
            back[a:b] = True
        assert np.array_equal(back, m)
