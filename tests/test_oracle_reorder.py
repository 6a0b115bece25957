"""Pins of the oracle's bitmap-aware row reordering (paper Sec. V-B, Eqs. 3-5, Alg. 1): hand-worked
cases, exhaustive search over every grouping of small tiles, closed forms, and agreement with the
IE-BME encoder's count of active union-mask entries. None of the checks reuses the oracle's own
cost or search code."""
import itertools

import numpy as np
import pytest

import oracle


def _golden_cases(path):
    lines = [l.strip() for l in path.read_text().splitlines() if l.strip() and not l.startswith("#")]
    i = 0
    while i < len(lines):
        H_L, K_L, R_A, C_A = map(int, lines[i].split())
        mask = np.array([[int(ch) for ch in lines[i + 1 + r]] for r in range(H_L)], dtype=np.uint8)
        assert mask.shape == (H_L, K_L)
        tail = list(map(int, lines[i + 1 + H_L].split()))
        yield mask, R_A, C_A, tail[0], tail[1:]
        i += H_L + 2


def test_hand_worked_cases(golden_dir):
    n = 0
    for mask, R_A, C_A, cost, perm in _golden_cases(golden_dir / "reorder_small.txt"):
        p, c = oracle.reorder_tile(mask, R_A, C_A)
        assert c == cost
        assert list(p) == perm
        n += 1
    assert n == 4


def _cost_of_groups(mask, groups, C_A):
    """Eqs. 3-4 written with numpy: fold the C_A column partitions, OR the rows of a group."""
    H_L, K_L = mask.shape
    folded = mask.reshape(H_L, C_A, K_L // C_A).any(axis=1)
    return int(sum(folded[list(g)].any(axis=0).sum() for g in groups))


def _all_groupings(rows, R_A):
    """Every split of `rows` into unordered groups of R_A (lowest row always placed first)."""
    if not rows:
        yield []
        return
    first, rest = rows[0], rows[1:]
    for partners in itertools.combinations(rest, R_A - 1):
        left = [r for r in rest if r not in partners]
        for tail in _all_groupings(left, R_A):
            yield [(first,) + partners] + tail


def _groups_of(perm, R_A):
    n_groups = len(perm) // R_A
    return [tuple(int(perm[p * n_groups + g]) for p in range(R_A)) for g in range(n_groups)]


def _check_canonical(perm, R_A):
    groups = _groups_of(perm, R_A)
    assert sorted(int(r) for r in perm) == list(range(len(perm)))
    assert all(list(g) == sorted(g) for g in groups)
    assert groups == sorted(groups)


@pytest.mark.parametrize("H_L,K_L,R_A,C_A,density,n_groupings", [
    (8, 64, 2, 1, 0.5, 105), (8, 64, 2, 2, 0.3, 105), (8, 32, 4, 1, 0.4, 35), (8, 64, 4, 2, 0.2, 35),
    (6, 24, 3, 1, 0.5, 10), (12, 48, 2, 1, 0.5, 10395), (12, 48, 3, 2, 0.25, 15400),
])
def test_optimum_equals_exhaustive_search(H_L, K_L, R_A, C_A, density, n_groupings):
    for seed in range(4):
        rng = np.random.default_rng([seed, H_L, R_A, C_A])
        mask = (rng.random((H_L, K_L)) < density).astype(np.uint8)
        costs = [_cost_of_groups(mask, g, C_A) for g in _all_groupings(list(range(H_L)), R_A)]
        assert len(costs) == n_groupings
        perm, cost = oracle.reorder_tile(mask, R_A, C_A)
        assert cost == min(costs)
        _check_canonical(perm, R_A)
        assert _cost_of_groups(mask, _groups_of(perm, R_A), C_A) == cost


def test_sixteen_rows_against_every_perfect_matching():
    # 15!! = 2 027 025 matchings of 16 rows; pair costs from a table keep the search quick.
    rng = np.random.default_rng(16)
    mask = (rng.random((16, 128)) < 0.5).astype(np.uint8)
    pair = np.array([[int((mask[a] | mask[b]).sum()) for b in range(16)] for a in range(16)])
    best = [10 ** 9]
    count = [0]

    def search(rows, acc):
        if not rows:
            count[0] += 1
            best[0] = min(best[0], acc)
            return
        a = rows[0]
        for i in range(1, len(rows)):
            search(rows[1:i] + rows[i + 1:], acc + pair[a][rows[i]])

    search(list(range(16)), 0)
    assert count[0] == 2027025
    perm, cost = oracle.reorder_tile(mask, 2, 1)
    assert cost == best[0]
    _check_canonical(perm, 2)


def test_duplicated_rows_with_disjoint_supports_pair_up():
    # Eight patterns on disjoint column ranges, each used by two rows at scattered positions:
    # pairing equal rows costs |a|, any other pair |a| + |b|, so the optimum is unique.
    rng = np.random.default_rng(5)
    K_L = 8 * 16
    patterns = np.zeros((8, K_L), np.uint8)
    for i in range(8):
        patterns[i, 16 * i: 16 * i + 16] = rng.random(16) < 0.6
        patterns[i, 16 * i] = 1
    where = rng.permutation(16)
    mask = np.zeros((16, K_L), np.uint8)
    for i in range(8):
        mask[where[2 * i]] = patterns[i]
        mask[where[2 * i + 1]] = patterns[i]
    perm, cost = oracle.reorder_tile(mask, 2, 1)
    assert cost == int(patterns.sum())
    want = sorted(tuple(sorted((int(where[2 * i]), int(where[2 * i + 1])))) for i in range(8))
    assert _groups_of(perm, 2) == want
    assert list(perm[:8]) == [g[0] for g in want] and list(perm[8:]) == [g[1] for g in want]


@pytest.mark.parametrize("R_A,C_A", [(2, 1), (2, 2), (4, 1), (1, 2)])
def test_cost_is_the_encoders_union_mask_popcount(R_A, C_A):
    # Reordering the rows of a tile as Alg. 1 says and encoding it must activate exactly F(all rows)
    # union-mask entries (Sec. V-A counts them as P_t), and never more than the given order does.
    rng = np.random.default_rng([R_A, C_A])
    H_L, K_L = 16, 128
    W = rng.integers(-8, 8, (H_L, K_L)).astype(np.int8)
    W[rng.random((H_L, K_L)) < 0.6] = 0
    perm, cost = oracle.reorder_tile(W != 0, R_A, C_A)
    before = oracle.encode(W, H_L, K_L, R_A, C_A)["stats"]["sum_P"]
    after = oracle.encode(W[perm], H_L, K_L, R_A, C_A)["stats"]["sum_P"]
    assert after == cost <= before
    assert oracle.encode(W[perm], H_L, K_L, R_A, C_A)["stats"]["nnz"] == int((W != 0).sum())


def test_degenerate_tiles_and_bad_arguments():
    perm, cost = oracle.reorder_tile(np.zeros((16, 64), np.uint8), 2, 1)
    assert cost == 0 and list(perm) == [0, 2, 4, 6, 8, 10, 12, 14, 1, 3, 5, 7, 9, 11, 13, 15]
    perm, cost = oracle.reorder_tile(np.ones((8, 32), np.uint8), 4, 2)
    assert cost == 2 * 16
    perm, cost = oracle.reorder_tile(np.eye(8, dtype=np.uint8), 8, 1)   # one group holds every row
    assert cost == 8 and list(perm) == list(range(8))
    with pytest.raises(ValueError):
        oracle.reorder_tile(np.zeros((6, 8), np.uint8), 4, 1)
    with pytest.raises(ValueError):
        oracle.reorder_tile(np.zeros((4, 9), np.uint8), 2, 2)
