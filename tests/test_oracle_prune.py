"""Pins for the pruning oracle: each check is written independently of ``oracle/`` (numpy /
pure Python / by hand) so that a wrong sign, index, group boundary or tie rule fails here."""
import itertools

import numpy as np
import pytest

import oracle


def _rng(seed):
    return np.random.default_rng(seed)


# ---- hand-worked examples (Sec. 3.1: L1 norm of a tile's column, N retained per M) ----------

def test_hand_example_tile2_2of4():
    # one tile of two rows, K = 8, groups {0..3} {4..7}
    w = np.array([[1, -5, 2, 0, 3, 3, -1, 0],
                  [2, 1, -4, 1, 0, 1, 6, -2]], dtype=np.float32)
    # column L1:  3  6  6  1 | 3  4  7  2   -> keep {1,2} and {5,6}
    values, indices = oracle.prune(w, 2, 4, 2)
    assert indices.tolist() == [[1, 2, 5, 6]]
    assert values.tolist() == [[-5, 2, 3, -1], [1, -4, 1, 6]]


def test_hand_example_two_tiles_differ():
    # T = 2 over 4 rows: each tile picks its own columns; all rows of a tile share them
    w = np.array([[9, 0, 0, 1],
                  [9, 0, 1, 0],
                  [0, 7, 1, 0],
                  [0, 7, 0, 2]], dtype=np.float32)
    values, indices = oracle.prune(w, 1, 4, 2)
    assert indices.tolist() == [[0], [1]]
    assert values.tolist() == [[9], [9], [7], [7]]
    # 3:4 (25 % sparsity, Table 1): drop only the weakest column of each tile
    values, indices = oracle.prune(w, 3, 4, 2)
    assert indices.tolist() == [[0, 2, 3], [1, 2, 3]]  # tile 0: col 1 has L1 0; tile 1: col 0 has L1 0


def test_hand_example_ties_keep_lower_column():
    w = np.array([[1, 1, 1, 1, 2, 1, 2, 1]], dtype=np.float32)
    _, indices = oracle.prune(w, 2, 4, 1)
    assert indices.tolist() == [[0, 1, 4, 6]]


def test_hand_example_tail_group_and_tail_tile():
    # K = 6 with M = 4: tail group {4,5} keeps min(N, 2); c_out = 3 with T = 2: tail tile has one row
    w = np.array([[5, 1, 1, 6, 1, 2],
                  [1, 1, 5, 1, 3, 1],
                  [0, 9, 8, 0, 0, 4]], dtype=np.float32)
    values, indices = oracle.prune(w, 3, 4, 2)
    # tile 0 L1: 6 2 6 7 | 4 3 -> drop col 1; tail keeps both.  tile 1: 0 9 8 0 -> tie 0,0: drop col 3
    assert indices.tolist() == [[0, 2, 3, 4, 5], [0, 1, 2, 4, 5]]
    assert values[2].tolist() == [0, 9, 8, 0, 4]
    assert oracle.kept_count(6, 3, 4) == 5
    assert oracle.kept_count(6, 1, 4) == 2
    assert oracle.kept_count(7, 2, 4) == 4


def test_hand_example_non_finite_scores():
    # The paper is silent on non-finite weights.  Reading: a NaN score ranks as +infinity (an
    # infinite score already does), ties by column; a group still keeps exactly N columns.
    nan, inf = float("nan"), float("inf")
    w = np.array([[nan, 3, 2, 1, 1, nan, nan, 5]], dtype=np.float32)
    _, indices = oracle.prune(w, 2, 4, 1)
    assert indices.tolist() == [[0, 1, 5, 6]]          # NaN first or later in the group: kept either way
    w = np.array([[1, 2, nan, 3, 7, -inf, 6, inf]], dtype=np.float32)
    _, indices = oracle.prune(w, 1, 4, 1)
    assert indices.tolist() == [[2, 5]]                # |-inf| = +inf ties with +inf: lower column
    # a NaN in one row of a wider tile poisons that column's L1 sum only
    w = np.array([[1, 9, 1, 1], [1, 1, nan, 1]], dtype=np.float32)
    values, indices = oracle.prune(w, 1, 4, 2)
    assert indices.tolist() == [[2]]
    assert values[0].tolist() == [1.0] and np.isnan(values[1, 0])
    # every (tile, group) still keeps exactly N
    rng = _rng(11)
    w = rng.standard_normal((8, 32)).astype(np.float32)
    w[rng.integers(0, 8, 20), rng.integers(0, 32, 20)] = nan
    _, indices = oracle.prune(w, 2, 4, 4)
    assert indices.shape == (2, 16)
    assert (indices // 4 == np.arange(16) // 2).all()


# ---- sparsity identities printed in the paper ------------------------------------------------

@pytest.mark.parametrize("n,m,sparsity", [(2, 4, 0.5), (3, 4, 0.25), (1, 4, 0.75), (4, 8, 0.5)])
def test_kept_fraction_matches_paper_ratios(n, m, sparsity):
    # Table 1: 3:4 <-> 25 %, 2:4 <-> 50 %, 1:4 <-> 75 %; Sec. 2.1: N=4, M=8 <-> 50 %
    k = 32 * m
    assert oracle.kept_count(k, n, m) == round((1 - sparsity) * k)
    w = _rng(n * 10 + m).standard_normal((16, k)).astype(np.float32)
    values, indices = oracle.prune(w, n, m, 8)
    assert values.shape == (16, k * n // m) and indices.shape == (2, k * n // m)


# ---- T = 1 is conventional row-wise N:M (Sec. 4.5): textbook magnitude rule -------------------

@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (3, 4), (2, 8), (4, 8), (5, 16)])
def test_tile1_equals_textbook_rowwise_nm(n, m):
    w = _rng(100 + n + m).standard_normal((12, 6 * m)).astype(np.float32)
    values, indices = oracle.prune(w, n, m, 1)
    for o in range(w.shape[0]):
        exp = []
        for g0 in range(0, w.shape[1], m):
            mag = np.abs(w[o, g0:g0 + m])
            order = np.argsort(-mag, kind="stable")[:n]  # N largest magnitudes, lower index on ties
            exp += sorted(int(g0 + i) for i in order)
        assert indices[o].tolist() == exp
        assert np.array_equal(values[o], w[o, exp])


# ---- exhaustive subset search on tiny inputs --------------------------------------------------

@pytest.mark.parametrize("seed", range(6))
def test_bruteforce_subset_search(seed):
    r = _rng(200 + seed)
    t = int(r.integers(1, 5))
    m = int(r.integers(2, 7))
    n = int(r.integers(1, m + 1))
    c_out = int(r.integers(1, 9))
    k = m * int(r.integers(1, 4)) + int(r.integers(0, m))  # sometimes a tail group
    # few distinct small integers: exact scores and plenty of ties
    w = r.integers(-2, 3, size=(c_out, k)).astype(np.float32)
    _, indices = oracle.prune(w, n, m, t)
    for tile in range(-(-c_out // t)):
        rows = w[tile * t:(tile + 1) * t]
        exp = []
        for g0 in range(0, k, m):
            cols = list(range(g0, min(g0 + m, k)))
            take = min(n, len(cols))
            best, best_score = None, None
            for sub in itertools.combinations(cols, take):  # lexicographic order
                sc = sum(float(np.abs(rows[:, c]).sum()) for c in sub)
                if best is None or sc > best_score:  # first (lexicographically smallest) maximum
                    best, best_score = sub, sc
            exp += list(best)
        assert indices[tile].tolist() == exp


# ---- invariants -------------------------------------------------------------------------------

@pytest.mark.parametrize("n,m,t,c_out,k", [(2, 4, 8, 32, 144), (1, 4, 32, 64, 256), (2, 8, 64, 128, 192),
                                           (3, 4, 5, 17, 50), (1, 8, 16, 48, 72), (7, 16, 3, 10, 100)])
def test_count_order_range_invariants(n, m, t, c_out, k):
    w = _rng(300 + n + m + t).standard_normal((c_out, k)).astype(np.float32)
    values, indices = oracle.prune(w, n, m, t)
    kk = oracle.kept_count(k, n, m)
    assert indices.shape == (-(-c_out // t), kk) and values.shape == (c_out, kk)
    for row in indices.astype(np.int64):
        assert np.all(np.diff(row) > 0)  # strictly ascending
        counts = np.bincount(row // m, minlength=-(-k // m))
        for g, cnt in enumerate(counts):  # exactly N per full group, min(N, m') in the tail
            assert cnt == min(n, min(m, k - g * m))
    # compressed layout: expansion equals w with the pruned columns zeroed, bit for bit
    dense = oracle.expand(values, indices, k, t)
    mask = np.zeros((c_out, k), dtype=bool)
    for o in range(c_out):
        mask[o, indices[o // t]] = True
    assert np.array_equal(dense.view(np.uint32), np.where(mask, w, np.float32(0)).view(np.uint32))
    # idempotent: pruning the expansion again changes nothing (kept columns still dominate; the
    # zeroed ones score 0 and random kept ones score > 0)
    v2, i2 = oracle.prune(dense, n, m, t)
    assert np.array_equal(i2, indices) and np.array_equal(v2, values)


def test_keep_all_is_identity():
    w = _rng(5).standard_normal((9, 21)).astype(np.float32)
    for m in (1, 3, 4, 21):
        values, indices = oracle.prune(w, m, m, 4)
        assert np.array_equal(indices, np.tile(np.arange(21, dtype=np.uint16), (3, 1)))
        assert np.array_equal(values.view(np.uint32), w.view(np.uint32))


def test_scale_and_row_permutation_invariance():
    r = _rng(6)
    w = r.integers(-8, 9, size=(16, 64)).astype(np.float32)  # exact sums in any order
    _, base = oracle.prune(w, 2, 4, 8)
    _, scaled = oracle.prune(w * np.float32(0.25), 2, 4, 8)
    assert np.array_equal(base, scaled)
    perm = np.concatenate([r.permutation(8), 8 + r.permutation(8)])  # shuffle rows inside each tile
    _, permuted = oracle.prune(w[perm], 2, 4, 8)
    assert np.array_equal(base, permuted)
    # moving a row to another tile may change the result: the kept set belongs to the tile
    w2 = w.copy()
    w2[0], w2[8] = w[8].copy(), w[0].copy()
    _, moved = oracle.prune(w2, 2, 4, 8)
    assert moved.shape == base.shape


def test_ohwi_flattening_of_4d_weights():
    # column k = (kh*Kw + kw)*C_in + c (Fig. 4 caption: kernel layout OHWI)
    w = np.zeros((1, 2, 3, 4), dtype=np.float32)
    w[0, 1, 2, 3] = 5.0   # k = (1*3+2)*4+3 = 23
    w[0, 0, 1, 0] = -7.0  # k = (0*3+1)*4+0 = 4
    values, indices = oracle.prune(w, 1, 4, 1)
    assert indices[0].tolist() == [0, 4, 8, 12, 16, 23]
    assert values[0].tolist() == [0, -7, 0, 0, 0, 5]


def test_rejects_bad_arguments():
    w = np.zeros((4, 8), dtype=np.float32)
    for n, m, t in ((0, 4, 2), (5, 4, 2), (2, 4, 0)):
        with pytest.raises(ValueError):
            oracle.prune(w, n, m, t)
