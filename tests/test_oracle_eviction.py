"""Pins for oracle/eviction.py: brute force on tiny heads, closed forms, invariants (Eq. 5-6 + policy)."""
import itertools

import numpy as np
import pytest

from oracle import eviction as oe


def _brute_force_keep(pos, score, R, n_sink, num, den):
    """Every subset of size R that holds all sinks and the recent window; the best one is the
    subset whose remaining members, ranked by (score desc, pos asc), come first lexicographically."""
    n = len(pos)
    W = ((R - n_sink) * num) // den
    t_max = max(pos)
    forced = {j for j in range(n) if pos[j] < n_sink or pos[j] > t_max - W}
    free = [j for j in range(n) if j not in forced]
    best, best_key = None, None
    for extra in itertools.combinations(free, R - len(forced)):
        key = sorted((-score[j], pos[j]) for j in extra)
        if best_key is None or key < best_key:
            best, best_key = extra, key
    return sorted(forced | set(best))


@pytest.mark.parametrize("seed", range(30))
def test_brute_force_on_tiny_heads(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(6, 13))
    n_sink = int(rng.integers(0, 4))
    R = int(rng.integers(n_sink + 1, n))
    den = int(rng.integers(1, 5)); num = int(rng.integers(0, den + 1))
    pos = rng.permutation(np.arange(n) + (0 if seed % 2 else 3))          # odd seeds keep the sink positions
    score = rng.integers(0, 4, n).astype(np.float64) / 4.0                 # many ties
    got = oe.select_keep(pos, score, R, n_sink, num, den)
    assert list(got) == _brute_force_keep(list(pos), list(score), R, n_sink, num, den)


def test_keeps_everything_when_it_fits():
    pos = np.array([5, 1, 9]); score = np.array([0.1, 0.2, 0.3])
    np.testing.assert_array_equal(oe.select_keep(pos, score, 3, 4, 1, 2), [0, 1, 2])
    np.testing.assert_array_equal(oe.select_keep(pos, score, 7, 4, 1, 2), [0, 1, 2])


def test_pure_window_policy_closed_form():
    # recent fraction 1: what stays is {0..n_sink-1} u {t-W+1..t} whatever the scores say
    n, n_sink = 40, 4
    for R in (10, 25, 39):
        rng = np.random.default_rng(R)
        pos = np.arange(n); score = rng.random(n)
        keep = oe.select_keep(pos, score, R, n_sink, 1, 1)
        W = R - n_sink
        assert list(pos[keep]) == list(range(n_sink)) + list(range(n - W, n))


def test_plain_top_k_against_a_full_sort():
    rng = np.random.default_rng(7)
    n, R = 200, 60
    pos = rng.permutation(n) + 1000
    score = np.round(rng.random(n), 1)                                    # ties
    keep = oe.select_keep(pos, score, R, 0, 0, 1)                         # no sinks, no window
    order = np.lexsort((pos, -score))                                     # primary: score desc, then pos asc
    assert sorted(order[:R]) == list(keep)


def test_steady_state_evicts_lowest_score_and_on_ties_the_later_token():
    n_sink, R = 2, 9                                                      # W = floor(7/2) = 3
    pos = np.arange(10)
    score = np.array([0.0, 0.0, 0.5, 0.2, 0.9, 0.2, 0.7, 0.0, 0.0, 0.0])
    keep = oe.select_keep(pos, score, R, n_sink, 1, 2)
    # candidates are positions 2..6 (7, 8, 9 are recent, 0 and 1 sinks); lowest score 0.2 at 3 and 5: 5 goes
    assert sorted(set(range(10)) - set(keep)) == [5]


def test_structure_invariants():
    rng = np.random.default_rng(11)
    for _ in range(200):
        n = int(rng.integers(20, 120)); n_sink = 4
        R = int(rng.integers(n_sink + 2, n))
        num, den = int(rng.integers(0, 4)), 3
        pos = np.sort(rng.choice(500, n, replace=False)); pos[:n_sink] = np.arange(n_sink)
        pos = rng.permutation(pos)
        score = rng.random(n).astype(np.float32)
        keep = oe.select_keep(pos, score, R, n_sink, num, den)
        assert len(keep) == R and len(set(keep)) == R
        kept_pos = set(pos[keep])
        assert all(p in kept_pos for p in range(n_sink))
        W = oe.recent_window(R, n_sink, num, den)
        assert all(p in kept_pos for p in pos if p > pos.max() - W)
        # nobody outside beats anybody inside among the free candidates
        free_in = [j for j in keep if pos[j] >= n_sink and pos[j] <= pos.max() - W]
        free_out = [j for j in range(n) if j not in set(keep)]
        if free_in and free_out:
            worst_in = max((-score[j], pos[j]) for j in free_in)
            best_out = min((-score[j], pos[j]) for j in free_out)
            assert worst_in < best_out


def test_bulk_evict_compacts_in_position_order():
    rng = np.random.default_rng(12)
    T, D, R = 64, 8, 20
    K = rng.standard_normal((T, D)); V = rng.standard_normal((T, D))
    pos = np.arange(T); score = rng.random(T)
    K2, V2, pos2, score2, idx = oe.bulk_evict(K, V, pos, score, R, 4, 1, 2)
    assert len(pos2) == R and np.all(np.diff(pos2) > 0)
    np.testing.assert_array_equal(K2, K[pos2]); np.testing.assert_array_equal(V2, V[pos2])
    np.testing.assert_array_equal(score2, score[pos2])
    np.testing.assert_array_equal(idx, oe.select_keep(pos, score, R, 4, 1, 2))
    # removing rows one at a time as Eq. 5-6 print it leaves the same sequence
    rows = list(range(T))
    for m in sorted(set(range(T)) - set(idx), reverse=True):
        del rows[m]
    assert rows == list(idx)


def test_compaction_in_place_is_eq_5_6_one_row_at_a_time():
    """Rows in arbitrary (slot) order: taking the losers out one by one, each time closing the gap as
    Eq. 5-6 print it, leaves the survivors in their original relative order; for rows already in
    position order it coincides with bulk_evict."""
    rng = np.random.default_rng(13)
    for trial in range(20):
        n, D = int(rng.integers(10, 60)), 4
        R = int(rng.integers(7, n + 3))                                   # sometimes nothing has to go
        K = rng.standard_normal((n, D)); V = rng.standard_normal((n, D))
        pos = rng.permutation(n + 5)[:n]; score = np.round(rng.random(n), 1)
        K2, V2, pos2, score2, idx = oe.compact_in_place(K, V, pos, score, R, 2, 1, 3)
        keep = set(int(i) for i in oe.select_keep(pos, score, R, 2, 1, 3))
        Kl, Vl, pl, sl = [list(x) for x in (K, V, pos, score)]
        alive = list(range(n))
        while True:
            losers = [m for m, j in enumerate(alive) if j not in keep]
            if not losers:
                break
            m = losers[0]                                                 # Eq. 5-6: [x_1..x_{m-1}, x_{m+1}..x_n]
            for lst in (Kl, Vl, pl, sl, alive):
                del lst[m]
        assert alive == list(idx)
        np.testing.assert_array_equal(np.array(Kl), K2); np.testing.assert_array_equal(np.array(Vl), V2)
        np.testing.assert_array_equal(np.array(pl), pos2); np.testing.assert_array_equal(np.array(sl), score2)
    T = 50
    K = rng.standard_normal((T, 4)); V = rng.standard_normal((T, 4)); score = rng.random(T)
    a = oe.compact_in_place(K, V, np.arange(T), score, 17, 4, 1, 2)
    b = oe.bulk_evict(K, V, np.arange(T), score, 17, 4, 1, 2)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
