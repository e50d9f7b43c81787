"""Pins for oracle/allocation.py (Algorithm 2): hand-worked cases and the invariants the algorithm implies."""
import json
import os

import numpy as np
import pytest

from oracle import allocation as oa

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "allocation_worked.json")


def _cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["note"][:40])
def test_hand_worked_cases(case):
    got = oa.allocate_group(case["I"], case["t"], case["r"][0], case["r"][1], case["total"], case["min"], case["max"])
    assert got == case["pages"]


def _random_groups(seed, count):
    rng = np.random.default_rng(seed)
    for _ in range(count):
        m = int(rng.integers(1, 24))
        I = np.exp(rng.normal(0, 1.2, m))
        base = int(rng.integers(4, 200))
        total = base * m + int(rng.integers(0, m))
        r_den = int(rng.integers(1, 9)); r_num = int(rng.integers(0, r_den + 1))
        mn = int(rng.integers(1, 4)); mx = base + 1 + int(rng.integers(0, 4 * base))
        yield I, float(np.exp(rng.normal(0, 0.7))), r_num, r_den, total, mn, mx


def test_total_is_conserved_and_bounds_hold():
    for I, t, rn, rd, total, mn, mx in _random_groups(1, 400):
        pages = oa.allocate_group(I, t, rn, rd, total, mn, mx)
        assert sum(pages) == total
        assert min(pages) >= mn and max(pages) <= mx


def test_uniform_importance_gives_uniform_budgets():
    for t in (0.5, 1.0, 2.0):
        pages = oa.allocate_group([1.0] * 8, t, 1, 2, 8 * 37, 1, 10_000)
        assert pages == [37] * 8


def test_zero_reduction_changes_nothing():
    for I, t, _, rd, total, mn, mx in _random_groups(2, 50):
        assert oa.allocate_group(I, t, 0, rd, total, mn, mx) == oa.uniform_pages(total, len(I))


def test_all_low_is_unchanged():
    I = [0.1, 0.2, 0.3]
    assert oa.allocate_group(I, 1.0, 1, 2, 31, 1, 100) == [11, 10, 10]


def test_more_important_never_gets_less():
    rng = np.random.default_rng(3)
    for _ in range(200):
        m = int(rng.integers(2, 16))
        I = np.exp(rng.normal(0, 1, m))
        pages = oa.allocate_group(I, 1.0, 1, 2, 64 * m, 1, 150)     # evenly divisible start
        order = np.argsort(I)
        assert all(pages[order[a]] <= pages[order[a + 1]] for a in range(m - 1))


def test_only_caches_below_threshold_shrink_and_only_others_grow():
    for I, t, rn, rd, total, mn, mx in _random_groups(4, 200):
        base = oa.uniform_pages(total, len(I))
        pages = oa.allocate_group(I, t, rn, rd, total, mn, 10 ** 9)    # no upper clipping
        for i in range(len(I)):
            if I[i] < t:
                assert pages[i] <= base[i]
                assert pages[i] >= min(base[i], max(mn, base[i] - (base[i] * rn) // rd))
            else:
                assert pages[i] >= base[i]
        grown = [i for i in range(len(I)) if pages[i] > base[i]]
        n = sum(1 for x in I if x < t)
        assert len(grown) <= min(n, len(I) - n)


def test_infeasible_total_is_an_error():
    with pytest.raises(oa.AllocationError):
        oa.allocate_group([1.0, 2.0], 1.0, 1, 2, 100, 1, 10)


def test_model_level_layout():
    rng = np.random.default_rng(5)
    L, Hkv, page = 3, 4, 16
    I = np.exp(rng.normal(0, 1, (L, Hkv)))
    cap, off, stride = oa.allocate(I, 1.0, 1, 2, L * Hkv * 20, 1, 100, page)
    assert cap.shape == (L, Hkv) and np.all(cap % page == 0)
    assert np.all(cap.reshape(L, -1).sum(axis=1) == Hkv * 20 * page)        # layer scope keeps each layer's total
    flat = cap.reshape(-1)
    np.testing.assert_array_equal(off.reshape(-1), np.concatenate([[0], np.cumsum(flat)[:-1]]))
    assert stride == flat.sum()
    for l in range(L):
        assert list(cap[l] // page) == oa.allocate_group(I[l], 1.0, 1, 2, Hkv * 20, 1, 100)
    capm, _, stridem = oa.allocate(I, 1.0, 1, 2, L * Hkv * 20, 1, 100, page, scope=oa.SCOPE_MODEL)
    assert list(capm.reshape(-1) // page) == oa.allocate_group(I.reshape(-1), 1.0, 1, 2, L * Hkv * 20, 1, 100)
    assert stridem == stride


def test_layer_importance_moves_budget_between_layers():
    I = np.ones((4, 2))
    cap, _, _ = oa.allocate(I, 1.0, 1, 2, 4 * 2 * 10, 1, 100, 16, layer_importance=[0.5, 2.0, 0.2, 3.0],
                            t_layer=1.0, rl_num=1, rl_den=2)
    # layers 0 and 2 give half of their 20 pages to layers 1 and 3; inside a layer importance is flat
    np.testing.assert_array_equal(cap // 16, [[5, 5], [15, 15], [5, 5], [15, 15]])
