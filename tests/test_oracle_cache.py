"""Pins for oracle/cache.py: the iterated decode step against definitions that do not use it."""
import numpy as np
import pytest

from oracle import attention as oa
from oracle import eviction as oe
from oracle.cache import CapacityError, HeadCache


def _stream(rng, steps, g, D):
    return (rng.standard_normal((steps, g, D)), rng.standard_normal((steps, D)) * 1.5, rng.standard_normal((steps, D)))


def test_full_budget_reproduces_dense_attention():
    # capacity above everything ever appended: every step equals Eq. 4 over the whole history
    rng = np.random.default_rng(1)
    g, D, T0, steps = 4, 16, 20, 12
    K0, V0 = rng.standard_normal((T0, D)), rng.standard_normal((T0, D))
    q, kn, vn = _stream(rng, steps, g, D)
    c = HeadCache(T0 + steps + 1, D, 4, 1, 2)
    c.load(K0, V0, np.arange(T0), np.zeros(T0))
    Kall, Vall = K0, V0
    for s in range(steps):
        o, lse, ev = c.step(q[s], kn[s], vn[s], T0 + s)
        Kall = np.vstack([Kall, kn[s]]); Vall = np.vstack([Vall, vn[s]])
        ref, _ = oa.decode_attention(q[s], Kall, Vall)
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-14)
        assert ev == -1
    assert c.length == T0 + steps and c.free_slot == c.length


def test_each_step_adds_g_to_the_total_score():
    rng = np.random.default_rng(2)
    g, D, C, steps = 3, 8, 12, 30
    q, kn, vn = _stream(rng, steps, g, D)
    c = HeadCache(C, D, 2, 1, 2)
    evicted_mass = 0.0
    for s in range(steps):
        before = c.score.copy()
        _, _, ev = c.step(q[s], kn[s], vn[s], s)
        if ev >= 0:
            evicted_mass += c.score[ev]
        live = c.valid_slots()
        assert abs(c.score[live].sum() + evicted_mass - g * (s + 1)) < 1e-9
        assert c.length <= C - 1


def test_zero_query_spreads_g_over_n():
    D, g = 8, 4
    rng = np.random.default_rng(3)
    c = HeadCache(64, D, 4, 1, 2)
    c.load(rng.standard_normal((10, D)), rng.standard_normal((10, D)), np.arange(10), np.zeros(10))
    c.step(np.zeros((g, D)), rng.standard_normal(D), rng.standard_normal(D), 10)
    np.testing.assert_allclose(c.score[:11], g / 11.0, rtol=1e-14)


def test_slot_reuse_equals_order_preserving_removal():
    """The same policy written the way Eq. 5-6 print it: rows held in a list, the evicted
    row deleted and the tail shifted.  Outputs and retained sets must agree every step."""
    rng = np.random.default_rng(4)
    g, D, C, steps, n_sink = 2, 8, 16, 60, 2
    q, kn, vn = _stream(rng, steps, g, D)
    c = HeadCache(C, D, n_sink, 1, 2)
    rows = []                                               # (pos, score, k, v)
    for s in range(steps):
        o, _, _ = c.step(q[s], kn[s], vn[s], s)
        rows.append([s, 0.0, kn[s], vn[s]])
        K = np.array([r[2] for r in rows]); V = np.array([r[3] for r in rows])
        ref, p = oa.decode_attention(q[s], K, V)
        for r, inc in zip(rows, p.sum(axis=0)):
            r[1] += inc
        if len(rows) > C - 1:
            keep = oe.select_keep([r[0] for r in rows], [r[1] for r in rows], C - 1, n_sink, 1, 2)
            rows = [rows[i] for i in keep]
        np.testing.assert_allclose(o, ref, rtol=1e-11, atol=1e-13)
        pos, score, _, _ = c.retained()
        assert list(pos) == [r[0] for r in rows]
        np.testing.assert_allclose(score, [r[1] for r in rows], rtol=1e-11)


def test_pure_window_trajectory_closed_form():
    rng = np.random.default_rng(5)
    g, D, C, n_sink = 2, 8, 12, 3
    c = HeadCache(C, D, n_sink, 1, 1)
    for s in range(40):
        c.step(rng.standard_normal((g, D)), rng.standard_normal(D), rng.standard_normal(D), s)
        pos, _, _, _ = c.retained()
        R = C - 1
        expect = list(range(s + 1)) if s + 1 <= R else list(range(n_sink)) + list(range(s + 1 - (R - n_sink), s + 1))
        assert list(pos) == expect


def test_flags_and_capacity():
    rng = np.random.default_rng(6)
    D, g = 4, 2
    c = HeadCache(4, D, 1, 1, 2)
    o, lse, _ = c.step(rng.standard_normal((g, D)), None, None, 0, append=False)
    assert np.all(o == 0) and np.all(np.isneginf(lse))
    for s in range(4):
        c.step(rng.standard_normal((g, D)), rng.standard_normal(D), rng.standard_normal(D), s, evict=False)
    assert c.length == 4
    with pytest.raises(CapacityError):
        c.step(rng.standard_normal((g, D)), rng.standard_normal(D), rng.standard_normal(D), 4)
    s0 = c.score.copy()
    o1, _, _ = c.step(rng.standard_normal((g, D)), None, None, 0, append=False, update_score=False)
    np.testing.assert_array_equal(c.score, s0)


def test_attention_skips_the_free_slot():
    rng = np.random.default_rng(7)
    D, g, C = 8, 2, 6
    c = HeadCache(C, D, 1, 1, 2)
    for s in range(9):
        c.step(rng.standard_normal((g, D)), rng.standard_normal(D), rng.standard_normal(D), s)
    assert c.free_slot < c.length                           # a hole in the middle
    slots = c.valid_slots()
    assert c.free_slot not in slots and len(slots) == C - 1
    q = rng.standard_normal((g, D))
    o, _, _ = c.step(q, None, None, 0, append=False, update_score=False)
    ref, _ = oa.decode_attention(q, c.K[slots], c.V[slots])
    np.testing.assert_allclose(o, ref, rtol=1e-13)
