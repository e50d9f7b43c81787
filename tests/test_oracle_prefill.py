"""Pins for oracle/prefill.py: the prompt's column sums must equal what token-by-token decoding accumulates."""
import numpy as np

from oracle.cache import HeadCache
from oracle.prefill import prefill_scores


def test_total_mass_is_g_times_T():
    rng = np.random.default_rng(1)
    Q, K = rng.standard_normal((3, 20, 8)), rng.standard_normal((20, 8))
    s = prefill_scores(Q, K)
    assert abs(s.sum() - 3 * 20) < 1e-10 and np.all(s > 0)


def test_equals_decoding_the_prompt_one_token_at_a_time():
    # a cache large enough to evict nothing, fed the prompt token by token, accumulates the same scores
    rng = np.random.default_rng(2)
    g, T, D = 2, 15, 8
    Q, K, V = rng.standard_normal((g, T, D)), rng.standard_normal((T, D)), rng.standard_normal((T, D))
    c = HeadCache(T + 2, D, 4, 1, 2)
    for t in range(T):
        c.step(Q[:, t], K[t], V[t], t)
    np.testing.assert_allclose(c.score[:T], prefill_scores(Q, K), rtol=1e-12)


def test_zero_queries_closed_form():
    # uniform attention: token j receives 1/(i+1) from every row i >= j, from each of the g heads
    T, g = 9, 3
    s = prefill_scores(np.zeros((g, T, 4)), np.ones((T, 4)))
    expect = [g * sum(1.0 / (i + 1) for i in range(j, T)) for j in range(T)]
    np.testing.assert_allclose(s, expect, rtol=1e-13)


def test_first_token_of_a_peaked_head_takes_everything():
    T, D = 6, 4
    K = np.zeros((T, D)); K[0, 0] = 1.0
    Q = np.zeros((1, T, D)); Q[0, :, 0] = 1e4
    s = prefill_scores(Q, K)
    np.testing.assert_allclose(s, [T, 0, 0, 0, 0, 0], atol=1e-12)
