"""Pins for oracle/attention.py: library routines, closed forms, invariants (Eq. 1, 4, 7)."""
import numpy as np
import pytest
import scipy.special
import torch
import torch.nn.functional as F

from oracle import attention as oa


def _rand(rng, *shape):
    return rng.standard_normal(shape)


@pytest.mark.parametrize("g,n,D", [(1, 1, 8), (4, 37, 64), (7, 130, 128)])
def test_decode_matches_library_sdpa(g, n, D):
    rng = np.random.default_rng(10 + n)
    q, K, V = _rand(rng, g, D), _rand(rng, n, D) * 1.7, _rand(rng, n, D)
    o, p = oa.decode_attention(q, K, V)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q)[None], torch.from_numpy(K)[None],
                                         torch.from_numpy(V)[None])[0].numpy()
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-13)
    assert p.shape == (g, n)


def test_decode_probabilities_match_scipy_softmax_and_scale():
    # the 1/sqrt(D) scale and the (q, k) orientation: logits recomputed row by row with math only
    rng = np.random.default_rng(3)
    q, K, V = _rand(rng, 2, 16), _rand(rng, 9, 16), _rand(rng, 9, 16)
    _, p = oa.decode_attention(q, K, V)
    logits = np.array([[sum(q[a, d] * K[j, d] for d in range(16)) / 4.0 for j in range(9)] for a in range(2)])
    np.testing.assert_allclose(p, scipy.special.softmax(logits, axis=1), rtol=1e-12)
    np.testing.assert_allclose(oa.log_sum_exp(q, K), scipy.special.logsumexp(logits, axis=1), rtol=1e-13)


def test_zero_query_gives_mean_of_values():
    rng = np.random.default_rng(4)
    K, V = _rand(rng, 23, 32), _rand(rng, 23, 32)
    o, p = oa.decode_attention(np.zeros((3, 32)), K, V)
    np.testing.assert_allclose(p, 1.0 / 23, rtol=1e-14)
    np.testing.assert_allclose(o, np.tile(V.mean(axis=0), (3, 1)), rtol=1e-12, atol=1e-14)


def test_single_row_returns_that_value():
    rng = np.random.default_rng(5)
    K, V = _rand(rng, 1, 8), _rand(rng, 1, 8)
    o, p = oa.decode_attention(_rand(rng, 4, 8), K, V)
    np.testing.assert_array_equal(p, np.ones((4, 1)))
    np.testing.assert_allclose(o, np.tile(V, (4, 1)), rtol=1e-15)


def test_row_order_does_not_matter():
    rng = np.random.default_rng(6)
    q, K, V = _rand(rng, 4, 64), _rand(rng, 50, 64), _rand(rng, 50, 64)
    perm = rng.permutation(50)
    o1, p1 = oa.decode_attention(q, K, V)
    o2, p2 = oa.decode_attention(q, K[perm], V[perm])
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(p1[:, perm], p2, rtol=1e-12)


def test_one_dominant_key_selects_its_value():
    # a key aligned with q and scaled up takes all the mass: o -> its v (sign and K/V pairing)
    D = 16
    q = np.zeros((1, D)); q[0, 0] = 1.0
    K = np.zeros((3, D)); K[1, 0] = 4000.0; K[2, 0] = -4000.0
    V = np.arange(3 * D, dtype=np.float64).reshape(3, D)
    o, p = oa.decode_attention(q, K, V)
    np.testing.assert_allclose(p[0], [0.0, 1.0, 0.0], atol=1e-300)
    np.testing.assert_allclose(o[0], V[1])


@pytest.mark.parametrize("T,D", [(1, 8), (5, 16), (33, 64)])
def test_causal_matches_library_sdpa(T, D):
    rng = np.random.default_rng(20 + T)
    Q, K, V = _rand(rng, T, D), _rand(rng, T, D), _rand(rng, T, D)
    O, A = oa.causal_attention(Q, K, V)
    ref = F.scaled_dot_product_attention(torch.from_numpy(Q)[None], torch.from_numpy(K)[None],
                                         torch.from_numpy(V)[None], is_causal=True)[0].numpy()
    np.testing.assert_allclose(O, ref, rtol=1e-12, atol=1e-13)
    assert np.all(np.triu(A, k=1) == 0.0)
    np.testing.assert_allclose(A.sum(axis=1), 1.0, rtol=1e-13)


def test_last_causal_row_is_the_decode_step():
    # Eq. 4: the cached single-token form equals the last row of Eq. 1 over the whole sequence
    rng = np.random.default_rng(8)
    Q, K, V = _rand(rng, 12, 32), _rand(rng, 12, 32), _rand(rng, 12, 32)
    O, _ = oa.causal_attention(Q, K, V)
    o, _ = oa.decode_attention(Q[-1:], K, V)
    np.testing.assert_allclose(o[0], O[-1], rtol=1e-12, atol=1e-14)
