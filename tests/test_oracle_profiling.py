"""Pins for oracle/profiling.py (Algorithm 1): closed forms the paper states and small worked cases."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import profiling as op


def test_identical_value_rows_give_similarity_one():
    rng = np.random.default_rng(1)
    T, D = 17, 16
    V = np.tile(rng.standard_normal((1, D)), (T, 1))
    s, c = op.head_similarity(rng.standard_normal((T, D)), rng.standard_normal((T, D)), V)
    np.testing.assert_allclose(c, 1.0, rtol=1e-12)
    assert abs(s - 1.0) < 1e-12


def test_identity_attention_gives_importance_zero():
    # the paper: the cosine reaches its maximum when the attention matrix is the identity
    T, D = 8, 8
    K = np.eye(T, D)
    Q = 1e4 * np.eye(T, D)
    V = np.random.default_rng(2).standard_normal((T, D))
    s, _ = op.head_similarity(Q, K, V)
    assert abs(s - 1.0) < 1e-12
    I = op.kv_importance(np.full((1, 1, 2), s), g=2)
    np.testing.assert_allclose(I, 0.0, atol=1e-12)


def test_single_token_prompt():
    rng = np.random.default_rng(3)
    s, c = op.head_similarity(rng.standard_normal((1, 4)), rng.standard_normal((1, 4)), rng.standard_normal((1, 4)))
    assert c.shape == (1,) and abs(s - 1.0) < 1e-12


def test_uniform_attention_worked_example():
    # zero queries: row t averages V_0..V_t.  V_0=(1,0), V_1=(0,1): cosines 1 and 1/sqrt(2).
    V = np.array([[1.0, 0.0], [0.0, 1.0]])
    s, c = op.head_similarity(np.zeros((2, 2)), np.ones((2, 2)), V)
    np.testing.assert_allclose(c, [1.0, 1.0 / math.sqrt(2.0)], rtol=1e-14)
    assert abs(s - (1.0 + 1.0 / math.sqrt(2.0)) / 2.0) < 1e-14


def test_output_opposite_to_input_gives_minus_one():
    # token 1 looks only at token 0 whose value points the other way: cos = -1; mean similarity 0
    V = np.array([[2.0, 0.0, 0.0], [-1e-6, 0.0, 0.0]])
    K = np.array([[1.0, 0.0, 0.0], [0.0, 0.0, 0.0]])
    Q = np.array([[0.0, 0.0, 0.0], [1e5, 0.0, 0.0]])
    s, c = op.head_similarity(Q, K, V)
    np.testing.assert_allclose(c, [1.0, -1.0], rtol=1e-9)
    assert abs(s) < 1e-9
    # similarity 0 normalises to 1/2, importance 1/2; similarity -1 would give importance 1
    np.testing.assert_allclose(op.kv_importance(np.array([[[s]]]), 1), [[0.5]], atol=1e-9)
    np.testing.assert_allclose(op.kv_importance(np.array([[[-1.0]]]), 1), [[1.0]])


def test_zero_value_row_does_not_divide_by_zero():
    V = np.zeros((3, 4)); V[1] = 1.0
    s, c = op.head_similarity(np.zeros((3, 4)), np.zeros((3, 4)), V)
    assert np.all(np.isfinite(c)) and c[0] == 0.0


def test_length_restricts_the_prompt():
    rng = np.random.default_rng(4)
    Q, K, V = (rng.standard_normal((9, 8)) for _ in range(3))
    s_full, c_full = op.head_similarity(Q, K, V)
    s5, c5 = op.head_similarity(Q, K, V, length=5)
    np.testing.assert_allclose(c5, c_full[:5], rtol=1e-12)   # causal: later tokens cannot change earlier rows
    assert abs(s5 - c_full[:5].mean()) < 1e-13


def test_profile_heads_group_mapping_and_library_attention():
    # query head h reads KV head h // g; outputs recomputed with the library's causal SDPA
    rng = np.random.default_rng(5)
    P, Hq, Hkv, T, D = 2, 4, 2, 11, 8
    Q = rng.standard_normal((P, Hq, T, D)); K = rng.standard_normal((P, Hkv, T, D)); V = rng.standard_normal((P, Hkv, T, D))
    s = op.profile_heads(Q, K, V)
    tQ, tK, tV = (torch.from_numpy(x) for x in (Q, K, V))
    O = F.scaled_dot_product_attention(tQ, tK.repeat_interleave(2, dim=1), tV.repeat_interleave(2, dim=1), is_causal=True)
    ref = F.cosine_similarity(O, tV.repeat_interleave(2, dim=1), dim=-1).mean(dim=-1).numpy()
    np.testing.assert_allclose(s, ref, rtol=1e-11)


def test_kv_importance_worked_example():
    # two prompts, one layer, four heads, groups of two
    s = np.array([[[1.0, 1.0, -1.0, -1.0]], [[1.0, 0.0, -1.0, 0.0]]])
    # prompt mean: [1, .5, -1, -.5] -> normalised [1, .75, 0, .25] -> group means [.875, .125]
    np.testing.assert_allclose(op.kv_importance(s, 2), [[0.125, 0.875]], rtol=1e-15)
    # g = 1: no grouping; g = 4: a single cache
    np.testing.assert_allclose(op.kv_importance(s, 1), [[0.0, 0.25, 1.0, 0.75]], rtol=1e-15)
    np.testing.assert_allclose(op.kv_importance(s, 4), [[0.5]], rtol=1e-15)


def test_importance_is_monotone_decreasing_in_similarity():
    s = np.linspace(-1, 1, 9).reshape(1, 1, 9)
    I = op.kv_importance(s, 1)[0]
    assert np.all(np.diff(I) < 0) and I[0] == 1.0 and I[-1] == 0.0
