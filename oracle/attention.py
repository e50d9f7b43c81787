"""Softmax attention in float64 (Eq. 1, Eq. 4, Eq. 7).  Test infrastructure only."""
import numpy as np


def softmax_rows(S):
    """Row-wise softmax of a float64 matrix (the softmax of Eq. 1).

    Rows whose entries are all -inf (fully masked) are not expected here.
    """
    S = np.asarray(S, dtype=np.float64)
    m = S.max(axis=-1, keepdims=True)
    E = np.exp(S - m)
    return E / E.sum(axis=-1, keepdims=True)


def decode_attention(q, K, V):
    """Single-token attention over a cache, Eq. 4 (and Eq. 7 once rows were evicted).

    q : [g, D]  the query vectors of the g query heads that share this KV head
    K : [n, D]  every row currently in the cache, the new token's row included
    V : [n, D]
    Returns (o [g, D], p [g, n]) with p = softmax(q K^T / sqrt(D)) and o = p V.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    D = q.shape[-1]
    S = (q @ K.T) / np.sqrt(float(D))
    P = softmax_rows(S)
    return P @ V, P


def log_sum_exp(q, K):
    """log sum_j exp(q k_j / sqrt(D)) per query head: the log of Eq. 7's normaliser."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    S = (q @ K.T) / np.sqrt(float(q.shape[-1]))
    m = S.max(axis=-1)
    return m + np.log(np.exp(S - m[:, None]).sum(axis=-1))


def causal_attention(Q, K, V):
    """Eq. 1 for a whole prompt with the causal mask a decoder applies.

    Q, K, V : [T, D] of one head.  Row t attends to rows 0..t.
    Returns (O [T, D], A [T, T]).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    T, D = Q.shape
    S = (Q @ K.T) / np.sqrt(float(D))
    future = np.triu(np.ones((T, T), dtype=bool), k=1)
    S = np.where(future, -np.inf, S)
    A = softmax_rows(S)
    return A @ V, A
