"""Accumulated attention a prompt leaves on its own tokens (the seed of the heavy-hitter scores).

Test infrastructure only.  The paper cites accumulated attention as the statistic behind heavy-hitter
eviction but does not print a formula; the reading used throughout this repository is that a cached
token's score is the attention probability it has received so far, summed over the query tokens and
over the g query heads that share the KV head.  For a prompt processed in one go that is the column
sum of the causal attention matrix of Eq. 1.
"""
import numpy as np

from .attention import causal_attention


def prefill_scores(Q, K):
    """Q : [g, T, D] query heads of one KV group;  K : [T, D].  Returns score [T] with
    score_j = sum_q sum_{i >= j} softmax_i(Q_q K^T / sqrt(D))[i, j]."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    g, T, D = Q.shape
    score = np.zeros(T, dtype=np.float64)
    for a in range(g):
        _, A = causal_attention(Q[a], K, np.zeros((T, 1)))
        score += A.sum(axis=0)
    return score
