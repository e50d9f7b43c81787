"""Head similarity and KV-cache importance (Algorithm 1).  Test infrastructure only."""
import numpy as np

from .attention import causal_attention

COS_EPS = 1e-12


def token_cosines(V, O):
    """Per-token cosine between a head's input V_t and its output O_t (Algorithm 1, step 1).

    V, O : [T, D].  A zero-norm row gives 0 (the denominator is floored at COS_EPS).
    """
    V = np.asarray(V, dtype=np.float64)
    O = np.asarray(O, dtype=np.float64)
    num = (V * O).sum(axis=-1)
    den = np.sqrt((V * V).sum(axis=-1)) * np.sqrt((O * O).sum(axis=-1))
    return num / np.maximum(den, COS_EPS)


def head_similarity(Q, K, V, length=None):
    """Mean over tokens of cos(V_t, (softmax(Q K^T / sqrt(D)) V)_t) for one head and one prompt.

    Algorithm 1, step 1.  The head output is the model's own: scaled logits and a
    causal mask (the algorithm's line omits both; Eq. 1 and "run inference" fix them).
    `length` restricts the prompt to its first `length` tokens.
    Returns (s, c) with c the per-token cosines.
    """
    if length is not None:
        Q, K, V = Q[:length], K[:length], V[:length]
    O, _ = causal_attention(Q, K, V)
    c = token_cosines(V, O)
    return float(c.mean()), c


def profile_heads(Q, K, V, lengths=None):
    """Algorithm 1, step 1 over prompts and heads of one layer.

    Q : [P, Hq, T, D];  K, V : [P, Hkv, T, D].  Query head h reads KV head h // g.
    Returns s [P, Hq].
    """
    P, Hq = Q.shape[0], Q.shape[1]
    Hkv = K.shape[1]
    g = Hq // Hkv
    s = np.zeros((P, Hq), dtype=np.float64)
    for p in range(P):
        n = None if lengths is None else int(lengths[p])
        for h in range(Hq):
            s[p, h], _ = head_similarity(Q[p, h], K[p, h // g], V[p, h // g], n)
    return s


def kv_importance(s, g):
    """Algorithm 1, step 2, with the normalisation of the head-importance paragraph.

    s : [P, L, Hq] per-prompt head similarities in [-1, 1].
    Prompts are reduced by an unweighted mean; the cosine range [-1, 1] is mapped
    affinely onto [0, 1] so that 1 still means "output identical to input"; each
    run of g consecutive heads (one KV cache) is averaged; importance is the
    complement.  Returns I [L, Hq // g].
    """
    s = np.asarray(s, dtype=np.float64)
    P, L, Hq = s.shape
    s_bar = s.mean(axis=0)                       # [L, Hq]
    s_hat = (s_bar + 1.0) / 2.0
    kv_sim = s_hat.reshape(L, Hq // g, g).mean(axis=-1)
    return 1.0 - kv_sim
