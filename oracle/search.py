"""Algorithm 3 (parameter search) with an attention-output loss in place of perplexity.

Test infrastructure only.  The paper scores a parameter pair (t, r) by the perplexity of a real
model on held-out chunks; without a model the stand-in used here is how far the budgeted cache
moves the attention output away from the dense cache's, per query head and decode step:

    loss = mean over rows i of  ||o_i - ref_i||^2 / max(||ref_i||^2, tiny)

(rows = every (step, layer, sequence, query head) output vector).  The outer loop is the paper's:
every configuration is evaluated on every chunk from a freshly made cache, the chunk losses are
averaged, and the first configuration with the strictly smallest average wins.
"""
import numpy as np

TINY = 1e-30


def output_error(out, ref):
    """Mean relative squared error of the rows of `out` [n, D] against `ref` [n, D] (float64)."""
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    num = ((out - ref) ** 2).sum(axis=1)
    den = np.maximum((ref ** 2).sum(axis=1), TINY)
    return float((num / den).mean()) if len(num) else 0.0


def pick_best(avg_losses):
    """Index of the configuration Algorithm 3 returns: the first strictly smallest average loss.
    A NaN never compares smaller, so it never wins; -1 if nothing beats +inf."""
    best, min_loss = -1, np.inf
    for i, x in enumerate(avg_losses):
        if x < min_loss:
            best, min_loss = i, x
    return best


def parameter_search(configs, chunks, make_cache, evaluate):
    """Algorithm 3.  `make_cache(params)` builds a cache for a configuration, `evaluate(cache, chunk)`
    returns that chunk's loss starting from the freshly made (or reset) cache.
    Returns (best params or None, list of average losses)."""
    averages = []
    for params in configs:
        cache = make_cache(params)
        losses = [evaluate(cache, chunk) for chunk in chunks]
        averages.append(sum(losses) / len(losses))
    best = pick_best(averages)
    return (configs[best] if best >= 0 else None), averages
