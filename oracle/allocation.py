"""Budget reallocation by head importance (Algorithm 2), in whole pages.  Test infrastructure only.

Algorithm 2 moves a reduction r from every KV cache whose importance is below a
threshold t to the most important caches.  It is silent on units, rounding and
bounds; the readings used here (all integer arithmetic on pages):

  * the starting allocation is uniform: total // m pages each, the remainder one
    page each to the first caches in index order;
  * r is a fraction r_num / r_den of the cache's current size, rounded down, and a
    cache never drops below min_pages;
  * the set the freed pages go to is the k = min(n, m - n) caches of highest
    importance among those at or above t (ties: lower index first); each gets
    freed // k, the remainder one page each from the most important down;
  * nothing is moved when no cache or every cache is below t;
  * a cache never exceeds max_pages: what it cannot take is handed on, one page at
    a time in descending importance, to the caches at or above t that still have
    room, and after those to the reduced caches.
"""
import numpy as np

SCOPE_LAYER = 0
SCOPE_MODEL = 1


class AllocationError(ValueError):
    pass


def uniform_pages(total_pages, m):
    base, rem = divmod(int(total_pages), int(m))
    return [base + (1 if i < rem else 0) for i in range(m)]


def _by_importance(indices, I):
    return sorted(indices, key=lambda i: (-I[i], i))


def allocate_group(I, t, r_num, r_den, total_pages, min_pages, max_pages):
    """Algorithm 2 on one group of m caches.  Returns a list of m page counts summing to total_pages."""
    I = [float(x) for x in I]
    m = len(I)
    alloc = uniform_pages(total_pages, m)
    if min(alloc) < min_pages or max(alloc) > max_pages:
        raise AllocationError("uniform share outside [min_pages, max_pages]")

    low = [i for i in range(m) if I[i] < t]
    n = len(low)
    if n == m or n == 0:
        return alloc

    freed = 0
    for i in low:
        d = min((alloc[i] * r_num) // r_den, alloc[i] - min_pages)
        alloc[i] -= d
        freed += d

    k = min(n, m - n)
    high = _by_importance([i for i in range(m) if not I[i] < t], I)
    top = high[:k]
    share, extra = divmod(freed, k)
    for rank, j in enumerate(top):
        alloc[j] += share + (1 if rank < extra else 0)

    excess = 0
    for j in top:
        if alloc[j] > max_pages:
            excess += alloc[j] - max_pages
            alloc[j] = max_pages
    for order in (high, _by_importance(low, I)):
        while excess > 0:
            gave = False
            for j in order:
                if excess == 0:
                    break
                if alloc[j] < max_pages:
                    alloc[j] += 1
                    excess -= 1
                    gave = True
            if not gave:
                break
    if excess > 0:
        raise AllocationError("total does not fit under max_pages")
    return alloc


def allocate(I, t, r_num, r_den, total_pages, min_pages, max_pages, page,
             scope=SCOPE_LAYER, layer_importance=None, t_layer=0.0, rl_num=0, rl_den=1):
    """Per-(layer, KV head) capacities for a whole model.

    I : [L, Hkv] KV-cache importances.  total_pages is the whole model's budget.
    SCOPE_LAYER: the budget is first split over layers (uniformly, or by Algorithm 2
    applied to `layer_importance` with (t_layer, rl_num / rl_den) and bounds scaled by
    Hkv), then Algorithm 2 runs inside each layer.  SCOPE_MODEL: one group of L * Hkv.
    Returns (cap [L, Hkv] tokens, slab_off [L, Hkv] tokens, seq_stride tokens).
    """
    I = np.asarray(I, dtype=np.float64)
    L, Hkv = I.shape
    if scope == SCOPE_MODEL:
        pages = np.array(allocate_group(I.reshape(-1), t, r_num, r_den, total_pages,
                                        min_pages, max_pages), dtype=np.int64).reshape(L, Hkv)
    else:
        if layer_importance is None:
            per_layer = uniform_pages(total_pages, L)
        else:
            per_layer = allocate_group(layer_importance, t_layer, rl_num, rl_den, total_pages,
                                       min_pages * Hkv, max_pages * Hkv)
        pages = np.array([allocate_group(I[l], t, r_num, r_den, per_layer[l], min_pages, max_pages)
                          for l in range(L)], dtype=np.int64)
    cap = pages * int(page)
    flat = cap.reshape(-1)
    off = np.concatenate([[0], np.cumsum(flat)[:-1]]).reshape(L, Hkv)
    return cap.astype(np.int32), off.astype(np.int64), int(flat.sum())
