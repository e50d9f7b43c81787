"""Which cache entries survive (Eq. 5-6 and the retention policy).  Test infrastructure only.

The paper evaluates a sink + recent-window policy and names accumulated-attention
heavy hitters as another usable policy; it defines neither in formulas.  The
reading used here, for a cache holding n entries that may keep R of them:

  * sinks   S   = entries whose token position is below n_sink;
  * recent  Rec = non-sink entries whose position lies in the last W positions,
                  pos > t_max - W, with t_max the largest position present and
                  W = floor((R - n_sink) * recent_num / recent_den);
  * heavy   HH  = the R - |S| - |Rec| remaining entries that come first when the
                  rest is ordered by (score descending, position ascending);
  * keep = S u Rec u HH; everything is kept when n <= R.

recent_num == recent_den gives the pure sink + window policy.  Removing an
entry is Eq. 5-6: the row leaves K and V together.
"""
import numpy as np


def recent_window(R, n_sink, recent_num, recent_den):
    return max(0, ((int(R) - int(n_sink)) * int(recent_num)) // int(recent_den))


def select_keep(pos, score, R, n_sink, recent_num, recent_den):
    """Indices (into pos/score) of the entries that stay, ascending by index.

    pos   : [n] distinct token positions
    score : [n] accumulated attention, compared exactly as given (no rounding)
    """
    pos = np.asarray(pos, dtype=np.int64)
    score = np.asarray(score)
    n = pos.shape[0]
    if n <= R:
        return np.arange(n, dtype=np.int64)
    W = recent_window(R, n_sink, recent_num, recent_den)
    t_max = int(pos.max())
    is_sink = pos < n_sink
    is_recent = (~is_sink) & (pos > t_max - W)
    rest = [int(j) for j in range(n) if not is_sink[j] and not is_recent[j]]
    n_hh = int(R) - int(is_sink.sum()) - int(is_recent.sum())
    if n_hh < 0:
        raise ValueError("sinks and recent window alone exceed the budget")
    rest.sort(key=lambda j: (-float(score[j]), int(pos[j])))
    keep = [int(j) for j in range(n) if is_sink[j] or is_recent[j]] + rest[:n_hh]
    return np.array(sorted(keep), dtype=np.int64)


def bulk_evict(K, V, pos, score, R, n_sink, recent_num, recent_den):
    """Cut a dense head down to at most R rows and compact it (Eq. 5-6 applied repeatedly).

    Kept rows come out in ascending position, which for a dense prefix is the
    order Eq. 5-6 leave them in.  Returns (K', V', pos', score', kept_index).
    """
    keep = select_keep(pos, score, R, n_sink, recent_num, recent_den)
    order = keep[np.argsort(np.asarray(pos)[keep], kind="stable")]
    return (np.asarray(K)[order], np.asarray(V)[order], np.asarray(pos)[order],
            np.asarray(score)[order], order)


def compact_in_place(K, V, pos, score, R, n_sink, recent_num, recent_den):
    """The same cut applied to a cache as it stands: Eq. 5-6 take rows out and leave the others in
    the order they had, whatever that order is.  Returns (K', V', pos', score', kept_index) with
    kept_index ascending."""
    keep = select_keep(pos, score, R, n_sink, recent_num, recent_den)
    return (np.asarray(K)[keep], np.asarray(V)[keep], np.asarray(pos)[keep], np.asarray(score)[keep], keep)

