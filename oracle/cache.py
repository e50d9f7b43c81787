"""One KV head's fixed-capacity cache and one decode step over it (Eq. 4-7 iterated).

Test infrastructure only.  State of a head with capacity C (tokens):

  K, V   [C, D]   rows;  pos [C] token position of each row;  score [C]
  length          number of valid rows (at most C - 1 between steps)
  free_slot       where the next token's row goes

Between steps the valid rows are the slots {0..length} without free_slot; while
the cache is still filling free_slot == length, so they are simply 0..length-1.
Attention does not depend on row order, so when a row is evicted its slot is
reused by the next token instead of shifting the tail down as Eq. 5-6 print it;
the set of rows is the same.

One step, in this order (budget R = C - 1 rows survive a step, so that with the
incoming token at most C rows are attended to, Eq. 7):
  1. append (k_t, v_t) at free_slot with pos = t and score = 0        (Eq. 4)
  2. p_q = softmax_j(q_q . k_j / sqrt(D)) over every valid row, o_q = sum_j p_qj v_j  (Eq. 7)
  3. score_j += sum over the g query heads of p_qj         (accumulated attention)
  4. keep = select_keep(...) with budget R                   (retention policy)
  5. the one row that is not kept, if any, frees its slot    (Eq. 5-6)
"""
import numpy as np

from .attention import decode_attention, log_sum_exp
from .eviction import select_keep


class CapacityError(RuntimeError):
    pass


class HeadCache:
    def __init__(self, C, D, n_sink, recent_num, recent_den):
        self.C, self.D = int(C), int(D)
        self.n_sink, self.recent_num, self.recent_den = int(n_sink), int(recent_num), int(recent_den)
        self.K = np.zeros((self.C, self.D), dtype=np.float64)
        self.V = np.zeros((self.C, self.D), dtype=np.float64)
        self.pos = np.full(self.C, -1, dtype=np.int64)
        self.score = np.zeros(self.C, dtype=np.float64)
        self.length = 0
        self.free_slot = 0

    def load(self, K, V, pos, score):
        """Fill slots 0..n-1 from already selected rows (the state a bulk eviction leaves)."""
        n = len(pos)
        if n > self.C - 1:
            raise CapacityError("more rows than capacity - 1")
        self.K[:n], self.V[:n] = K, V
        self.pos[:n], self.score[:n] = pos, score
        self.length, self.free_slot = n, n

    def valid_slots(self):
        return np.array([j for j in range(self.length + 1) if j != self.free_slot][: self.length],
                        dtype=np.int64)

    def step(self, q, k_new, v_new, t, append=True, update_score=True, evict=True):
        """One decode step.  q [g, D]; k_new, v_new [D]; t the new token's position.

        Returns (o [g, D], lse [g], evicted_slot or -1).
        """
        if append:
            if self.length >= self.C:
                raise CapacityError("append into a full cache")
            slots = list(self.valid_slots())
            a = self.free_slot
            self.K[a], self.V[a] = k_new, v_new
            self.pos[a], self.score[a] = int(t), 0.0
            slots = np.array(sorted(slots + [a]), dtype=np.int64)
            self.length += 1
        else:
            slots = self.valid_slots()
        n = len(slots)
        if n == 0:
            g = np.asarray(q).shape[0]
            return np.zeros((g, self.D)), np.full(g, -np.inf), -1

        o, p = decode_attention(q, self.K[slots], self.V[slots])
        lse = log_sum_exp(q, self.K[slots])
        if update_score:
            self.score[slots] += p.sum(axis=0)

        evicted = -1
        R = self.C - 1
        if append:
            if evict and n > R:
                keep = select_keep(self.pos[slots], self.score[slots], R,
                                   self.n_sink, self.recent_num, self.recent_den)
                gone = sorted(set(range(n)) - set(int(i) for i in keep))
                assert len(gone) == 1, "a decode step evicts exactly one row"
                evicted = int(slots[gone[0]])
                self.free_slot = evicted
                self.length = n - 1
            else:
                # slots are 0..n-1 here (a hole only exists when the cache is full)
                self.free_slot = n
        return o, lse, evicted

    def retained(self):
        """(pos, score, K, V) of the valid rows sorted by position: the slot-independent state."""
        s = self.valid_slots()
        order = s[np.argsort(self.pos[s], kind="stable")]
        return self.pos[order], self.score[order], self.K[order], self.V[order]
