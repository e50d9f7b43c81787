"""Batches whose sequences are at different positions: baklava_evict_varlen and
baklava_decode_attn_varlen against per-sequence oracle twins (Eq. 4-7 are per sequence, so the
oracle is the same HeadCache driven with each sequence's own position)."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import eviction as oevict
from oracle.cache import HeadCache
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl
from tests.harness import Session, assert_close, f64

pytestmark = pytest.mark.gpu


class VarlenSession(Session):
    """Session whose sequences hold prompts of different lengths and advance independently."""

    def __init__(self, w, prompt_len, **kw):
        super().__init__(w, prefill=False, **kw)
        self.prompt_len = list(prompt_len)
        self.t_seq = list(prompt_len)
        self._prefill_varlen()

    def _prefill_varlen(self):
        w = self.w
        ews = torch.empty((bk.baklava_evict_workspace_size(self.shape, w.B, 1, w.T),), dtype=torch.uint8,
                          device=self.device)
        plen = torch.tensor(self.prompt_len, dtype=torch.int32, device=self.device)
        for l in range(self.lb, self.le):
            k, v = wl.dense_kv_layer(w, l, self.scales, self.device)
            sc = wl.prefill_scores(w, l, self.device)
            bk.baklava_evict_varlen(self.shape, self.cache, l, l + 1, k, v, sc, w.T, plen,
                                    0, w.Hkv * w.T, w.T, 1, ews)
            torch.cuda.synchronize()
        for (b, l, h) in self.heads:
            n = self.prompt_len[b]
            C = int(self.cap[l, h])
            hc = HeadCache(C, w.D, w.n_sink, w.recent_num, w.recent_den)
            if n > 0:
                k, v = wl.dense_kv(w, l, b, h, self.scales)
                sc = wl.prefill_scores(w, l)[b, h]
                K2, V2, pos2, s2, _ = oevict.bulk_evict(f64(k)[:n], f64(v)[:n], np.arange(n), f64(sc)[:n], C - 1,
                                                       w.n_sink, w.recent_num, w.recent_den)
                hc.load(K2, V2, pos2, s2)
            self.twins[(b, l, h)] = hc

    def step_varlen(self, step_index, idle=(), flags=0):
        w = self.w
        q, kn, vn = wl.decode_inputs(w, step_index, self.scales, self.device, layers=(self.lb, self.le))
        t_host = [-1 if b in idle else self.t_seq[b] for b in range(w.B)]
        t_dev = torch.tensor(t_host, dtype=torch.int32, device=self.device)
        self.out.fill_(7.0)                    # idle sequences must leave their rows alone
        self.lse.fill_(7.0)
        before = {b: (self.cache.len[b].clone(), self.cache.free_slot[b].clone()) for b in idle}
        if self.layer_plans is None:
            bk.baklava_decode_attn_varlen(self.shape, self.cache, q, kn, vn, t_dev, self.out, self.lse, flags,
                                          self.plan, self.ws)
        else:                                  # the layer loop of a model, every call after the first overlapping
            torch.cuda.synchronize()
            for i, (plan, ws) in enumerate(self.layer_plans):
                bk.baklava_decode_attn_varlen(self.shape, self.cache, q[i:i + 1], kn[i:i + 1], vn[i:i + 1], t_dev,
                                              self.out[i:i + 1], self.lse[i:i + 1],
                                              flags | (bk.FLAG_OVERLAP_PREV if i > 0 else 0), plan, ws)
        torch.cuda.synchronize()
        qh, knh, vnh = f64(q), f64(kn), f64(vn)
        out, lse = f64(self.out), f64(self.lse)
        g = w.g
        for (b, l, h) in self.heads:
            li = l - self.lb
            tag = "step %d head (b%d,l%d,h%d)" % (step_index, b, l, h)
            if b in idle:
                assert (out[li, b, h * g:(h + 1) * g] == 7.0).all(), tag + " idle out touched"
                assert (lse[li, b, h * g:(h + 1) * g] == 7.0).all(), tag + " idle lse touched"
                self.check_state(b, l, h, tag + " idle")
                continue
            tw = self.twins[(b, l, h)]
            o_ref, lse_ref, _ = tw.step(qh[li, b, h * g:(h + 1) * g], knh[li, b, h], vnh[li, b, h], t_host[b],
                                        append=True, update_score=True, evict=True)
            assert_close(out[li, b, h * g:(h + 1) * g], o_ref, tag + " out")
            assert_close(lse[li, b, h * g:(h + 1) * g], lse_ref, tag + " lse")
            self.check_state(b, l, h, tag)
        for b in idle:
            assert torch.equal(self.cache.len[b], before[b][0]) and torch.equal(self.cache.free_slot[b], before[b][1])
        for b in range(w.B):
            if b not in idle:
                self.t_seq[b] += 1
        assert int(self.cache.status.item()) == 0


def test_bulk_evict_with_prompt_lengths_matches_oracle():
    w = wl.scaled(wl.TINY, B=5)
    s = VarlenSession(w, [512, 300, 37, 0, 255])       # over budget, over, under, empty, about one base budget
    for (b, l, h) in s.heads:
        s.check_state(b, l, h, "after bulk evict")
        st = s.head_state(b, l, h)
        assert st["len"] == min(s.prompt_len[b], int(s.cap[l, h]) - 1)


def test_decode_steps_at_per_sequence_positions():
    w = wl.scaled(wl.TINY, B=4)
    s = VarlenSession(w, [512, 300, 37, 0])
    for i in range(6):
        s.step_varlen(i)
    # positions written are each sequence's own
    for b in range(w.B):
        st = s.head_state(b, 0, 0)
        live = st["pos"][s.valid_slots(st)]
        assert live.max() == s.prompt_len[b] + 5


def test_idle_sequences_are_left_untouched():
    w = wl.scaled(wl.TINY, B=4)
    s = VarlenSession(w, [512, 128, 37, 0])
    s.step_varlen(0, idle=(3,))                         # the empty sequence has not joined yet
    s.step_varlen(1, idle=(1, 3))
    s.step_varlen(2, idle=(0, 1, 2))                    # it joins alone: position 0
    s.step_varlen(3)
    s.step_varlen(4, idle=(0, 1, 2, 3))                 # a step with nobody in it
    st = s.head_state(3, 0, 0)
    assert st["len"] == 2


def test_idle_sequences_in_overlapping_per_layer_calls():
    """Per-layer calls with the overlap flag on a batch where sequences sit steps out: the CTAs of an idle
    sequence have nothing to do but still take part in keeping the stream's order."""
    w = wl.scaled(wl.TINY, B=4, L=4)
    s = VarlenSession(w, [512, 128, 37, 0], per_layer=True)
    s.step_varlen(0, idle=(3,))
    s.step_varlen(1, idle=(1, 3))
    s.step_varlen(2, idle=(0, 1, 2))
    s.step_varlen(3)
    s.step_varlen(4, idle=(0, 1, 2, 3))
    s.step_varlen(5)


def test_short_sequence_grows_into_its_budget_and_starts_evicting():
    w = wl.scaled(wl.TINY, B=2, budget=0.0625, steps=64)     # 32-token base budget
    s = VarlenSession(w, [512, 3])
    C_min = int(s.cap.min())
    for i in range(C_min + 6):                          # the short sequence fills its smallest head and evicts
        s.step_varlen(i)
    l, h = np.unravel_index(int(np.argmin(s.cap)), s.cap.shape)
    st = s.head_state(1, int(l), int(h))
    assert st["len"] == C_min - 1 and st["free"] < C_min


def test_uniform_positions_equal_the_scalar_entry_point():
    w = wl.scaled(wl.TINY, B=2)
    a = Session(w)
    b = VarlenSession(w, [w.T, w.T])
    for i in range(3):
        a.step(i)
        b.step_varlen(i)
    assert torch.equal(a.cache.pos, b.cache.pos) and torch.equal(a.cache.score, b.cache.score)
    assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
    assert torch.equal(a.cache.len, b.cache.len) and torch.equal(a.cache.free_slot, b.cache.free_slot)
    for (bb, l, h) in a.heads:                          # slab rows that hold tokens (the rest is never written)
        sa, sb = a.head_state(bb, l, h), b.head_state(bb, l, h)
        rows = a.valid_slots(sa)
        np.testing.assert_array_equal(sa["K"][rows], sb["K"][rows])
        np.testing.assert_array_equal(sa["V"][rows], sb["V"][rows])


def test_varlen_argument_errors():
    w = wl.scaled(wl.TINY, B=2)
    s = VarlenSession(w, [64, 64])
    q, kn, vn = wl.decode_inputs(w, 0, s.scales, s.device)
    rc = bk.lib().baklava_decode_attn_varlen(
        ctypes.byref(s.shape), ctypes.byref(s.cache.struct), q.data_ptr(), kn.data_ptr(),
        vn.data_ptr(), None, s.out.data_ptr(), None, 0, s.plan.items_dev.data_ptr(),
        ctypes.byref(s.plan.info), s.ws.data_ptr(), s.ws.numel(), None)
    assert rc == -1
    with pytest.raises(bk.BaklavaError):
        bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, -1, s.out, s.lse, 0, s.plan, s.ws)


@pytest.mark.parametrize("seed", range(6))
def test_random_prompt_lengths_and_idle_patterns(seed):
    rng = np.random.default_rng(500 + seed)
    B = int(rng.integers(2, 6))
    w = wl.scaled(wl.TINY, B=B, D=int(rng.choice([64, 128])), budget=float(rng.choice([0.125, 0.25, 0.5])),
                  seed=wl.MASTER_SEED + 200 + seed)
    lens = [int(x) for x in rng.integers(0, w.T + 1, size=B)]
    s = VarlenSession(w, lens, chunk_tokens=int(rng.choice([0, 64, 192])))
    for i in range(6):
        idle = tuple(int(b) for b in range(B) if rng.random() < 0.3)
        s.step_varlen(i, idle=idle)
