"""Shared set-up for the GPU parity tests: builds the same budgeted cache through the CUDA library
(on the device) and through the oracle (on the host) from the same seeded inputs.

Nothing computed by the library ever feeds the oracle here, except where a test says so
explicitly (selection re-checked on the library's own score array)."""
import numpy as np
import torch

from oracle import allocation as oalloc
from oracle import eviction as oevict
from oracle import fp8 as ofp8
from oracle.cache import HeadCache
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl

ABS_TOL = 1e-2
REL_TOL = 1e-2


def assert_close(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        err = np.where(got == ref, 0.0, np.abs(got - ref))
    bad = err > ABS_TOL + REL_TOL * np.abs(ref)
    assert not bad.any(), "%s: max abs err %.3e, %d of %d outside |d| <= 1e-2 + 1e-2 |ref|" % (
        what, err.max(), int(bad.sum()), bad.size)


def shape_of(w):
    return bk.make_shape(w.L, w.Hq, w.Hkv, w.D, w.page, w.n_sink, w.recent_num, w.recent_den)


def f64(t):
    return t.detach().to("cpu", torch.float64).numpy()


class Session:
    """One workload on the device (library) with oracle twins for the heads in `heads`."""

    def __init__(self, w, heads=None, chunk_tokens=0, layers=None, prefill=True, device="cuda", caps=None,
                 kv_dtype=bk.KV_BF16, per_layer=False):
        """`per_layer`: every step is issued as one call per layer, each with its own plan and workspace and, from
        the second layer on, BAKLAVA_FLAG_OVERLAP_PREV (the form a model's layer loop uses)."""
        self.w, self.device = w, device
        self.kv_dtype = kv_dtype
        self.shape = shape_of(w)
        self.scales = wl.kv_scales(w)
        self.imp = wl.importance(w).numpy()
        if caps is None:
            self.cap, self.off, self.stride = bk.baklava_allocate(
                self.shape, self.imp, w.t, w.r_num, w.r_den, w.total_pages * w.page,
                w.min_pages * w.page, w.max_pages * w.page)
            ocap, ooff, ostride = oalloc.allocate(self.imp, w.t, w.r_num, w.r_den, w.total_pages, w.min_pages,
                                                  w.max_pages, w.page)
            np.testing.assert_array_equal(self.cap, ocap)
            np.testing.assert_array_equal(self.off, ooff)
            assert self.stride == ostride
        else:                                   # capacities given directly (whole pages)
            self.cap = np.asarray(caps, dtype=np.int32).reshape(w.L, w.Hkv)
            flat = self.cap.reshape(-1).astype(np.int64)
            self.off = np.concatenate([[0], np.cumsum(flat)[:-1]]).reshape(w.L, w.Hkv)
            self.stride = int(flat.sum())
        self.fp8_scales = wl.kv_fp8_scales(w, self.scales) if kv_dtype == bk.KV_FP8_E4M3 else None
        self.cache = bk.Cache(self.shape, self.cap, self.off, self.stride, w.B, device, kv_dtype=kv_dtype,
                              kv_scale=self.fp8_scales)
        self.lb, self.le = (0, w.L) if layers is None else layers
        self.plan = bk.baklava_decode_plan(self.shape, self.cap, w.B, self.lb, self.le, self.stride,
                                           chunk_tokens=chunk_tokens,
                                           n_sm=torch.cuda.get_device_properties(0).multi_processor_count, kv_dtype=kv_dtype).to(device)
        self.ws = bk.decode_workspace(self.plan, device)
        self.layer_plans = None
        if per_layer:
            self.layer_plans = []
            for l in range(self.lb, self.le):
                plan = bk.baklava_decode_plan(self.shape, self.cap, w.B, l, l + 1, self.stride, chunk_tokens=chunk_tokens,
                                              n_sm=torch.cuda.get_device_properties(0).multi_processor_count, kv_dtype=kv_dtype).to(device)
                self.layer_plans.append((plan, bk.decode_workspace(plan, device)))
        nl = self.le - self.lb
        self.out = torch.zeros((nl, w.B, w.Hq, w.D), dtype=torch.bfloat16, device=device)
        self.lse = torch.zeros((nl, w.B, w.Hq), dtype=torch.float32, device=device)
        self.heads = heads if heads is not None else [(b, l, h) for b in range(w.B)
                                                      for l in range(self.lb, self.le) for h in range(w.Hkv)]
        self.twins = {}
        self.near_ties = []                     # (where, oracle gap) of every victim settled as a near tie
        self.held_rows = {}                     # teacher-forced heads: K, V rows carried on the host
        self.t = w.T if prefill else 0
        if prefill:
            self._prefill()
        else:
            for (b, l, h) in self.heads:
                self.twins[(b, l, h)] = HeadCache(int(self.cap[l, h]), w.D, w.n_sink, w.recent_num, w.recent_den)

    def as_stored(self, rows, l, h, which):
        """The values the cache holds for `rows` (float64) of head (l, h): themselves, or their FP8 round trip.
        which: 0 = K, 1 = V."""
        if self.kv_dtype != bk.KV_FP8_E4M3:
            return rows
        four = self.cache.kv_scale_host[l, h]
        return ofp8.quantise_rows(rows, four[2 * which], four[2 * which + 1])[1]

    def _prefill(self):
        w = self.w
        ews = torch.empty((bk.baklava_evict_workspace_size(self.shape, w.B, 1, w.T),), dtype=torch.uint8,
                          device=self.device)
        for l in range(self.lb, self.le):
            k, v = wl.dense_kv_layer(w, l, self.scales, self.device)
            sc = wl.prefill_scores(w, l, self.device)
            bk.baklava_evict(self.shape, self.cache, l, l + 1, k, v, sc, w.T,
                             0, w.Hkv * w.T, w.T, 1, ews)
            torch.cuda.synchronize()
        for (b, l, h) in self.heads:
            k, v = wl.dense_kv(w, l, b, h, self.scales)
            sc = wl.prefill_scores(w, l)[b, h]
            C = int(self.cap[l, h])
            K2, V2, pos2, s2, _ = oevict.bulk_evict(self.as_stored(f64(k), l, h, 0), self.as_stored(f64(v), l, h, 1),
                                                   np.arange(w.T), f64(sc), C - 1,
                                                   w.n_sink, w.recent_num, w.recent_den)
            hc = HeadCache(C, w.D, w.n_sink, w.recent_num, w.recent_den)
            hc.load(K2, V2, pos2, s2)
            self.twins[(b, l, h)] = hc

    # ---- device state of one head, as numpy
    def head_state(self, b, l, h):
        lo, hi = self.cache.rows(b, l, h)
        c = self.cache
        if self.kv_dtype == bk.KV_FP8_E4M3:
            four = c.kv_scale_host[l, h]
            K = ofp8.decode(c.k_slab[lo:hi].cpu().numpy()) * float(four[0])
            V = ofp8.decode(c.v_slab[lo:hi].cpu().numpy()) * float(four[2])
        else:
            K, V = f64(c.k_slab[lo:hi]), f64(c.v_slab[lo:hi])
        return dict(K=K, V=V, pos=c.pos[lo:hi].cpu().numpy().astype(np.int64),
                    score=c.score[lo:hi].cpu().numpy(), len=int(c.len[b, l, h]), free=int(c.free_slot[b, l, h]))

    def valid_slots(self, st):
        return np.array([j for j in range(st["len"] + 1) if j != st["free"]][: st["len"]], dtype=np.int64)

    def check_state(self, b, l, h, what="", exact_rows=True):
        """Slot-by-slot comparison of the device head with its oracle twin."""
        st, tw = self.head_state(b, l, h), self.twins[(b, l, h)]
        tag = "%s head (b%d,l%d,h%d)" % (what, b, l, h)
        assert st["len"] == tw.length, tag + " len"
        assert st["free"] == tw.free_slot, tag + " free_slot"
        s = self.valid_slots(st)
        np.testing.assert_array_equal(st["pos"][s], tw.pos[s], err_msg=tag + " pos")
        if exact_rows:
            np.testing.assert_array_equal(st["K"][s], tw.K[s], err_msg=tag + " K rows")
            np.testing.assert_array_equal(st["V"][s], tw.V[s], err_msg=tag + " V rows")
        assert_close(st["score"][s], tw.score[s], tag + " score")

    # ---- near ties (two rows whose scores the two sides order differently although both are right)
    def _settle_victim(self, tw, dev_free, ref_score, dev_score, t_pos, tag):
        """The library evicted slot `dev_free`, the oracle twin `tw.free_slot`.  That is accepted, and counted,
        only when the oracle's own scores of the two rows differ by less than the deviation between the two
        sides' scores that this very step shows (plus 1e-6 relative), and the library's row was a lawful
        candidate; the twin then follows the library so that the run can go on.  Anything else fails."""
        a, b = int(dev_free), int(tw.free_slot)
        w = self.w
        W = oevict.recent_window(tw.C - 1, w.n_sink, w.recent_num, w.recent_den)
        assert w.n_sink <= tw.pos[a] <= t_pos - W, tag + " evicted a protected row"
        gap = abs(float(ref_score[a]) - float(ref_score[b]))
        slack = 2.0 * float(np.max(np.abs(dev_score - ref_score))) + 1e-6 * max(abs(float(ref_score[a])), abs(float(ref_score[b])))
        assert gap <= slack, tag + " victim differs from the oracle's beyond a near tie (gap %.3e, slack %.3e)" % (gap, slack)
        self.near_ties.append((tag, gap))
        tw.free_slot = a

    def _launch(self, step_index, flags):
        w = self.w
        q, kn, vn = wl.decode_inputs(w, step_index, self.scales, self.device, layers=(self.lb, self.le))
        t_pos = self.t
        if self.layer_plans is None:
            bk.baklava_decode_attn(self.shape, self.cache, q, kn, vn, t_pos, self.out, self.lse, flags, self.plan, self.ws)
        else:
            torch.cuda.synchronize()                        # the inputs of every layer are complete before the first call
            for i, (plan, ws) in enumerate(self.layer_plans):
                bk.baklava_decode_attn(self.shape, self.cache, q[i:i + 1], kn[i:i + 1], vn[i:i + 1], t_pos,
                                       self.out[i:i + 1], self.lse[i:i + 1],
                                       flags | (bk.FLAG_OVERLAP_PREV if i > 0 else 0), plan, ws)
        torch.cuda.synchronize()
        if not (flags & bk.FLAG_NO_APPEND):
            self.t += 1
        return q, kn, vn, t_pos

    def step(self, step_index, flags=0, check=True, check_selection=True, teacher=None, hold=None):
        """One decode step on the device, compared with the oracle in two ways.
        Free-running (the heads in `self.heads`): each twin evolves from the seeded inputs alone.
        Teacher-forced (the heads in `teacher`): the oracle restarts from the state the device held before the
        step, so that a deviation cannot build up over a long run and every step is judged on its own.  The K / V
        rows of the teacher-forced heads in `hold` (default: all of them) stay on the host between steps (only
        appended rows change); the others are downloaded whenever they are checked."""
        w = self.w
        g = w.g
        if teacher:
            pre = self._snapshot(teacher)
        q, kn, vn, t_pos = self._launch(step_index, flags)
        append = not (flags & bk.FLAG_NO_APPEND)
        if not check:
            return
        qh, knh, vnh = f64(q), f64(kn), f64(vn)
        out, lse = f64(self.out), f64(self.lse)
        evicting = not (flags & bk.FLAG_NO_EVICT) and (not (flags & bk.FLAG_NO_SCORE) or w.recent_num == w.recent_den)
        for (b, l, h) in self.heads:
            tw = self.twins[(b, l, h)]
            li = l - self.lb
            o_ref, lse_ref, ev = tw.step(qh[li, b, h * g:(h + 1) * g], self.as_stored(knh[li, b, h], l, h, 0),
                                         self.as_stored(vnh[li, b, h], l, h, 1), t_pos,
                                         append=append, update_score=not (flags & bk.FLAG_NO_SCORE), evict=evicting)
            tag = "step %d head (b%d,l%d,h%d)" % (step_index, b, l, h)
            assert_close(out[li, b, h * g:(h + 1) * g], o_ref, tag + " out")
            assert_close(lse[li, b, h * g:(h + 1) * g], lse_ref, tag + " lse")
            st = self.head_state(b, l, h)
            if check_selection and ev >= 0:
                # the retention rule applied to the library's own post-update scores must name the
                # same victim the library chose, bit for bit
                C = int(self.cap[l, h])
                keep = oevict.select_keep(st["pos"], st["score"], C - 1, w.n_sink, w.recent_num, w.recent_den)
                gone = sorted(set(range(C)) - set(int(i) for i in keep))
                assert gone == [st["free"]], tag + " victim on the library's own scores"
            if ev >= 0 and st["free"] != tw.free_slot:
                self._settle_victim(tw, st["free"], tw.score, st["score"].astype(np.float64), t_pos, tag)
            self.check_state(b, l, h, tag)
        if teacher:
            post = self._snapshot(teacher)
            for key in teacher:
                self._check_teacher(key, pre[key], post[key], qh, knh, vnh, out, lse, t_pos, step_index, flags,
                                    hold is None or key in hold)
        assert int(self.cache.status.item()) == 0

    # ---- teacher-forced checking
    def _snapshot(self, heads):
        """pos, score, len, free_slot of `heads` as the device holds them now: {head: dict}; two gathers, two copies."""
        key = tuple(heads)
        if getattr(self, "_snap_key", None) != key:
            spans, idx = {}, []
            at = 0
            for (b, l, h) in heads:
                lo, hi = self.cache.rows(b, l, h)
                spans[(b, l, h)] = (at, at + hi - lo)
                idx.append(torch.arange(lo, hi, dtype=torch.int64))
                at += hi - lo
            self._snap_key, self._snap_spans = key, spans
            self._snap_rows = torch.cat(idx).to(self.device)
            flat = [(b * self.w.L + l) * self.w.Hkv + h for (b, l, h) in heads]
            self._snap_heads = torch.tensor(flat, dtype=torch.int64, device=self.device)
        c = self.cache
        pos = c.pos[self._snap_rows].cpu().numpy().astype(np.int64)
        score = c.score[self._snap_rows].cpu().numpy()
        ln = c.len.reshape(-1)[self._snap_heads].cpu().numpy()
        fr = c.free_slot.reshape(-1)[self._snap_heads].cpu().numpy()
        snap = {}
        for i, hd in enumerate(heads):
            a, z = self._snap_spans[hd]
            snap[hd] = dict(pos=pos[a:z], score=score[a:z], len=int(ln[i]), free=int(fr[i]))
        return snap

    def _rows_host(self, b, l, h):
        lo, hi = self.cache.rows(b, l, h)
        c = self.cache
        if self.kv_dtype == bk.KV_FP8_E4M3:
            four = c.kv_scale_host[l, h]
            return (ofp8.decode(c.k_slab[lo:hi].cpu().numpy()) * float(four[0]),
                    ofp8.decode(c.v_slab[lo:hi].cpu().numpy()) * float(four[2]))
        return f64(c.k_slab[lo:hi]), f64(c.v_slab[lo:hi])

    def _check_teacher(self, key, pre, post, qh, knh, vnh, out, lse, t_pos, step_index, flags, hold_rows):
        w, g = self.w, self.w.g
        b, l, h = key
        li = l - self.lb
        C = int(self.cap[l, h])
        tag = "teacher-forced step %d head (b%d,l%d,h%d)" % (step_index, b, l, h)
        append = not (flags & bk.FLAG_NO_APPEND)
        k_row = self.as_stored(knh[li, b, h], l, h, 0)
        v_row = self.as_stored(vnh[li, b, h], l, h, 1)
        held = self.held_rows.get(key) if hold_rows else None
        if held is None:
            K, V = self._rows_host(b, l, h)                 # as after the step: only the appended row is new
            if append and pre["len"] < C:
                np.testing.assert_array_equal(K[pre["free"]], k_row, err_msg=tag + " appended K row")
                np.testing.assert_array_equal(V[pre["free"]], v_row, err_msg=tag + " appended V row")
            if hold_rows:
                self.held_rows[key] = (K, V)
        else:
            K, V = held                                     # the oracle's own append keeps them current;
            if append and pre["len"] < C:                   # the device's appended row is checked on its own
                lo, _ = self.cache.rows(b, l, h)
                row = lo + pre["free"]
                kd, vd = self.cache.k_slab[row:row + 1], self.cache.v_slab[row:row + 1]
                if self.kv_dtype == bk.KV_FP8_E4M3:
                    four = self.cache.kv_scale_host[l, h]
                    kd = ofp8.decode(kd.cpu().numpy()) * float(four[0]); vd = ofp8.decode(vd.cpu().numpy()) * float(four[2])
                else:
                    kd, vd = f64(kd), f64(vd)
                np.testing.assert_array_equal(kd[0], k_row, err_msg=tag + " appended K row")
                np.testing.assert_array_equal(vd[0], v_row, err_msg=tag + " appended V row")
        tw = HeadCache(C, w.D, w.n_sink, w.recent_num, w.recent_den)
        tw.K, tw.V = K, V
        tw.pos = pre["pos"].copy()
        tw.score = pre["score"].astype(np.float64)
        tw.length, tw.free_slot = pre["len"], pre["free"]
        evicting = not (flags & bk.FLAG_NO_EVICT) and (not (flags & bk.FLAG_NO_SCORE) or w.recent_num == w.recent_den)
        o_ref, lse_ref, ev = tw.step(qh[li, b, h * g:(h + 1) * g], k_row, v_row, t_pos, append=append,
                                     update_score=not (flags & bk.FLAG_NO_SCORE), evict=evicting)
        assert_close(out[li, b, h * g:(h + 1) * g], o_ref, tag + " out")
        assert_close(lse[li, b, h * g:(h + 1) * g], lse_ref, tag + " lse")
        assert post["len"] == tw.length, tag + " len"
        dev_score = post["score"].astype(np.float64)
        if ev >= 0:
            keep = oevict.select_keep(post["pos"], post["score"], C - 1, w.n_sink, w.recent_num, w.recent_den)
            gone = sorted(set(range(C)) - set(int(i) for i in keep))
            assert gone == [post["free"]], tag + " victim on the library's own scores"
            if post["free"] != tw.free_slot:
                self._settle_victim(tw, post["free"], tw.score, dev_score, t_pos, tag)
        assert post["free"] == tw.free_slot, tag + " free_slot"
        s = tw.valid_slots()
        np.testing.assert_array_equal(post["pos"][s], tw.pos[s], err_msg=tag + " pos")
        assert_close(dev_score[s], tw.score[s], tag + " score")

    def check_held_rows(self):
        """At the end of a long teacher-forced run: the rows the oracle carried along (appends only) are, bit for
        bit, the rows the device holds."""
        for (b, l, h), (K, V) in self.held_rows.items():
            Kd, Vd = self._rows_host(b, l, h)
            n = int(self.cache.len[b, l, h]); f = int(self.cache.free_slot[b, l, h])
            s = np.array([j for j in range(n + 1) if j != f][:n], dtype=np.int64)
            np.testing.assert_array_equal(Kd[s], K[s], err_msg="held K rows of head (b%d,l%d,h%d)" % (b, l, h))
            np.testing.assert_array_equal(Vd[s], V[s], err_msg="held V rows of head (b%d,l%d,h%d)" % (b, l, h))
