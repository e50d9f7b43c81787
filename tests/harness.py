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
                 kv_dtype=bk.KV_BF16):
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
                                           n_sm=torch.cuda.get_device_properties(0).multi_processor_count).to(device)
        self.ws = bk.decode_workspace(self.plan, device)
        nl = self.le - self.lb
        self.out = torch.zeros((nl, w.B, w.Hq, w.D), dtype=torch.bfloat16, device=device)
        self.lse = torch.zeros((nl, w.B, w.Hq), dtype=torch.float32, device=device)
        self.heads = heads if heads is not None else [(b, l, h) for b in range(w.B)
                                                      for l in range(self.lb, self.le) for h in range(w.Hkv)]
        self.twins = {}
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

    def step(self, step_index, flags=0, check=True, check_selection=True):
        """One decode step on the device and on the oracle twins; compares outputs and state."""
        w = self.w
        q, kn, vn = wl.decode_inputs(w, step_index, self.scales, self.device, layers=(self.lb, self.le))
        t_pos = self.t
        bk.baklava_decode_attn(self.shape, self.cache, q, kn, vn, t_pos, self.out, self.lse, flags, self.plan, self.ws)
        torch.cuda.synchronize()
        append = not (flags & bk.FLAG_NO_APPEND)
        if append:
            self.t += 1
        if not check:
            return
        qh, knh, vnh = f64(q), f64(kn), f64(vn)
        out, lse = f64(self.out), f64(self.lse)
        g = w.g
        for (b, l, h) in self.heads:
            tw = self.twins[(b, l, h)]
            li = l - self.lb
            o_ref, lse_ref, ev = tw.step(qh[li, b, h * g:(h + 1) * g], self.as_stored(knh[li, b, h], l, h, 0),
                                         self.as_stored(vnh[li, b, h], l, h, 1), t_pos,
                                         append=append, update_score=not (flags & bk.FLAG_NO_SCORE),
                                         evict=not (flags & bk.FLAG_NO_EVICT) and
                                         (not (flags & bk.FLAG_NO_SCORE) or w.recent_num == w.recent_den))
            tag = "step %d head (b%d,l%d,h%d)" % (step_index, b, l, h)
            assert_close(out[li, b, h * g:(h + 1) * g], o_ref, tag + " out")
            assert_close(lse[li, b, h * g:(h + 1) * g], lse_ref, tag + " lse")
            if check_selection and ev >= 0:
                # the retention rule applied to the library's own post-update scores must name the
                # same victim the library chose, bit for bit
                st = self.head_state(b, l, h)
                C = int(self.cap[l, h])
                keep = oevict.select_keep(st["pos"], st["score"], C - 1, w.n_sink, w.recent_num, w.recent_den)
                gone = sorted(set(range(C)) - set(int(i) for i in keep))
                assert gone == [st["free"]], tag + " victim on the library's own scores"
            self.check_state(b, l, h, tag)
        assert int(self.cache.status.item()) == 0
