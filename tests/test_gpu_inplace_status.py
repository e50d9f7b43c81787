"""GPU tests of two corners of the boundary: compaction of a slab in place (baklava_evict without a
dense source, Eq. 5-6 applied to the rows a cache already holds) against the oracle, and the device
status word (BAD_STATE, TIMEOUT) reached without faulting or hanging anything: bad state is written
from the host, the time-out is a bounded wait on a tile that is never requested."""
import numpy as np
import pytest
import torch

from oracle import eviction as oe
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth
from paper_2502_13176_b200 import workloads as wl

from harness import Session, f64

pytestmark = pytest.mark.gpu


def _scrambled_cache(L, Hkv, B, D, caps, n_sink, num, den, seed, kv_dtype=bk.KV_BF16, ties=False):
    """A cache whose heads hold rows in arbitrary slot order (as slot reuse leaves them), some with a hole."""
    dev = "cuda"
    shape = bk.make_shape(L, Hkv, Hkv, D, 16, n_sink, num, den)
    cap = np.array(caps, dtype=np.int32).reshape(L, Hkv)
    off = np.concatenate([[0], np.cumsum(cap.reshape(-1))[:-1]]).reshape(L, Hkv).astype(np.int64)
    stride = int(cap.sum())
    scale = None
    if kv_dtype == bk.KV_FP8_E4M3:
        scale = np.tile(np.array([0.02, 1.0 / np.float32(0.02), 0.02, 1.0 / np.float32(0.02)], dtype=np.float32), (L, Hkv, 1))
    cache = bk.Cache(shape, cap, off, stride, B, dev, kv_dtype=kv_dtype, kv_scale=scale)
    rng = np.random.default_rng(seed)
    rows = B * stride
    if kv_dtype == bk.KV_FP8_E4M3:
        cache.k_slab.copy_(torch.from_numpy(rng.integers(0, 120, (rows, D)).astype(np.uint8)))
        cache.v_slab.copy_(torch.from_numpy(rng.integers(0, 120, (rows, D)).astype(np.uint8)))
    else:
        cache.k_slab.copy_(synth.normal_bf16(seed, 1, (rows, D), dev))
        cache.v_slab.copy_(synth.normal_bf16(seed, 2, (rows, D), dev))
    pos = np.full(rows, -1, dtype=np.int32)
    score = rng.random(rows).astype(np.float32)
    if ties:
        score = np.round(score * 4) / 4
    ln = np.zeros((B, L, Hkv), dtype=np.int32)
    fr = np.zeros((B, L, Hkv), dtype=np.int32)
    for b in range(B):
        for l in range(L):
            for h in range(Hkv):
                C = int(cap[l, h])
                lo = b * stride + int(off[l, h])
                kind = rng.integers(0, 4)
                if kind == 0:                        # full cache (NO_EVICT ran it up): no hole
                    n, f = C, C
                elif kind == 1:                      # steady state: C - 1 rows and a hole somewhere
                    n = C - 1
                    f = int(rng.integers(0, n + 1))
                elif kind == 2:                      # still filling
                    n = int(rng.integers(1, C))
                    f = n
                else:                                # a few rows and a hole
                    n = int(rng.integers(1, C - 1))
                    f = int(rng.integers(0, n + 1))
                span = n + (1 if f < n else 0)
                p = rng.permutation(n + 7)[:n]       # distinct positions, sinks mostly present
                slots = [j for j in range(span) if j != f]
                pos[lo + np.array(slots)] = p
                ln[b, l, h], fr[b, l, h] = n, f
    cache.pos.copy_(torch.from_numpy(pos))
    cache.score.copy_(torch.from_numpy(score))
    cache.len.copy_(torch.from_numpy(ln))
    cache.free_slot.copy_(torch.from_numpy(fr))
    return shape, cache, cap, off, stride


def _check_in_place(shape, cache, cap, off, stride, reserve, B, L, Hkv, n_sink, num, den):
    before = dict(k=cache.k_slab.cpu(), v=cache.v_slab.cpu(), pos=cache.pos.cpu().numpy(),
                  score=cache.score.cpu().numpy(), len=cache.len.cpu().numpy(), free=cache.free_slot.cpu().numpy())
    T = int(cap.max())
    ws = torch.empty((bk.baklava_evict_workspace_size(shape, B, L, T),), dtype=torch.uint8, device="cuda")
    bk.baklava_evict(shape, cache, 0, L, None, None, None, T, 0, 0, 0, reserve, ws)
    torch.cuda.synchronize()
    assert int(cache.status.item()) == 0
    moved = 0
    for b in range(B):
        for l in range(L):
            for h in range(Hkv):
                C = int(cap[l, h]); lo = b * stride + int(off[l, h])
                n, f = int(before["len"][b, l, h]), int(before["free"][b, l, h])
                slots = np.array([j for j in range(n + 1) if j != f][:n], dtype=np.int64)
                K = before["k"][lo:lo + C][slots]; V = before["v"][lo:lo + C][slots]
                pos = before["pos"][lo:lo + C][slots]; sc = before["score"][lo:lo + C][slots]
                _, _, pos2, s2, idx = oe.compact_in_place(np.zeros((n, 1)), np.zeros((n, 1)), pos, sc, C - reserve,
                                                          n_sink, num, den)
                m = len(idx)
                assert int(cache.len[b, l, h]) == m and int(cache.free_slot[b, l, h]) == m, (b, l, h)
                np.testing.assert_array_equal(cache.pos[lo:lo + m].cpu().numpy(), pos2)
                np.testing.assert_array_equal(cache.score[lo:lo + m].cpu().numpy(), s2)
                assert torch.equal(cache.k_slab[lo:lo + m].cpu(), K[idx])
                assert torch.equal(cache.v_slab[lo:lo + m].cpu(), V[idx])
                moved += int(m < n)
    return moved


@pytest.mark.parametrize("D,kv,ties", [(128, bk.KV_BF16, False), (64, bk.KV_BF16, True), (128, bk.KV_FP8_E4M3, True)])
def test_in_place_compaction_matches_oracle(D, kv, ties):
    L, Hkv, B = 2, 3, 2
    caps = [64, 160, 1200, 2064, 48, 3008]
    for seed, reserve in [(1, 1), (2, 17), (3, 40)]:                 # close the holes; shrink the budgets
        shape, cache, cap, off, stride = _scrambled_cache(L, Hkv, B, D, caps, 4, 1, 2, seed, kv, ties)
        moved = _check_in_place(shape, cache, cap, off, stride, reserve, B, L, Hkv, 4, 1, 2)
        assert moved > 0 or reserve == 1


def test_in_place_after_decode_steps_then_decoding_goes_on():
    """A cache run up to its capacity under NO_EVICT, cut back in place, then decoded further: the oracle twin
    gets the same cut (compact_in_place on its own rows) and the steps after it still agree."""
    w = wl.scaled(wl.LLAMA3_8B_32K, L=2, T=700, steps=8)
    s = Session(w, chunk_tokens=128)
    for i in range(3):
        s.step(i)
    s.step(3, flags=bk.FLAG_NO_EVICT)                                # every head is full now
    T = int(s.cap.max())
    ws = torch.empty((bk.baklava_evict_workspace_size(s.shape, w.B, w.L, T),), dtype=torch.uint8, device="cuda")
    reserve = 9
    bk.baklava_evict(s.shape, s.cache, 0, w.L, None, None, None, T, 0, 0, 0, reserve, ws)
    torch.cuda.synchronize()
    for (b, l, h), tw in s.twins.items():
        slots = tw.valid_slots()
        K2, V2, pos2, s2, _ = oe.compact_in_place(tw.K[slots], tw.V[slots], tw.pos[slots], tw.score[slots],
                                                  tw.C - reserve, w.n_sink, w.recent_num, w.recent_den)
        tw.load(K2, V2, pos2, s2)
        s.check_state(b, l, h, "after the cut in place")
    for i in range(4, 8):
        s.step(i)


def test_in_place_refuses_mixed_arguments_and_small_workspace_rows():
    shape, cache, cap, off, stride = _scrambled_cache(1, 2, 1, 64, [64, 128], 4, 1, 2, 5)
    ws = torch.empty((bk.baklava_evict_workspace_size(shape, 1, 1, 128),), dtype=torch.uint8, device="cuda")
    k = torch.zeros((2 * 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bk.BaklavaError) as e:                        # one dense source only
        bk.baklava_evict(shape, cache, 0, 1, k, None, None, 128, 0, 256, 128, 1, ws)
    assert e.value.code == -1
    sc = torch.zeros((256,), dtype=torch.float32, device="cuda")
    with pytest.raises(bk.BaklavaError) as e:                        # dense scores without dense rows
        bk.baklava_evict(shape, cache, 0, 1, None, None, sc, 128, 0, 256, 128, 1, ws)
    assert e.value.code == -1
    before = cache.len.clone()
    bk.baklava_evict(shape, cache, 0, 1, None, None, None, 64, 0, 0, 0, 1, ws)   # T below the larger capacity
    torch.cuda.synchronize()
    assert int(cache.status.item()) & bk.STATUS_BAD_STATE
    assert int(cache.len[0, 0, 1]) == int(before[0, 0, 1])          # that head is left alone


# ---------------------------------------------------------------- status word
def test_bad_state_written_from_the_host_is_reported_and_contained():
    w = wl.scaled(wl.TINY, T=300, steps=3)
    s = Session(w, chunk_tokens=64)
    s.step(0)
    victim = s.heads[1]
    b, l, h = victim
    good_len = int(s.cache.len[b, l, h])
    for bad_len, bad_free in [(int(s.cap[l, h]) + 5, 0), (-3, 0), (good_len, int(s.cap[l, h]) + 1)]:
        s.cache.len[b, l, h] = bad_len
        free_before = int(s.cache.free_slot[b, l, h])
        if bad_free:
            s.cache.free_slot[b, l, h] = bad_free
        lo, hi = s.cache.rows(b, l, h)
        score_before = s.cache.score[lo:hi].clone()
        q, kn, vn = wl.decode_inputs(w, 1, s.scales, "cuda")
        bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t, s.out, s.lse, bk.FLAG_NO_APPEND, s.plan, s.ws)
        torch.cuda.synchronize()
        assert int(s.cache.status.item()) == bk.STATUS_BAD_STATE
        assert int(s.cache.len[b, l, h]) == bad_len                  # the head is skipped, not repaired
        assert torch.equal(score_before, s.cache.score[lo:hi])
        for key, tw in s.twins.items():                              # every other head did an ordinary step
            if key != victim:
                bb, ll, hh = key
                tw.step(f64(q)[ll, bb, hh * w.g:(hh + 1) * w.g], None, None, s.t, append=False)
                s.check_state(bb, ll, hh, "beside the bad head")
        s.cache.status.zero_()
        s.cache.len[b, l, h] = good_len
        s.cache.free_slot[b, l, h] = free_before
    s.step(1)                                                        # healthy again: full parity on every head
    s.step(2)


def test_capacity_too_small_for_sinks_and_window_is_reported():
    # every row of a 16-token cache is a sink: when the cache fills there is nothing to evict
    w = wl.scaled(wl.TINY, T=64, steps=20, n_sink=40)
    s = Session(w, prefill=False, chunk_tokens=64, caps=[16, 16, 16, 16])
    for i in range(14):
        s.step(i)
    q, kn, vn = wl.decode_inputs(w, 14, s.scales, "cuda")
    bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t, s.out, s.lse, 0, s.plan, s.ws)      # 15th row: still fits
    bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t + 1, s.out, s.lse, 0, s.plan, s.ws)  # 16th: nobody may leave
    torch.cuda.synchronize()
    assert int(s.cache.status.item()) == bk.STATUS_BAD_STATE
    assert torch.all(s.cache.len == 16)
    s.cache.status.zero_()
    bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t + 2, s.out, s.lse, 0, s.plan, s.ws)  # now it is simply full
    torch.cuda.synchronize()
    assert int(s.cache.status.item()) == bk.STATUS_OVERFLOW


@pytest.mark.parametrize("one_kernel", [False, True], ids=["two-kernels", "one-kernel"])
@pytest.mark.parametrize("kv", [bk.KV_BF16, bk.KV_FP8_E4M3], ids=["bf16", "fp8"])
def test_wait_that_runs_out_sets_timeout_and_leaves_everything_usable(kv, one_kernel):
    """The first chunk of every head is fed one tile only (test flag), so the consumers' bounded wait for the
    second tile runs out after a short limit: TIMEOUT is set, no head changes, and the next step on the same
    workspace is an ordinary, correct step.  A launch this short ends in a second kernel for the score update;
    with BAKLAVA_FLAG_OVERLAP_PREV (nothing is in flight here, so the flag is lawful) the CTA that finishes a head
    does it, and that path must drop the head's step just as cleanly."""
    w = wl.scaled(wl.LLAMA3_8B_32K, L=2, T=3000, steps=4)
    s = Session(w, chunk_tokens=256, kv_dtype=kv)
    assert int(s.cap.min()) > 2 * 128
    s.step(0)
    state = [t.clone() for t in (s.cache.len, s.cache.free_slot, s.cache.score)]
    q, kn, vn = wl.decode_inputs(w, 1, s.scales, "cuda")
    bk.baklava_set_wait_limit(2_000_000)                             # about a millisecond
    try:
        s.out.fill_(7.0)
        flags = bk.FLAG_TEST_STALL | (bk.FLAG_OVERLAP_PREV if one_kernel else 0)
        bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t, s.out, s.lse, flags, s.plan, s.ws)
        torch.cuda.synchronize()
    finally:
        bk.baklava_set_wait_limit(100_000_000)
    assert int(s.cache.status.item()) == bk.STATUS_TIMEOUT
    assert torch.equal(state[0], s.cache.len) and torch.equal(state[1], s.cache.free_slot)
    valid = s.cache.pos.ne(-1) & (s.cache.pos < s.t)
    assert torch.equal(state[2][valid], s.cache.score[valid])
    assert torch.all(s.out == 7.0)                                   # a lost head writes no output
    s.cache.status.zero_()
    for i in range(1, 4):                                            # the same workspace, no re-zeroing
        s.step(i)
    with pytest.raises(bk.BaklavaError):
        bk.baklava_set_wait_limit(0)
