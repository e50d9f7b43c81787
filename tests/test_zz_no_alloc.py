"""baklava_evict_static: the bulk eviction for callers that cannot allocate device memory at the
call site (a frozen or exhausted framework memory pool, a plug-in that only receives its input and
output buffers, start-up code that runs before any allocator exists).  Its scratch is a fixed array
inside the library, so the test checks that it gives exactly what baklava_evict gives with a
caller-provided workspace, twice in a row (the array keeps the first call's contents), and that a
request beyond the array's size is refused on the host."""
import numpy as np
import pytest
import torch

from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(seed, L, B, Hkv, T, D, dev):
    k = synth.normal_bf16(seed, 1, (L, B, Hkv, T, D), dev)
    v = synth.normal_bf16(seed, 2, (L, B, Hkv, T, D), dev)
    sc = synth.uniform_f64(seed, 3, 0, L * B * Hkv * T, dev).to(torch.float32).reshape(L, B, Hkv, T)
    return k, v, sc


def test_static_scratch_matches_workspace_version_twice():
    dev = "cuda"
    L, Hkv, B, D = 2, 3, 2, 128
    shape = bk.make_shape(L, Hkv * 2, Hkv, D)
    cap = np.array([[64, 320, 1024], [512, 16, 2000 // 16 * 16]], dtype=np.int32)
    off = np.concatenate([[0], np.cumsum(cap.reshape(-1))[:-1]]).reshape(L, Hkv).astype(np.int64)
    stride = int(cap.sum())
    for call, (seed, T) in enumerate([(11, 1500), (12, 700)]):      # second call: shorter prompt, stale tail in the array
        k, v, sc = _inputs(seed, L, B, Hkv, T, D, dev)
        ref = bk.Cache(shape, cap, off, stride, B, dev)
        got = bk.Cache(shape, cap, off, stride, B, dev)
        for c in (ref, got):
            c.k_slab.zero_(); c.v_slab.zero_()
        ws = torch.empty((bk.baklava_evict_workspace_size(shape, B, L, T),), dtype=torch.uint8, device=dev)
        bk.baklava_evict(shape, ref, 0, L, k, v, sc, T, B * Hkv * T, Hkv * T, T, 1, ws)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        bk.baklava_evict_static(shape, got, 0, L, k, v, sc, T, B * Hkv * T, Hkv * T, T, 1)
        torch.cuda.synchronize()
        if call > 0:                                     # after the first call's one-time set-up: the call itself
            assert torch.cuda.mem_get_info()[0] == free_before   # takes no device memory and returns none
        assert int(got.status.item()) == 0 and int(ref.status.item()) == 0
        assert torch.equal(got.len, ref.len) and torch.equal(got.free_slot, ref.free_slot), "call %d" % call
        assert torch.equal(got.pos, ref.pos) and torch.equal(got.score, ref.score), "call %d" % call
        assert torch.equal(got.k_slab, ref.k_slab) and torch.equal(got.v_slab, ref.v_slab), "call %d" % call
        assert int(got.len.sum()) > 0


def test_request_beyond_the_fixed_array_is_refused():
    dev = "cuda"
    shape = bk.make_shape(1, 2, 2, 64)
    T = bk.EVICT_STATIC_MAX_ENTRIES // 2 + 16            # 2 heads * T just over the limit
    cap = np.array([[64, 64]], dtype=np.int32)
    cache = bk.Cache(shape, cap, np.array([[0, 64]], dtype=np.int64), 128, 1, dev)
    k = torch.zeros((2 * T, 64), dtype=torch.bfloat16, device=dev)
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_evict_static(shape, cache, 0, 1, k, k, None, T, 0, 2 * T, T, 1)
    assert e.value.code == -4
    torch.cuda.synchronize()
    assert int(cache.len.sum()) == 0
