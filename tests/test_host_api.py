"""CPU tests of the C-ABI library: it loads, exports what the header declares, and its host code
(Algorithm 1 step 2, Algorithm 2, the decode plan, argument checks) agrees with the oracle."""
import ctypes
import json
import os
import re

import numpy as np
import pytest

from oracle import allocation as oa
from oracle import profiling as op
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import build as bkbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    bkbuild.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "baklava.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(baklava_[a-z_]+)\s*\(", header))
    assert {"baklava_profile_heads", "baklava_allocate", "baklava_decode_attn", "baklava_evict"} <= names
    L = bk.lib()
    for n in names:
        assert hasattr(L, n), n
    assert bk.strerror(0) == "ok" and "shape" in bk.strerror(-2)


def test_allocate_matches_oracle_on_hand_worked_cases():
    cases = json.load(open(os.path.join(ROOT, "tests", "golden", "allocation_worked.json")))["cases"]
    for c in cases:
        m = len(c["I"])
        shape = bk.make_shape(1, m if m <= 8 else m, m, 64)
        cap, off, stride = bk.baklava_allocate(shape, np.array(c["I"]).reshape(1, m), c["t"], c["r"][0], c["r"][1],
                                               c["total"] * 16, c["min"] * 16, c["max"] * 16)
        assert list(cap[0] // 16) == c["pages"]
        assert stride == c["total"] * 16 and list(off[0]) == list(np.concatenate([[0], np.cumsum(cap[0])[:-1]]))


@pytest.mark.parametrize("scope", [bk.SCOPE_LAYER, bk.SCOPE_MODEL])
def test_allocate_bit_exact_vs_oracle_random(scope):
    rng = np.random.default_rng(100 + scope)
    for trial in range(150):
        L, Hkv = int(rng.integers(1, 6)), int(rng.integers(1, 9))
        page = 16 * int(rng.integers(1, 3))
        shape = bk.make_shape(L, Hkv, Hkv, 128, page=page)
        I = np.exp(rng.normal(0, 1.2, (L, Hkv)))
        if trial % 5 == 0:
            I = np.round(I, 1)                                       # ties
        base = int(rng.integers(3, 300))
        total = (base * L * Hkv + int(rng.integers(0, L * Hkv)))
        r_den = int(rng.integers(1, 9)); r_num = int(rng.integers(0, r_den + 1))
        mn, mx = int(rng.integers(1, 3)), base + 1 + int(rng.integers(0, 3 * base))
        t = float(np.exp(rng.normal(0, 0.5)))
        li = np.exp(rng.normal(0, 1, L)) if (scope == bk.SCOPE_LAYER and trial % 3 == 0) else None
        kw = dict(layer_importance=li, t_layer=1.0, rl_num=1, rl_den=3) if li is not None else {}
        try:
            want = oa.allocate(I, t, r_num, r_den, total, mn, mx, page, scope=scope, **kw)
        except oa.AllocationError:
            with pytest.raises(bk.BaklavaError) as e:
                bk.baklava_allocate(shape, I, t, r_num, r_den, total * page, mn * page, mx * page, scope=scope, **kw)
            assert e.value.code == -3
            continue
        cap, off, stride = bk.baklava_allocate(shape, I, t, r_num, r_den, total * page, mn * page, mx * page,
                                               scope=scope, **kw)
        np.testing.assert_array_equal(cap, want[0])
        np.testing.assert_array_equal(off, want[1])
        assert stride == want[2]


def test_importance_matches_oracle():
    rng = np.random.default_rng(7)
    P, L, Hq, Hkv = 3, 4, 8, 2
    s = rng.uniform(-1, 1, (P, L, Hq)).astype(np.float32)
    got = bk.baklava_importance(bk.make_shape(L, Hq, Hkv, 128), s)
    np.testing.assert_allclose(got, op.kv_importance(s.astype(np.float64), Hq // Hkv), rtol=1e-14, atol=1e-15)


def test_decode_plan_covers_every_head_once():
    rng = np.random.default_rng(9)
    for trial in range(40):
        L, Hkv, B = int(rng.integers(1, 5)), int(rng.integers(1, 5)), int(rng.integers(1, 4))
        shape = bk.make_shape(L, Hkv * 2, Hkv, 128)
        cap = (rng.integers(1, 400, (L, Hkv)) * 16).astype(np.int32)
        lb = int(rng.integers(0, L)); le = int(rng.integers(lb + 1, L + 1))
        chunk = int(rng.choice([0, 64, 100, 512, 4096]))
        plan = bk.baklava_decode_plan(shape, cap, B, lb, le, int(cap.sum()), chunk_tokens=chunk, n_sm=148)
        it, info = plan.items, plan.info
        assert info.n_units == (le - lb) * B * Hkv and info.ws_bytes > 0
        assert info.n_items + info.n_score_items == len(it)
        _check_cover(it[:info.n_items], info, cap, lb, B, Hkv)
        if info.n_score_items:
            assert info.n_items <= 148 * 3
            _check_cover(it[info.n_items:], info, cap, lb, B, Hkv)


def _check_cover(it, info, cap, lb, B, Hkv):
    seen = {}
    prev_cap = None
    for row, (unit, begin, clen, packed) in enumerate(it):
        piece, pieces = packed & 0xffff, packed >> 16
        li, rem = divmod(unit, B * Hkv); b, h = divmod(rem, Hkv)
        c = int(cap[lb + li, h])
        assert clen % 64 == 0 and begin == piece * clen and begin < c and pieces * clen >= c
        assert (pieces - 1) * clen < c
        seen.setdefault(unit, []).append(piece)
        if piece == 0:
            assert prev_cap is None or c <= prev_cap       # largest heads first
            prev_cap = c
        else:
            assert it[row - 1][0] == unit and (it[row - 1][3] & 0xffff) == piece - 1   # a head's chunks are adjacent
    assert sorted(seen) == list(range(info.n_units))
    for unit, pcs in seen.items():
        assert pcs == list(range(len(pcs)))


def test_argument_errors_are_codes_not_crashes():
    shape = bk.make_shape(2, 4, 2, 128)
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_allocate(bk.make_shape(2, 4, 2, 96), np.ones((2, 2)), 1.0, 1, 2, 64, 16, 64)
    assert e.value.code == -2
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_allocate(bk.make_shape(2, 18, 2, 128), np.ones((2, 2)), 1.0, 1, 2, 64, 16, 64)     # g = 9
    assert e.value.code == -2
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_allocate(shape, np.ones((2, 2)), 1.0, 3, 2, 64, 16, 64)                             # r > 1
    assert e.value.code == -1
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_allocate(shape, np.ones((2, 2)), 1.0, 1, 2, 65, 16, 64)                             # not whole pages
    assert e.value.code == -1
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_decode_plan(shape, np.full((2, 2), 64, np.int32), 1, 1, 1, 256)                      # empty range
    assert e.value.code == -1
    L = bk.lib()
    assert L.baklava_decode_attn(None, None, None, None, None, 0, None, None, 0, None, None, None, 0, None) == -1
    assert L.baklava_evict(ctypes.byref(shape), None, 0, 1, None, None, None, 4, 0, 0, 4, 1, None, 0, None) == -1


def test_misaligned_state_arrays_and_odd_strides_are_refused_on_the_host():
    """pos and score are read in 16-byte vectors: a pointer or a sequence stride that breaks that must come
    back as an argument error before anything touches the device (the addresses here are never dereferenced)."""
    shape = bk.make_shape(2, 4, 2, 128)
    info = bk.PlanInfo(4, 4, 4, 256, 0, 2, 1, 1 << 20)
    base = 0x7f0000000000

    def call(pos_off=0, score_off=0, stride=4096, flags=0):
        c = bk.CacheStruct(base, base + (1 << 24), base + (2 << 24) + pos_off, base + (3 << 24) + score_off,
                           base + (4 << 24), base + (5 << 24), base + (6 << 24), base + (7 << 24), stride, 1,
                           base + (8 << 24), bk.KV_BF16, None)
        return bk.lib().baklava_decode_attn(ctypes.byref(shape), ctypes.byref(c), base + (9 << 24), base + (10 << 24),
                                            base + (11 << 24), 5, base + (12 << 24), None, flags, base + (13 << 24),
                                            ctypes.byref(info), base + (14 << 24), 1 << 30, None)
    assert call(pos_off=4) == -1
    assert call(score_off=8) == -1
    assert call(stride=4104) == -1
    assert call(flags=1 << 20) == -1
    assert bk.lib().baklava_set_wait_limit(-5) == -1


def test_search_pick_matches_oracle_rule():
    from oracle import search as osearch
    rng = np.random.default_rng(9)
    cases = [[3.0, 1.0, 2.0, 1.0], [np.nan, 2.0, np.nan, 1.5], [np.inf, np.inf], [], [0.0], [np.nan]]
    cases += [list(rng.integers(0, 4, size=n).astype(float)) for n in (2, 5, 17)]
    for c in cases:
        assert bk.baklava_search_pick(c) == osearch.pick_best(c), c
