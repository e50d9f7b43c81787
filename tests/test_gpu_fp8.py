"""FP8 E4M3 slabs: the quantising bulk eviction and the decode step against the oracle run on the values the
codes stand for.  Codes, positions, kept sets and slots must agree exactly; outputs within the usual tolerance."""
import numpy as np
import pytest
import torch

from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl
from tests.harness import Session

pytestmark = pytest.mark.gpu

W8 = wl.scaled(wl.TINY, name="tiny-d128", D=128)


def test_bulk_evict_quantises_rows_exactly():
    s = Session(W8, kv_dtype=bk.KV_FP8_E4M3)
    for (b, l, h) in s.heads:
        s.check_state(b, l, h, "after bulk evict")


def test_decode_steps_match_oracle_on_dequantised_values():
    s = Session(W8, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(8):
        s.step(i)


@pytest.mark.parametrize("chunk", [64, 128, 192])
def test_chunkings_and_ragged_tails(chunk):
    w = wl.scaled(W8, T=300, budget=0.9)                  # capacities that are no multiple of the 128-token stage
    s = Session(w, chunk_tokens=chunk, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(4):
        s.step(i)


def test_filling_from_empty_then_evicting():
    w = wl.scaled(W8, budget=0.0625, steps=64)             # 32-token base budget
    s = Session(w, prefill=False, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(int(s.cap.max()) + 4):
        s.step(i)


def test_group_of_seven_and_batch():
    w = wl.scaled(W8, Hq=14, Hkv=2, B=3, T=256)
    s = Session(w, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(3):
        s.step(i)


def test_window_only_policy_without_scores():
    w = wl.scaled(W8, recent_num=1, recent_den=1)
    s = Session(w, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(6):
        s.step(i, flags=bk.FLAG_NO_SCORE)


def test_flags_no_append_and_no_evict():
    s = Session(W8, kv_dtype=bk.KV_FP8_E4M3)
    s.step(0)
    s.step(1, flags=bk.FLAG_NO_APPEND)
    s.step(2, flags=bk.FLAG_NO_APPEND | bk.FLAG_NO_SCORE)
    s.step(3)


def test_head_dimension_64_is_refused():
    w = wl.TINY
    with pytest.raises(bk.BaklavaError) as e:
        Session(w, kv_dtype=bk.KV_FP8_E4M3)
    assert e.value.code == -7


def test_saturating_rows_stay_finite():
    # scales far too small for the data: most elements saturate at +-448 and the step still runs and agrees
    s = Session(W8, prefill=False, kv_dtype=bk.KV_FP8_E4M3)
    s.cache.kv_scale_host[...] = np.float32(1e-3)
    s.cache.kv_scale_host[..., 1] = np.float32(1.0) / np.float32(1e-3)
    s.cache.kv_scale_host[..., 3] = np.float32(1.0) / np.float32(1e-3)
    s.cache.kv_scale.copy_(torch.from_numpy(s.cache.kv_scale_host))
    for i in range(3):
        s.step(i)
    st = s.head_state(0, 0, 0)
    rows = st["K"][: st["len"]]
    assert np.isfinite(rows).all() and np.abs(rows).max() == 448.0 * float(np.float32(1e-3))
