"""Seeded random configurations: shapes, group sizes, budgets, policies, chunkings, slab formats and flag
sequences drawn at random, every step of every head compared with the oracle (the harness also checks the
allocation, the slot layout and the selection on the library's own scores)."""
import numpy as np
import pytest

from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl

from harness import Session

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4, 4]))
    g = int(rng.integers(1, 9))
    L = int(rng.integers(1, 4))
    B = int(rng.integers(1, 4))
    T = int(rng.integers(1, 700))
    n_sink = int(rng.choice([0, 1, 4]))
    recent = [(0, 1), (1, 3), (1, 2), (1, 1)][int(rng.integers(0, 4))]
    budget = float(rng.choice([0.1, 0.3, 0.6, 1.2]))
    page = 16
    base_pages = max(int(budget * T / page + 1e-9), -(-(n_sink + 2) // page) + 1)
    base_pages = min(base_pages, -(-(T + 16) // page))          # never above the dense length plus the steps
    w = wl.scaled(wl.TINY, name="random-%d" % seed, L=L, Hq=g * Hkv, Hkv=Hkv, D=D, B=B, T=T,
                  budget=base_pages * page / T + 1e-9, steps=16, n_sink=n_sink, recent_num=recent[0], recent_den=recent[1],
                  importance_sigma=float(rng.choice([0.3, 1.0, 2.0])), seed=wl.MASTER_SEED + 100 + seed,
                  kv_recipe=str(rng.choice(["plain", "channel_lognormal", "outlier", "head_rms"])),
                  r_num=int(rng.integers(1, 4)), r_den=4)
    kv = bk.KV_FP8_E4M3 if (D == 128 and rng.random() < 0.5) else bk.KV_BF16
    chunk = int(rng.choice([0, 64, 128, 320]))
    window_only = recent[0] == recent[1]
    flags = []
    for _ in range(7):
        u = rng.random()
        if u < 0.55:
            flags.append(0)
        elif u < 0.7:
            flags.append(bk.FLAG_NO_APPEND)
        elif u < 0.85:
            flags.append(bk.FLAG_NO_APPEND | bk.FLAG_NO_SCORE)
        else:
            flags.append(bk.FLAG_NO_SCORE if window_only else bk.FLAG_NO_APPEND | bk.FLAG_NO_SCORE | bk.FLAG_NO_EVICT)
    return w, kv, chunk, flags


@pytest.mark.parametrize("seed", range(20))
def test_random_configuration(seed):
    w, kv, chunk, flags = draw(seed)
    assert w.base_pages >= w.min_pages
    s = Session(w, chunk_tokens=chunk, kv_dtype=kv)
    for (b, l, h) in s.heads:
        s.check_state(b, l, h, "after prefill")
    for i, f in enumerate(flags):
        s.step(i, flags=f)
