"""Parity at the benchmark's full sizes and launch configuration (one call per step over all layers,
automatic chunking): the oracle follows a handful of sampled heads, chosen to include the largest and
the smallest capacities, from the seeded inputs alone."""
import numpy as np
import pytest

from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl

from harness import Session

pytestmark = pytest.mark.gpu


def _sampled_heads(s, count):
    w = s.w
    flat = [(int(s.cap[l, h]), l, h) for l in range(w.L) for h in range(w.Hkv)]
    flat.sort()
    picks = [flat[0], flat[-1], flat[len(flat) // 2]]
    rng = np.random.default_rng(w.seed)
    for i in rng.choice(len(flat), count - len(picks), replace=False):
        picks.append(flat[int(i)])
    heads = []
    for j, (_, l, h) in enumerate(picks):
        heads.append((j % w.B, l, h))
    return sorted(set(heads))


@pytest.mark.parametrize("w,steps,count,kv", [(wl.LLAMA3_8B_32K, 3, 6, bk.KV_BF16), (wl.QWEN25_7B_8K_B16, 2, 6, bk.KV_BF16),
                                             (wl.LLAMA3_8B_32K, 2, 4, bk.KV_FP8_E4M3)],
                         ids=["llama3-8b-32k", "qwen2.5-7b-8k-b16", "llama3-8b-32k-fp8"])
def test_full_workload_sampled_heads(w, steps, count, kv):
    probe = Session(w, heads=[], prefill=False)            # capacities only, to choose the sample
    heads = _sampled_heads(probe, count)
    del probe
    s = Session(w, heads=heads, kv_dtype=kv)
    assert int(s.cap.max()) > 2 * int(s.cap.min())          # the budgets really are ragged
    for (b, l, h) in heads:
        s.check_state(b, l, h, "after prefill")
    for i in range(steps):
        s.step(i)
    # every head of the workload, not only the sampled ones, holds what its budget allows
    expect = np.minimum(s.cap[None] - 1, w.T + steps)
    np.testing.assert_array_equal(s.cache.len.cpu().numpy(), np.broadcast_to(expect, (w.B, w.L, w.Hkv)))
