"""GPU parity of baklava_evict with the oracle's bulk eviction: kept sets, row order, rows and scores
are compared exactly (selection works on the given fp32 scores on both sides)."""
import numpy as np
import pytest
import torch

from oracle import eviction as oe
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth

pytestmark = pytest.mark.gpu


def _run_case(L, Hkv, B, D, T, caps, n_sink, num, den, score_mode, reserve=1, seed=1, pad=0):
    dev = "cuda"
    shape = bk.make_shape(L, Hkv, Hkv, D, 16, n_sink, num, den)
    cap = np.array(caps, dtype=np.int32).reshape(L, Hkv)
    off = np.concatenate([[0], np.cumsum(cap.reshape(-1))[:-1]]).reshape(L, Hkv).astype(np.int64)
    stride = int(cap.sum())
    cache = bk.Cache(shape, cap, off, stride, B, dev)
    Tp = T + pad                                              # head stride larger than T
    k = synth.normal_bf16(seed, 1, (L, B, Hkv, Tp, D), dev)
    v = synth.normal_bf16(seed, 2, (L, B, Hkv, Tp, D), dev)
    if score_mode == "none":
        sc = None
    else:
        sc = synth.uniform_f64(seed, 3, 0, L * B * Hkv * Tp, dev).to(torch.float32).reshape(L, B, Hkv, Tp)
        if score_mode == "ties":
            sc = torch.round(sc * 8) / 8
        if score_mode == "signed":
            sc = sc - 0.5
    ws = torch.empty((bk.baklava_evict_workspace_size(shape, B, L, T),), dtype=torch.uint8, device=dev)
    bk.baklava_evict(shape, cache, 0, L, k, v, sc, T, B * Hkv * Tp, Hkv * Tp, Tp, reserve, ws)
    torch.cuda.synchronize()
    assert int(cache.status.item()) == 0
    kc, vc = k.cpu(), v.cpu()
    scc = None if sc is None else sc.cpu().numpy()
    for l in range(L):
        for b in range(B):
            for h in range(Hkv):
                C = int(cap[l, h])
                s_in = np.zeros(T, np.float32) if scc is None else scc[l, b, h, :T]
                _, _, pos2, s2, idx = oe.bulk_evict(kc[l, b, h, :T].double().numpy(), vc[l, b, h, :T].double().numpy(), np.arange(T), s_in,
                                                    C - reserve, n_sink, num, den)
                n = len(pos2)
                assert int(cache.len[b, l, h]) == n and int(cache.free_slot[b, l, h]) == n
                lo, _ = cache.rows(b, l, h)
                np.testing.assert_array_equal(cache.pos[lo:lo + n].cpu().numpy(), pos2)
                np.testing.assert_array_equal(cache.score[lo:lo + n].cpu().numpy(), s2)
                assert torch.equal(cache.k_slab[lo:lo + n].cpu(), kc[l, b, h][idx])
                assert torch.equal(cache.v_slab[lo:lo + n].cpu(), vc[l, b, h][idx])


@pytest.mark.parametrize("score_mode", ["random", "ties", "none", "signed"])
def test_small_heads(score_mode):
    _run_case(L=2, Hkv=2, B=2, D=64, T=300, caps=[64, 160, 304, 512], n_sink=4, num=1, den=2,
              score_mode=score_mode, pad=4)


def test_window_only_policy_and_no_sinks():
    _run_case(L=1, Hkv=2, B=1, D=128, T=1000, caps=[128, 640], n_sink=4, num=1, den=1, score_mode="random")
    _run_case(L=1, Hkv=2, B=1, D=128, T=1000, caps=[128, 640], n_sink=0, num=0, den=1, score_mode="ties")


def test_long_head_many_scan_blocks_and_reserve():
    _run_case(L=1, Hkv=3, B=1, D=128, T=5000, caps=[16, 2048, 4992], n_sink=4, num=1, den=3,
              score_mode="random", reserve=3, seed=5)


def test_all_rows_fit():
    _run_case(L=1, Hkv=2, B=2, D=64, T=100, caps=[112, 256], n_sink=4, num=1, den=2, score_mode="random")
