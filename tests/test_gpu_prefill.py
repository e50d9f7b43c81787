"""GPU parity of baklava_prefill_scores with the oracle's column sums, and its use as the seed of a bulk eviction."""
import numpy as np
import pytest
import torch

from oracle import eviction as oe
from oracle.prefill import prefill_scores
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth

from harness import assert_close, f64

pytestmark = pytest.mark.gpu


def _run(B, Hq, Hkv, T, D, lens=None, seed=5, q_scale=1.0):
    dev = "cuda"
    shape = bk.make_shape(1, Hq, Hkv, D)
    q = synth.normal_bf16(seed, 1, (B, Hq, T, D), dev, torch.tensor(q_scale))
    k = synth.normal_bf16(seed, 2, (B, Hkv, T, D), dev)
    plen = None if lens is None else torch.tensor(lens, dtype=torch.int32, device=dev)
    score = torch.full((B, Hkv, T), -1.0, dtype=torch.float32, device=dev)
    ws = torch.empty((bk.baklava_prefill_workspace_size(shape, B, T),), dtype=torch.uint8, device=dev)
    bk.baklava_prefill_scores(shape, q, k, plen, B, T, score, ws)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0
    Q, K = f64(q), f64(k)
    g = Hq // Hkv
    got = score.cpu().numpy()
    for b in range(B):
        n = T if lens is None else lens[b]
        for c in range(Hkv):
            ref = prefill_scores(Q[b, c * g:(c + 1) * g, :n], K[b, c, :n])
            assert_close(got[b, c, :n], ref, "scores b%d kv%d" % (b, c))
            assert np.all(got[b, c, n:] == 0.0)
            assert abs(got[b, c].sum() - g * n) <= 1e-3 * g * n          # every row hands out exactly 1 per head
    return q, k, score


@pytest.mark.parametrize("T", [1, 63, 64, 65, 200])
def test_lengths_around_the_tile_size(T):
    _run(B=2, Hq=4, Hkv=2, T=T, D=64)


def test_llama_head_shape_with_prompt_lengths_and_peaked_attention():
    _run(B=3, Hq=8, Hkv=2, T=300, D=128, lens=[300, 129, 1], q_scale=3.0)


def test_many_tiles_wrap_the_rings():
    _run(B=1, Hq=2, Hkv=1, T=1200, D=128, lens=[1170])
    _run(B=1, Hq=2, Hkv=2, T=900, D=64)


def test_group_of_seven():
    _run(B=1, Hq=7, Hkv=1, T=150, D=128)


def test_with_the_rows_normaliser_supplied_one_pass_gives_the_same_scores():
    """The caller's log-sum-exp (here the oracle's own, rounded to fp32) replaces the first pass."""
    from oracle.attention import log_sum_exp
    dev = "cuda"
    B, Hq, Hkv, T, D = 2, 8, 2, 333, 128
    lens = [333, 140]
    shape = bk.make_shape(1, Hq, Hkv, D)
    g = Hq // Hkv
    q = synth.normal_bf16(11, 1, (B, Hq, T, D), dev, torch.tensor(2.0))
    k = synth.normal_bf16(11, 2, (B, Hkv, T, D), dev)
    Q, K = f64(q), f64(k)
    lse = np.full((B, Hq, T), np.nan, dtype=np.float32)            # rows past the prompt must never be read
    for b in range(B):
        for h in range(Hq):
            for i in range(lens[b]):
                lse[b, h, i] = log_sum_exp(Q[b, h, i:i + 1], K[b, h // g, :i + 1])[0]
    plen = torch.tensor(lens, dtype=torch.int32, device=dev)
    ws = torch.empty((bk.baklava_prefill_workspace_size(shape, B, T),), dtype=torch.uint8, device=dev)
    got = []
    for given in (torch.from_numpy(lse).to(dev), None):
        score = torch.full((B, Hkv, T), -1.0, dtype=torch.float32, device=dev)
        bk.baklava_prefill_scores(shape, q, k, plen, B, T, score, ws, lse=given)
        torch.cuda.synchronize()
        assert bk.workspace_error(ws) == 0
        got.append(score.cpu().numpy())
    for b in range(B):
        n = lens[b]
        for c in range(Hkv):
            ref = prefill_scores(Q[b, c * g:(c + 1) * g, :n], K[b, c, :n])
            assert_close(got[0][b, c, :n], ref, "one pass, scores b%d kv%d" % (b, c))
            assert np.all(got[0][b, c, n:] == 0.0)
    np.testing.assert_allclose(got[0], got[1], rtol=2e-3, atol=1e-5)


def test_seeds_a_bulk_eviction_like_the_oracle():
    dev = "cuda"
    B, Hq, Hkv, T, D = 1, 4, 2, 400, 64
    shape = bk.make_shape(1, Hq, Hkv, D)
    q, k, score = _run(B, Hq, Hkv, T, D, seed=9)
    v = synth.normal_bf16(9, 3, (B, Hkv, T, D), dev)
    cap = np.array([[96, 208]], dtype=np.int32)
    cache = bk.Cache(shape, cap, np.array([[0, 96]], dtype=np.int64), 304, B, dev)
    ws = torch.empty((bk.baklava_evict_workspace_size(shape, B, 1, T),), dtype=torch.uint8, device=dev)
    bk.baklava_evict(shape, cache, 0, 1, k, v, score, T, 0, Hkv * T, T, 1, ws)
    torch.cuda.synchronize()
    sc = score.cpu().numpy()
    for h in range(Hkv):
        keep = oe.select_keep(np.arange(T), sc[0, h], int(cap[0, h]) - 1, 4, 1, 2)     # the rule on the library's scores
        lo, _ = cache.rows(0, 0, h)
        np.testing.assert_array_equal(cache.pos[lo:lo + len(keep)].cpu().numpy(), keep)
