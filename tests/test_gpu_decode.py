"""GPU parity of baklava_decode_attn (through the C ABI) with the oracle's decode step.

Free-running: the oracle twin of every checked head evolves from the seeded inputs alone; outputs,
log-normalisers and scores must agree within |d| <= 1e-2 + 1e-2 |ref| (bf16 inputs, fp32
accumulation), positions, rows, lengths and free slots exactly.  In addition the retention rule is
re-run on the library's own fp32 scores and must name the same victim bit for bit."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import workloads as wl

from harness import Session, assert_close, f64

pytestmark = pytest.mark.gpu


def test_tiny_workload_all_heads_all_steps():
    s = Session(wl.TINY)
    for (b, l, h) in s.heads:
        s.check_state(b, l, h, "after prefill")
    for i in range(wl.TINY.steps):
        s.step(i)


@pytest.mark.parametrize("chunk", [64, 192, 0])
def test_llama_shape_many_chunks_and_ragged_tail(chunk):
    w = wl.scaled(wl.LLAMA3_8B_32K, L=2, T=2000, steps=6)           # caps are not multiples of the chunk
    s = Session(w, chunk_tokens=chunk)
    for i in range(w.steps):
        s.step(i)


def test_qwen_shape_group_of_seven_batched():
    w = wl.scaled(wl.QWEN25_7B_8K_B16, L=2, B=3, T=1500, steps=4)
    s = Session(w, chunk_tokens=256)
    for i in range(w.steps):
        s.step(i)


def test_layer_range_launch():
    w = wl.scaled(wl.LLAMA3_8B_32K, L=3, T=700, steps=3)
    s = Session(w, layers=(1, 3), chunk_tokens=128)
    for i in range(w.steps):
        s.step(i)
    assert int(s.cache.len[0, 0].sum()) == 0                         # layer 0 was never touched


@pytest.mark.parametrize("chunk", [64, 0])
def test_one_call_per_layer_overlapping_the_previous_layers_tail(chunk):
    """The layer loop of a model: one call per layer with its own plan and workspace, every call after the first
    flagged as independent of the one before it.  Same results as the oracle, step after step."""
    w = wl.scaled(wl.LLAMA3_8B_32K, L=5, T=2000, steps=6)
    s = Session(w, chunk_tokens=chunk, per_layer=True)
    for i in range(w.steps):
        s.step(i)
    w = wl.scaled(wl.QWEN25_7B_8K_B16, L=3, B=3, T=1500, steps=4)
    s = Session(w, chunk_tokens=chunk, per_layer=True)
    for i in range(w.steps):
        s.step(i)
    w = wl.scaled(wl.LLAMA3_8B_32K, L=3, T=1800, steps=4)             # FP8 slabs through the same layer loop
    s = Session(w, chunk_tokens=chunk, per_layer=True, kv_dtype=bk.KV_FP8_E4M3)
    for i in range(w.steps):
        s.step(i)


def test_window_policy_one_call_per_layer():
    w = wl.scaled(wl.LLAMA3_8B_32K, L=3, T=900, steps=12, recent_num=1, recent_den=1)
    s = Session(w, chunk_tokens=128, per_layer=True)
    for i in range(w.steps):
        s.step(i, flags=bk.FLAG_NO_SCORE)


def test_one_call_per_layer_leaves_the_same_cache_as_one_call_for_all_layers():
    # same chunks either way, so scores, victims and rows agree bit for bit; the outputs are summed over the chunks
    # in an order that depends on how the launch is cut into score pieces, so they may differ in the last place
    w = wl.scaled(wl.LLAMA3_8B_32K, L=4, T=3000, steps=3)
    outs = []
    for per_layer in (False, True):
        s = Session(w, heads=[], chunk_tokens=128, per_layer=per_layer)
        for i in range(w.steps):
            s.step(i, check=False)
        outs.append((s.cache.score.clone(), s.cache.free_slot.clone(), s.cache.pos.clone(), s.cache.k_slab.clone(),
                     s.out.float().clone()))
    assert all(torch.equal(a, b) for a, b in zip(outs[0][:4], outs[1][:4]))
    assert torch.allclose(outs[0][4], outs[1][4], rtol=2 ** -7, atol=1e-4)


def test_filling_from_empty_then_steady_state():
    w = wl.scaled(wl.TINY, T=64, budget=0.5, steps=80)               # capacities of 16 .. 48 tokens
    s = Session(w, prefill=False, chunk_tokens=64)
    for i in range(w.steps):
        s.step(i)
    assert all(tw.length == tw.C - 1 for tw in s.twins.values())


def test_full_budget_reproduces_dense_attention():
    # capacity above everything ever stored: each step is Eq. 4 over the whole history
    w = wl.scaled(wl.LLAMA3_8B_32K, L=1, Hq=8, Hkv=2, T=500, steps=5)
    s = Session(w, chunk_tokens=128, caps=[512, 528])
    hist = {}
    for (b, l, h) in s.heads:
        k, v = wl.dense_kv(w, l, b, h, s.scales)
        hist[(b, l, h)] = [f64(k), f64(v)]
    for i in range(w.steps):
        q, kn, vn = wl.decode_inputs(w, i, s.scales)
        s.step(i)
        out = f64(s.out)
        for (b, l, h) in s.heads:
            K = np.vstack([hist[(b, l, h)][0], f64(kn)[l, b, h][None]])
            V = np.vstack([hist[(b, l, h)][1], f64(vn)[l, b, h][None]])
            hist[(b, l, h)] = [K, V]
            ref, _ = oa.decode_attention(f64(q)[l, b, h * w.g:(h + 1) * w.g], K, V)
            assert_close(out[l, b, h * w.g:(h + 1) * w.g], ref, "dense step %d" % i)


@pytest.mark.parametrize("Hq,Hkv,D", [(2, 2, 64), (16, 2, 128), (6, 2, 64)])
def test_group_sizes(Hq, Hkv, D):
    w = wl.scaled(wl.TINY, Hq=Hq, Hkv=Hkv, D=D, T=300, steps=3)
    s = Session(w, chunk_tokens=64)
    for i in range(w.steps):
        s.step(i)


def test_flags():
    w = wl.scaled(wl.TINY, T=200, steps=4)
    s = Session(w, chunk_tokens=64)
    s.step(0)                                                        # every head is full now: a hole exists
    assert any(tw.free_slot < tw.length for tw in s.twins.values())
    s.step(1, flags=bk.FLAG_NO_APPEND)                               # attention skips the hole, scores move
    s.step(1, flags=bk.FLAG_NO_APPEND | bk.FLAG_NO_SCORE)            # nothing moves
    s.step(2, flags=bk.FLAG_NO_SCORE)                                # append without scoring or evicting
    assert all(tw.length == tw.C for tw in s.twins.values())


def test_window_only_policy_without_scores():
    """The paper's evaluated policy (sinks + recent window): with NO_SCORE the library keeps no scores and
    still evicts, by position.  Checked against the oracle and against the closed form of what must remain."""
    w = wl.scaled(wl.LLAMA3_8B_32K, L=2, T=900, steps=40, recent_num=1, recent_den=1)
    s = Session(w, chunk_tokens=128)
    score_before = s.cache.score.clone()
    for i in range(w.steps):
        s.step(i, flags=bk.FLAG_NO_SCORE)
    assert torch.equal(score_before[s.cache.pos.ne(-1) & (s.cache.pos < w.T)],
                       s.cache.score[s.cache.pos.ne(-1) & (s.cache.pos < w.T)])      # old rows' scores untouched
    t_last = w.T + w.steps - 1
    for (b, l, h) in s.heads:
        st = s.head_state(b, l, h)
        kept = sorted(st["pos"][s.valid_slots(st)])
        R = int(s.cap[l, h]) - 1
        if t_last + 1 <= R:
            assert kept == list(range(t_last + 1))
        else:
            assert kept == list(range(w.n_sink)) + list(range(t_last + 1 - (R - w.n_sink), t_last + 1))
    # filling an empty cache under the same policy
    w2 = wl.scaled(wl.TINY, T=64, steps=70, recent_num=1, recent_den=1)
    s2 = Session(w2, prefill=False, chunk_tokens=64)
    for i in range(w2.steps):
        s2.step(i, flags=bk.FLAG_NO_SCORE)
    assert all(tw.length == tw.C - 1 for tw in s2.twins.values())


def test_overflow_sets_status_and_keeps_state():
    w = wl.scaled(wl.TINY, T=200, steps=4)
    s = Session(w, chunk_tokens=64)
    s.step(0, flags=bk.FLAG_NO_EVICT)                                # caches are now full (len == cap)
    before = s.cache.len.clone()
    q, kn, vn = wl.decode_inputs(w, 1, s.scales, "cuda")
    bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, s.t, s.out, s.lse, 0, s.plan, s.ws)
    torch.cuda.synchronize()
    assert int(s.cache.status.item()) & bk.STATUS_OVERFLOW
    assert torch.equal(before, s.cache.len)
    # the output is still the attention over the rows that are there
    for (b, l, h) in s.heads[:2]:
        tw = s.twins[(b, l, h)]
        ref, _, _ = tw.step(f64(q)[l, b, h * w.g:(h + 1) * w.g], None, None, 0, append=False, update_score=False)
        assert_close(f64(s.out)[l, b, h * w.g:(h + 1) * w.g], ref, "overflow step output")


def test_empty_cache_without_append():
    w = wl.scaled(wl.TINY, T=64)
    s = Session(w, prefill=False)
    s.out.fill_(1.0)
    s.step(0, flags=bk.FLAG_NO_APPEND)
    assert torch.all(s.out == 0) and torch.all(torch.isneginf(s.lse))


def test_repeatable_bit_for_bit():
    w = wl.scaled(wl.LLAMA3_8B_32K, L=2, T=3000, steps=3)
    outs = []
    for _ in range(2):
        s = Session(w, heads=[], chunk_tokens=128)
        for i in range(w.steps):
            s.step(i, check=False)
        outs.append((s.out.clone(), s.cache.score.clone(), s.cache.free_slot.clone()))
    assert all(torch.equal(a, b) for a, b in zip(outs[0], outs[1]))


def test_workspace_too_small_and_bad_pointers_are_refused():
    w = wl.scaled(wl.TINY, T=64)
    s = Session(w, prefill=False)
    q, kn, vn = wl.decode_inputs(w, 0, s.scales, "cuda")
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, 0, s.out, s.lse, 0, s.plan, s.ws[:256])
    assert e.value.code == -4
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_decode_attn(s.shape, s.cache, q.view(-1)[1:], kn, vn, 0, s.out, s.lse, 0, s.plan, s.ws)
    assert e.value.code == -1
    with pytest.raises(bk.BaklavaError) as e:
        bk.baklava_decode_attn(s.shape, s.cache, q, kn, vn, 0, s.out, s.lse, 64, s.plan, s.ws)
    assert e.value.code == -1
