"""Parity at the depth the configurations state: every decode step of the Llama-shaped (64) and Qwen-shaped
(128) workloads at full size and in the benchmark's launch configuration, heads of a 131 072-token context, and
the prompt-side kernels at the profiling configuration's prompt length.

Long runs are teacher-forced (the oracle restarts every step from the state the device held before it), so
that each step is judged on its own and a legitimate near tie cannot derail the run; a few heads are followed
free-running as well.  Victims that differ from the oracle's are accepted only as near ties (see
harness.Session._settle_victim), counted and printed.  Inputs are generated on the device; only the sampled
heads travel to the host."""
import numpy as np
import pytest
import torch

from oracle import profiling as op
from oracle.prefill import prefill_scores
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth
from paper_2502_13176_b200 import workloads as wl

from harness import Session, assert_close, f64

pytestmark = pytest.mark.gpu


def _caps_of(w):
    s = Session(w, heads=[], prefill=False)
    return s.cap


def _sample(w, cap, count, sequences=(0,)):
    """`count` heads including the smallest, the largest and the median capacity, spread over `sequences`."""
    flat = sorted((int(cap[l, h]), l, h) for l in range(w.L) for h in range(w.Hkv))
    picks = [flat[0], flat[-1], flat[len(flat) // 2]]
    rng = np.random.default_rng(w.seed)
    for i in rng.permutation(len(flat)):
        if len(picks) >= count:
            break
        if flat[int(i)] not in picks:
            picks.append(flat[int(i)])
    return [(sequences[j % len(sequences)], l, h) for j, (_, l, h) in enumerate(picks)]


def _report(s, what):
    print("%s: %d near ties settled%s" % (what, len(s.near_ties),
                                         "".join("\n  %s gap %.3e" % nt for nt in s.near_ties[:8])))


@pytest.mark.parametrize("kv,n_teacher,n_free,all_heads_at", [(bk.KV_BF16, 16, 3, (0, 1, 63)), (bk.KV_FP8_E4M3, 8, 0, (63,))],
                         ids=["bf16", "fp8"])
def test_llama_32k_all_64_steps(kv, n_teacher, n_free, all_heads_at):
    w = wl.LLAMA3_8B_32K
    cap = _caps_of(w)
    teacher = _sample(w, cap, n_teacher)
    s = Session(w, heads=teacher[:n_free], kv_dtype=kv)
    everyone = [(0, l, h) for l in range(w.L) for h in range(w.Hkv)]
    hold = set(teacher)
    for i in range(w.steps):
        if i in all_heads_at:
            s.step(i, teacher=everyone, hold=hold)
        else:
            s.step(i, teacher=teacher, hold=hold)
    s.check_held_rows()
    _report(s, "llama 32K %s" % ("fp8" if kv else "bf16"))
    assert len(s.near_ties) <= 0.01 * w.steps * (n_teacher + n_free) + 4
    expect = np.minimum(s.cap[None] - 1, w.T + w.steps)
    np.testing.assert_array_equal(s.cache.len.cpu().numpy(), np.broadcast_to(expect, (w.B, w.L, w.Hkv)))


def test_qwen_8k_batch16_all_128_steps():
    w = wl.QWEN25_7B_8K_B16
    cap = _caps_of(w)
    teacher = _sample(w, cap, 12, sequences=(0, w.B - 1))
    s = Session(w, heads=teacher[:2])
    for i in range(w.steps):
        s.step(i, teacher=teacher)
    s.check_held_rows()
    _report(s, "qwen 8K x 16")
    assert len(s.near_ties) <= 0.01 * w.steps * 14 + 4
    expect = np.minimum(s.cap[None] - 1, w.T + w.steps)
    np.testing.assert_array_equal(s.cache.len.cpu().numpy(), np.broadcast_to(expect, (w.B, w.L, w.Hkv)))


def test_llama_32k_one_call_per_layer():
    """The full-size Llama workload issued layer by layer (32 calls per step, each after the first overlapping the
    tail of the one before it), all heads checked at the first and the last step."""
    w = wl.scaled(wl.LLAMA3_8B_32K, steps=12)
    cap = _caps_of(w)
    teacher = _sample(w, cap, 12)
    s = Session(w, heads=teacher[:2], per_layer=True)
    everyone = [(0, l, h) for l in range(w.L) for h in range(w.Hkv)]
    for i in range(w.steps):
        s.step(i, teacher=everyone if i in (0, w.steps - 1) else teacher, hold=set(teacher))
    s.check_held_rows()
    _report(s, "llama 32K, one call per layer")


def test_heads_of_a_131072_token_context():
    # two layers of the sweep's longest point: 90 % of a 128K context, heads of 59K .. 177K rows, tens of chunks each
    w = wl.scaled(wl.sweep_point(1, 131072, 0.9), L=2, steps=4)
    s = Session(w, heads=[])
    assert int(s.cap.max()) > 100000 and s.plan.info.n_items > 16 * 20
    teacher = _sample(w, s.cap, 5)
    for i in range(w.steps):
        s.step(i, teacher=teacher)
    s.check_held_rows()
    _report(s, "128K context")


# ---------------------------------------------------------------- prompt side at the profiling configuration's length
def test_profile_heads_at_4096_tokens():
    """Eight full (prompt, head) instances of the profiling workload (4096-token prompts, Llama head shape),
    head means and every token's cosine."""
    w = wl.LLAMA3_8B_32K
    dev, T, P = "cuda", 4096, 2
    shape = bk.make_shape(1, w.Hq, w.Hkv, w.D)
    parts = [wl.profile_inputs(w, p, 0, T, dev) for p in range(P)]
    q = torch.stack([x[0] for x in parts]); k = torch.stack([x[1] for x in parts]); v = torch.stack([x[2] for x in parts])
    head_cos = torch.empty((P, w.Hq), dtype=torch.float32, device=dev)
    tok = torch.empty((P, w.Hq, T), dtype=torch.float32, device=dev)
    ws = torch.empty((bk.baklava_profile_workspace_size(shape, P, T),), dtype=torch.uint8, device=dev)
    bk.baklava_profile_heads(shape, q, k, v, None, P, T, head_cos, tok, ws)
    torch.cuda.synchronize()
    assert bk.workspace_error(ws) == 0
    for (p, h) in [(0, 0), (0, 5), (0, 17), (0, 31), (1, 2), (1, 12), (1, 22), (1, 29)]:
        c = h // w.g
        s_ref, c_ref = op.head_similarity(f64(q[p, h]), f64(k[p, c]), f64(v[p, c]), T)
        assert abs(float(head_cos[p, h]) - s_ref) <= 1e-3, (p, h)
        assert_close(tok[p, h].cpu().numpy(), c_ref, "token cosines p%d h%d" % (p, h))


def test_prefill_scores_at_8192_tokens():
    """One KV group (four query heads) of an 8192-token prompt against the oracle's column sums."""
    w = wl.LLAMA3_8B_32K
    dev, T, B = "cuda", 8192, 1
    shape = bk.make_shape(1, w.Hq, w.Hkv, w.D)
    q = synth.normal_bf16(w.seed, wl.T_PROFILE_Q, (B, w.Hq, T, w.D), dev)
    k = synth.normal_bf16(w.seed, wl.T_PROFILE_K, (B, w.Hkv, T, w.D), dev)
    score = torch.empty((B, w.Hkv, T), dtype=torch.float32, device=dev)
    ws = torch.empty((bk.baklava_prefill_workspace_size(shape, B, T),), dtype=torch.uint8, device=dev)
    bk.baklava_prefill_scores(shape, q, k, None, B, T, score, ws)
    torch.cuda.synchronize()
    assert bk.workspace_error(ws) == 0
    got = score.cpu().numpy()
    for c in (5,):
        ref = prefill_scores(f64(q[0, c * w.g:(c + 1) * w.g]), f64(k[0, c]))
        assert_close(got[0, c], ref, "scores kv%d" % c)
    assert np.all(np.abs(got.sum(axis=2) - w.g * T) <= 1e-3 * w.g * T)
