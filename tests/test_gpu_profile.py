"""GPU parity of baklava_profile_heads (Algorithm 1, step 1) with the oracle, and the host step 2 on top."""
import numpy as np
import pytest
import torch

from oracle import profiling as op
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import synth

from harness import assert_close, f64

pytestmark = pytest.mark.gpu


def _run(P, Hq, Hkv, T, D, lens=None, seed=3, want_tokens=True, v=None, k_edit=None):
    dev = "cuda"
    shape = bk.make_shape(1, Hq, Hkv, D)
    q = synth.normal_bf16(seed, 1, (P, Hq, T, D), dev)
    k = synth.normal_bf16(seed, 2, (P, Hkv, T, D), dev)
    if k_edit is not None:
        k = k_edit(k)
    if v is None:
        v = synth.normal_bf16(seed, 3, (P, Hkv, T, D), dev)
    plen = None if lens is None else torch.tensor(lens, dtype=torch.int32, device=dev)
    head_cos = torch.full((P, Hq), 7.0, dtype=torch.float32, device=dev)
    tok = torch.full((P, Hq, T), 7.0, dtype=torch.float32, device=dev) if want_tokens else None
    ws = torch.empty((bk.baklava_profile_workspace_size(shape, P, T),), dtype=torch.uint8, device=dev)
    bk.baklava_profile_heads(shape, q, k, v, plen, P, T, head_cos, tok, ws)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0
    Q, K, V = f64(q), f64(k), f64(v)
    g = Hq // Hkv
    for p in range(P):
        n = T if lens is None else lens[p]
        for h in range(Hq):
            s_ref, c_ref = op.head_similarity(Q[p, h], K[p, h // g], V[p, h // g], n)
            assert abs(float(head_cos[p, h]) - s_ref) <= 1e-3, (p, h, float(head_cos[p, h]), s_ref)
            if want_tokens:
                assert_close(tok[p, h, :n].cpu().numpy(), c_ref, "token cosines p%d h%d" % (p, h))
                assert torch.all(tok[p, h, n:] == 7.0)              # rows past the prompt are untouched
    return head_cos.cpu().numpy()


@pytest.mark.parametrize("T", [1, 63, 64, 65, 200])
def test_lengths_around_the_tile_size(T):
    _run(P=2, Hq=4, Hkv=2, T=T, D=64)


def test_llama_head_shape_and_prompt_lengths():
    _run(P=3, Hq=8, Hkv=2, T=300, D=128, lens=[300, 129, 1])


def test_many_key_tiles_wrap_the_rings():
    # ten 128-key tiles per row block: every stage, accumulator and probability buffer is reused several times
    _run(P=1, Hq=2, Hkv=1, T=1200, D=128, want_tokens=True, lens=[1170])
    _run(P=1, Hq=2, Hkv=2, T=900, D=64, want_tokens=False)


def test_key_far_above_the_first_tile_stays_in_range():
    # logits of one late key tower over everything in the first key tile, but by less than the fp32 range:
    # the one-pass kernel's probabilities exceed 1 there and the cosines must still come out right
    def edit(k):
        k = k.clone()
        k[:, :, 300] *= 12.0
        return k
    _run(P=1, Hq=4, Hkv=2, T=520, D=128, k_edit=edit)


def test_key_beyond_the_range_is_redone_exactly():
    # here the gap is hundreds of octaves: the one-pass kernel overflows on the rows that see the key, flags
    # their row blocks, and the exact two-pass kernel redoes them; rows before the key are finished in one pass
    def edit(k):
        k = k.clone()
        k[:, :, 400] *= 300.0
        return k
    _run(P=2, Hq=4, Hkv=2, T=650, D=128, k_edit=edit, lens=[650, 500])
    _run(P=1, Hq=2, Hkv=1, T=300, D=64, k_edit=edit if False else (lambda k: torch.cat([k[:, :, :200], k[:, :, 200:] * 250.0], dim=2)))


def test_rows_on_both_sides_of_the_range_limit():
    # a late key whose logits reach a few hundred octaves for some rows and stay small for others: some rows of a
    # block overflow (the block is redone exactly), others would have been fine either way
    def edit(k):
        k = k.clone()
        k[:, :, 200] *= 40.0
        return k
    _run(P=2, Hq=4, Hkv=2, T=400, D=128, k_edit=edit)
    _run(P=1, Hq=2, Hkv=1, T=300, D=64, k_edit=edit)


def test_group_of_seven():
    _run(P=1, Hq=7, Hkv=1, T=150, D=128, want_tokens=False)


def test_identical_value_rows_give_one():
    dev = "cuda"
    row = synth.normal_bf16(9, 1, (1, 1, 1, 64), dev)
    s = _run(P=1, Hq=2, Hkv=1, T=130, D=64, v=row.expand(1, 1, 130, 64).contiguous())
    np.testing.assert_allclose(s, 1.0, atol=1e-3)


def test_importance_from_profile_matches_oracle_end_to_end():
    dev = "cuda"
    P, L, Hq, Hkv, T, D = 2, 2, 4, 2, 96, 64
    shape = bk.make_shape(L, Hq, Hkv, D)
    s_dev = np.zeros((P, L, Hq), dtype=np.float32)
    s_ref = np.zeros((P, L, Hq))
    ws = torch.empty((bk.baklava_profile_workspace_size(shape, P, T),), dtype=torch.uint8, device=dev)
    for l in range(L):
        q = synth.normal_bf16(20 + l, 1, (P, Hq, T, D), dev)
        k = synth.normal_bf16(20 + l, 2, (P, Hkv, T, D), dev)
        v = synth.normal_bf16(20 + l, 3, (P, Hkv, T, D), dev)
        hc = torch.empty((P, Hq), dtype=torch.float32, device=dev)
        bk.baklava_profile_heads(shape, q, k, v, None, P, T, hc, None, ws)
        torch.cuda.synchronize()
        s_dev[:, l] = hc.cpu().numpy()
        s_ref[:, l] = op.profile_heads(f64(q), f64(k), f64(v))
    got = bk.baklava_importance(shape, s_dev)
    np.testing.assert_allclose(got, op.kv_importance(s_ref, Hq // Hkv), atol=1e-3)


def test_profile_to_budgets_chain_at_four_total_budgets():
    """The whole one-time pass of the method in small: profile every layer over the prompts (device), reduce to
    KV-cache importance (host), allocate at 10 / 30 / 50 / 70 % of dense (host) -- against the oracle's chain."""
    from oracle import allocation as oalloc
    dev = "cuda"
    P, L, Hq, Hkv, T, D, page = 4, 3, 8, 2, 256, 128, 16
    shape = bk.make_shape(L, Hq, Hkv, D)
    s_dev = np.zeros((P, L, Hq), dtype=np.float32)
    s_ref = np.zeros((P, L, Hq))
    ws = torch.empty((bk.baklava_profile_workspace_size(shape, P, T),), dtype=torch.uint8, device=dev)
    for l in range(L):
        q = synth.normal_bf16(40 + l, 1, (P, Hq, T, D), dev)
        k = synth.normal_bf16(40 + l, 2, (P, Hkv, T, D), dev)
        # heads differ: some value rows share a common direction, so their outputs resemble their inputs more
        v = synth.normal_bf16(40 + l, 3, (P, Hkv, T, D), dev)
        common = synth.normal_bf16(40 + l, 4, (1, Hkv, 1, D), dev).float()
        mix = torch.tensor([0.0, 1.5], device=dev).reshape(1, Hkv, 1, 1) * (l + 1)
        v = (v.float() + mix * common).to(torch.bfloat16)
        hc = torch.empty((P, Hq), dtype=torch.float32, device=dev)
        bk.baklava_profile_heads(shape, q, k, v, None, P, T, hc, None, ws)
        torch.cuda.synchronize()
        s_dev[:, l] = hc.cpu().numpy()
        s_ref[:, l] = op.profile_heads(f64(q), f64(k), f64(v))
    imp_dev = bk.baklava_importance(shape, s_dev)
    imp_ref = op.kv_importance(s_ref, Hq // Hkv)
    np.testing.assert_allclose(imp_dev, imp_ref, atol=1e-3)
    assert imp_ref.max() - imp_ref.min() > 0.05                     # the heads really differ
    t = float(np.median(imp_ref))
    for pct in (10, 30, 50, 70):
        base_pages = max(1, T * pct // 100 // page)
        total = base_pages * L * Hkv * page
        cap, off, stride = bk.baklava_allocate(shape, imp_dev, t, 1, 2, total, page, (T // page) * page)
        # the host code on the device's importances = the oracle's rule on the same numbers, bit for bit
        ocap, ooff, ostride = oalloc.allocate(imp_dev, t, 1, 2, base_pages * L * Hkv, 1, T // page, page)
        np.testing.assert_array_equal(cap, ocap)
        np.testing.assert_array_equal(off, ooff)
        assert stride == ostride == total
        # and, unless an importance sits within the fp32 noise of the threshold, the oracle's own chain agrees
        if np.abs(imp_ref - t).min() > 2e-3:
            rcap, _, _ = oalloc.allocate(imp_ref, t, 1, 2, base_pages * L * Hkv, 1, T // page, page)
            np.testing.assert_array_equal(cap, rcap)
