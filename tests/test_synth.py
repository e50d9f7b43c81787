"""The seeded generator: reproducible, sliceable, and shaped like the distributions it stands for."""
import torch

from paper_2502_13176_b200 import synth, workloads as wl


def test_slices_regenerate_identically():
    full = synth.normal_f32(7, 3, 0, 5000)
    part = synth.normal_f32(7, 3, 1234, 100)
    assert torch.equal(full[1234:1334], part)
    assert not torch.equal(full, synth.normal_f32(8, 3, 0, 5000))
    assert not torch.equal(full, synth.normal_f32(7, 4, 0, 5000))


def test_matches_the_definition_in_plain_integers():
    key = synth.stream_key(11, 5)
    z = synth.normal_f32(11, 5, 0, 64)
    for i in (0, 1, 63):
        total = 0
        for j in range(3):
            w = synth._mix_int(key + synth._GOLDEN * (3 * i + j + 1))
            total += sum((w >> (16 * f)) & 0xFFFF for f in range(4))
        assert z[i].item() == (total - 6 * 65535) / 65536.0


def test_moments():
    z = synth.normal_f32(1, 1, 0, 1 << 20).double()
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3
    assert abs((z ** 4).mean() - 3.0) < 0.15
    u = synth.uniform_f64(1, 2, 0, 1 << 16)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 5e-3


def test_workload_slices_agree_with_layer_tensor():
    w = wl.scaled(wl.TINY, T=64)
    sc = wl.kv_scales(w)
    kl, vl = wl.dense_kv_layer(w, 1, sc)
    k, v = wl.dense_kv(w, 1, 0, 1, sc)
    assert torch.equal(kl[0, 1], k) and torch.equal(vl[0, 1], v)
    q, kn, vn = wl.decode_inputs(w, 3, sc)
    q1, kn1, vn1 = wl.decode_inputs(w, 3, sc, layers=(1, 2))
    assert torch.equal(q[1:2], q1) and torch.equal(kn[1:2], kn1) and torch.equal(vn[1:2], vn1)


def test_recipes():
    ks, vs = wl.kv_scales(wl.LLAMA3_8B_32K)
    assert ks.shape == (32, 8, 128) and torch.all((ks == 8).sum(-1) == 1) and torch.equal(ks, vs)
    ks, vs = wl.kv_scales(wl.QWEN25_7B_8K_B16)
    assert ks.min() >= 0.5 and ks.max() <= 2.0 and torch.all(ks[..., 0] == ks[..., 5])
    assert wl.LLAMA3_8B_32K.base_pages == 614 and wl.LLAMA3_8B_32K.total_pages == 157184
    assert wl.QWEN25_7B_8K_B16.base_pages == 153 and wl.TINY.total_pages == 64
    assert wl.LLAMA3_8B_32K.max_pages == 2052
    I = wl.importance(wl.LLAMA3_8B_32K)
    assert I.shape == (32, 8) and I.min() > 0
