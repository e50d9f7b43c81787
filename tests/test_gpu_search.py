"""Algorithm 3 on the device: the loss kernel against its definition, and the whole search (allocate,
make cache, decode the chunks, loss, pick) against the same loop run with the oracle's pieces."""
import numpy as np
import pytest
import torch

from oracle import allocation as oalloc
from oracle import eviction as oevict
from oracle import search as osearch
from oracle.cache import HeadCache
from paper_2502_13176_b200 import binding as bk
from paper_2502_13176_b200 import search as gsearch
from paper_2502_13176_b200 import synth
from paper_2502_13176_b200 import workloads as wl
from tests.harness import f64

pytestmark = pytest.mark.gpu


def device_loss(out, ref):
    loss = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    rows = out.numel() // out.shape[-1]
    ws = torch.empty((max(4, bk.baklava_output_error_workspace_size(rows)),), dtype=torch.uint8, device="cuda")
    bk.baklava_output_error(out, ref, loss, ws)
    torch.cuda.synchronize()
    return float(loss.item())


@pytest.mark.parametrize("rows,D", [(1, 64), (8, 128), (1037, 128), (4099, 64), (100000, 128)])
def test_output_error_matches_definition(rows, D):
    ref = synth.normal_bf16(11, 60, (rows, D), "cuda")
    noise = synth.normal_bf16(11, 61, (rows, D), "cuda")
    out = (ref.float() + 0.25 * noise.float()).to(torch.bfloat16)
    got = device_loss(out, ref)
    want = osearch.output_error(f64(out), f64(ref))
    assert abs(got - want) <= 1e-5 * want


def test_output_error_special_cases():
    ref = synth.normal_bf16(12, 60, (300, 128), "cuda")
    assert device_loss(ref, ref) == 0.0
    assert abs(device_loss(torch.zeros_like(ref), ref) - 1.0) < 1e-6
    assert abs(device_loss((-ref.float()).to(torch.bfloat16), ref) - 4.0) < 1e-5
    zero = torch.zeros((5, 64), dtype=torch.bfloat16, device="cuda")
    assert device_loss(zero, zero) == 0.0
    empty = torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda")
    assert device_loss(empty, empty) == 0.0


def oracle_chunk_outputs(w, data, cap, steps, scales):
    """Outputs [steps, L, B, Hq, D] of the oracle's budgeted caches on one chunk."""
    g = w.g
    outs = np.zeros((steps, w.L, w.B, w.Hq, w.D))
    feeds = [tuple(f64(x) for x in wl.decode_inputs(data, i, scales)) for i in range(steps)]
    for l in range(w.L):
        sc_l = wl.prefill_scores(data, l)
        for b in range(w.B):
            for h in range(w.Hkv):
                C = int(cap[l, h])
                k, v = wl.dense_kv(data, l, b, h, scales)
                K2, V2, pos2, s2, _ = oevict.bulk_evict(f64(k), f64(v), np.arange(w.T), f64(sc_l[b, h]), C - 1,
                                                       w.n_sink, w.recent_num, w.recent_den)
                hc = HeadCache(C, w.D, w.n_sink, w.recent_num, w.recent_den)
                hc.load(K2, V2, pos2, s2)
                for i in range(steps):
                    q, kn, vn = feeds[i]
                    o, _, _ = hc.step(q[l, b, h * g:(h + 1) * g], kn[l, b, h], vn[l, b, h], w.T + i)
                    outs[i, l, b, h * g:(h + 1) * g] = o
    return outs


def test_search_matches_the_oracle_loop():
    w = wl.TINY
    steps, chunks = 6, 2
    configs = [(t, rn, rd) for t in (0.6, 1.0, 1.8) for (rn, rd) in ((0, 1), (1, 2), (3, 4))]
    res = gsearch.parameter_search(w, configs, chunks=chunks, steps=steps)

    imp = wl.importance(w).numpy()
    scales = wl.kv_scales(w)
    dense_cap = np.full((w.L, w.Hkv), -(-(w.T + steps + 1) // w.page) * w.page)
    refs = [oracle_chunk_outputs(w, gsearch.chunk_workload(w, c), dense_cap, steps, scales) for c in range(chunks)]

    def make_cache(params):
        t, rn, rd = params
        cap, _, _ = oalloc.allocate(imp, t, rn, rd, w.total_pages, w.min_pages, w.max_pages, w.page)
        return cap

    def evaluate(cap, c):
        outs = oracle_chunk_outputs(w, gsearch.chunk_workload(w, c), cap, steps, scales)
        return osearch.output_error(outs.reshape(-1, w.D), refs[c].reshape(-1, w.D))

    best, averages = osearch.parameter_search(configs, list(range(chunks)), make_cache, evaluate)
    got = [row["loss"] for row in res["candidates"]]
    for (cfg, a, b) in zip(configs, got, averages):
        # the device rounds its outputs to bf16 (2^-9 relative per element) before the loss sees them
        assert abs(a - b) <= 2e-2 * b + 1e-4, "loss of %s: device %.6f oracle %.6f" % (cfg, a, b)
    # r = 0 moves nothing, so its loss does not depend on t
    assert got[0] == got[3] == got[6]
    order = np.argsort(averages)
    if averages[order[1]] - averages[order[0]] > 4e-2 * averages[order[0]]:       # a clear winner must be found
        assert (res["best"]["t"], res["best"]["r"]) == (best[0], "%d/%d" % (best[1], best[2]))
    # the reported winner is the rule applied to the device's own losses
    assert res["best"]["loss"] == got[osearch.pick_best(got)]
