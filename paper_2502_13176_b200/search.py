"""Algorithm 3 (parameter search over the threshold t and the reduction r) on synthetic data.

    python -m paper_2502_13176_b200.search [--workload tiny|llama-small] [--t 0.5,1,2] [--r 1/4,1/2,3/4]
                                           [--chunks 2] [--steps 16]

The paper scores a candidate (t, r) by a model's perplexity on evaluation chunks.  There is no
model here, so the loss is the one the attention path can give by itself: the relative squared
distance of the budgeted cache's attention outputs from the dense cache's (baklava_output_error),
averaged over the chunks.  Each chunk is another seeded prompt through the same heads (same
importances, same channel scales).  The loop is the paper's: for every candidate make the cache,
evaluate every chunk from a reset cache, average, keep the first strictly smallest average.

Call sequencing and buffers only: allocation, bulk eviction, decode steps, the loss and the
selection all run inside libbaklava.so.
"""
import argparse
import json
import sys

import numpy as np
import torch

from . import binding as bk
from . import workloads as wl
from .engine import DecodeSession


def chunk_workload(w, c):
    """The c-th evaluation chunk: the same shapes and heads, another prompt."""
    return wl.scaled(w, seed=w.seed + 1000 * (c + 1))


def run_chunk(sess, w, data, steps, outs):
    """RESET_CACHE, MAKE_CACHE from the chunk's dense prompt, then `steps` decode steps; the outputs of
    all steps land in `outs` [steps, layers, B, Hq, D]."""
    sess.cache.reset()
    sess.prefill_synthetic(data=data)
    for i in range(steps):
        q, kn, vn = wl.decode_inputs(data, i, sess.scales, sess.device)
        outs[i].copy_(sess.step(q, kn, vn))
    sess.check_status()


def dense_reference(w, chunks, steps, device, importance):
    """Attention outputs of the dense cache (every head holds the whole context) for every chunk."""
    pages = -(-(w.T + steps + 1) // w.page)
    dense = wl.scaled(w, steps=steps + 1 + w.page)
    sess = DecodeSession(dense, device, uniform=True, importance=importance,
                         total_tokens=pages * w.page * w.L * w.Hkv)
    refs = []
    for c in range(chunks):
        outs = torch.empty((steps,) + tuple(sess.out.shape), dtype=torch.bfloat16, device=device)
        run_chunk(sess, w, chunk_workload(w, c), steps, outs)
        refs.append(outs)
    return refs


def parameter_search(w, configs, chunks=2, steps=16, device="cuda", importance=None):
    """Algorithm 3.  configs: list of (t, r_num, r_den).  Returns a dict with every candidate's average
    loss, the capacities' spread, and the winner."""
    device = torch.device(device)
    importance = wl.importance(w).numpy() if importance is None else importance
    refs = dense_reference(w, chunks, steps, device, importance)
    loss_dev = torch.zeros((1,), dtype=torch.float64, device=device)
    rows = refs[0].numel() // w.D
    ews = torch.empty((bk.baklava_output_error_workspace_size(rows),), dtype=torch.uint8, device=device)
    outs = torch.empty_like(refs[0])
    table, averages = [], []
    for (t, r_num, r_den) in configs:
        try:
            sess = DecodeSession(w, device, alloc=(t, r_num, r_den), importance=importance)    # MAKE_CACHE's budgets
        except bk.BaklavaError as e:
            table.append({"t": t, "r": "%d/%d" % (r_num, r_den), "loss": None, "error": str(e)})
            averages.append(float("nan"))
            continue
        losses = []
        for c in range(chunks):
            run_chunk(sess, w, chunk_workload(w, c), steps, outs)
            bk.baklava_output_error(outs, refs[c], loss_dev, ews)
            losses.append(float(loss_dev.item()))
        avg = sum(losses) / len(losses)
        averages.append(avg)
        table.append({"t": t, "r": "%d/%d" % (r_num, r_den), "loss": avg, "chunk_losses": losses,
                      "cap_min": int(sess.cap.min()), "cap_max": int(sess.cap.max())})
        del sess
    best = bk.baklava_search_pick(np.asarray(averages))
    return {"workload": w.name, "chunks": chunks, "steps": steps, "candidates": table,
            "best": None if best < 0 else table[best]}


WORKLOADS = {"tiny": wl.TINY,
             "llama-small": wl.scaled(wl.LLAMA3_8B_32K, name="llama3-8b-4l-8k-30pct", L=4, T=8192)}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama-small", choices=sorted(WORKLOADS))
    ap.add_argument("--t", default="0.5,1.0,2.0")
    ap.add_argument("--r", default="0/1,1/4,1/2,3/4")
    ap.add_argument("--chunks", type=int, default=2)
    ap.add_argument("--steps", type=int, default=16)
    args = ap.parse_args(argv)
    ts = [float(x) for x in args.t.split(",")]
    rs = [tuple(int(y) for y in x.split("/")) for x in args.r.split(",")]
    configs = [(t, rn, rd) for t in ts for (rn, rd) in rs]
    res = parameter_search(WORKLOADS[args.workload], configs, args.chunks, args.steps)
    print(json.dumps(res))
    return 0


if __name__ == "__main__":
    sys.exit(main())
