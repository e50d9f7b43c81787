"""Long-context sweep on the LLaMA-3-8B attention shape: batch x context x budget, ragged (Algorithm 2)
against uniform capacities of the same total.

    python -m paper_2502_13176_b200.sweep [--batches 1,8,32] [--contexts 32768,131072]
                                          [--budgets 10,20,...,90] [--steps 32] [--max-gb 40]

One JSON line per point.  A point whose retained K+V would not fit in --max-gb runs on its first L'
layers only (layers are independent, so GB/s is unaffected; tokens/s is then extrapolated to 32 layers
and marked so).  Calls only the library (through `engine.DecodeSession`); no oracle here.
"""
import argparse
import json
import sys

import torch

from . import workloads as wl
from .engine import DecodeSession


def run_point(B, T, budget, steps, warmup, max_bytes, uniform, dev):
    w = wl.sweep_point(B, T, budget)
    per_layer = w.base_pages * w.page * w.Hkv * B * w.D * 4            # bytes of K+V retained per layer
    layers = max(1, min(w.L, int(max_bytes // max(1, per_layer))))
    if layers < w.L:
        w = wl.scaled(w, L=layers)
    sess = DecodeSession(w, dev, uniform=uniform)
    sess.prefill_synthetic()
    feeds = [wl.decode_inputs(w, i, sess.scales, dev) for i in range(4)]
    for i in range(warmup):
        sess.step(*feeds[i % 4])
    torch.cuda.synchronize(dev)
    rows = int(sess.cache.len.sum().item()) + sess.plan.info.n_units
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        sess.step(*feeds[i % 4])
    e1.record()
    torch.cuda.synchronize(dev)
    sess.check_status()
    ms = e0.elapsed_time(e1) / steps
    bytes_per_step = rows * w.D * 4
    cap = sess.cap
    out = {"B": B, "T": T, "budget": budget, "uniform": uniform, "layers_run": layers, "layers_model": 32,
           "kv_gb_per_step": bytes_per_step / 1e9, "us_per_step": ms * 1e3,
           "gbs": bytes_per_step / (ms * 1e-3) / 1e9,
           "tokens_per_s_32_layers": B / (ms * 1e-3) * layers / 32.0, "extrapolated": layers < 32,
           "cap_min": int(cap.min()), "cap_max": int(cap.max()), "items": int(sess.plan.info.n_items)}
    del sess, feeds
    torch.cuda.empty_cache()
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,8,32")
    ap.add_argument("--contexts", default="32768,131072")
    ap.add_argument("--budgets", default="10,20,30,40,50,60,70,80,90")
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--max-gb", type=float, default=40.0)
    ap.add_argument("--peak-gbs", type=float, default=0.0, help="bandwidth to report fractions of (0: omit)")
    args = ap.parse_args(argv)
    dev = torch.device("cuda", 0)
    for T in [int(x) for x in args.contexts.split(",")]:
        for B in [int(x) for x in args.batches.split(",")]:
            for pct in [int(x) for x in args.budgets.split(",")]:
                pair = {}
                for uniform in (False, True):
                    r = run_point(B, T, pct / 100.0, args.steps, args.warmup, args.max_gb * 1e9, uniform, dev)
                    if args.peak_gbs:
                        r["frac_of_peak"] = r["gbs"] / args.peak_gbs
                    pair[uniform] = r
                    print(json.dumps(r), flush=True)
                print(json.dumps({"B": B, "T": T, "budget": pct / 100.0,
                                  "ragged_over_uniform": pair[False]["gbs"] / pair[True]["gbs"]}), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
