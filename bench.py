#!/usr/bin/env python
"""Decode-step benchmark: retained-KV GB/s of append + attention + score update + eviction over all
layers of a synthetic LLaMA-3-8B-shaped cache (32K context, 30 % budget) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama|qwen|tiny] [--impl ours|reference]

Prints one JSON line.  `value` is timed with the cache resident in HBM; `e2e` copies each step's
q / k_new / v_new from pinned host memory and reads the output back inside the timed region.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
With N > 1 (under torchrun) every rank runs an independent replica of the workload.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2502_13176_b200 import workloads as wl  # noqa: E402

METRIC = "decode-step retained-KV GB/s"
WORKLOADS = {"llama": wl.LLAMA3_8B_32K, "qwen": wl.QWEN25_7B_8K_B16, "tiny": wl.TINY}
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
KERNEL_SOURCES = {"decode_chunk_kernel": ["decode.cu", "ptx.cuh", "common.h", "fp8.cuh"],
                  "profile_pv_kernel": ["profile.cu", "ptx.cuh", "common.h"],
                  "qk_pass_kernel": ["prefill.cu", "ptx.cuh", "common.h"]}


def source_digest(kernel):
    """Short hash of the source files a kernel is compiled from: the key that says whether an ncu capture
    still describes the kernel as it is now."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, "paper_2502_13176_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def ncu_traffic(workload, kernel):
    """dram bytes (read + write) per launch from the table of ncu captures under profiles/: lines of
    `workload kernel source-digest bytes`.  None when there is no capture of this workload, or when the
    kernel's sources have changed since it was taken."""
    if not os.path.exists(TRAFFIC_TABLE):
        return None
    digest = source_digest(kernel)
    with open(TRAFFIC_TABLE) as f:
        for line in f:
            parts = line.split()
            if len(parts) >= 4 and not line.startswith("#") and parts[0] == workload and parts[1] == kernel \
                    and parts[2] == digest:
                return int(parts[3])
    return None


def measured_peaks(key="hbm_gbs", fallback=6650.0):
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)[key]), "measured"
    return fallback, "fallback"


class ClockSampler:
    """Polls SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index):
        self.index, self.rows, self.stop, self.thread, self.max_mhz = index, [], False, None, None

    def __enter__(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(self.index).uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None
        return self

    def _poll(self):
        nv = self.nv
        while not self.stop:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    why = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    why = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.rows.append((time.perf_counter(), mhz, why))
            except Exception:
                pass
            time.sleep(0.002)

    def __exit__(self, *a):
        self.stop = True
        if self.thread:
            self.thread.join(timeout=2)

    def summary(self, t0=None, t1=None):
        rows = [r for r in self.rows if t0 is None or t0 <= r[0] <= t1] or self.rows
        reasons = sorted(n for n, bit in self.REASONS.items() if any(r[2] & bit for r in rows))
        return {"sm_mhz": statistics.median(r[1] for r in rows) if rows else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(rows)}


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(world, units_per_rank_step, steps, elapsed_ms):
    """Aggregate throughput of `world` independent replicas: all units processed / slowest rank's time."""
    return world * units_per_rank_step * steps / (elapsed_ms * 1e-3)


class OracleSample:
    """A bounded sample of the workload for the CPU oracle: a few heads with their full retained caches, built
    once from the seeded generator; `step()` runs one oracle decode step (append, attention, score update,
    eviction) over all of them, one thread per head, and returns the K+V bytes it attended."""

    def __init__(self, w):
        import threadpoolctl

        from oracle import allocation as oalloc
        from oracle.cache import HeadCache
        from paper_2502_13176_b200 import synth

        self.w = w
        imp = wl.importance(w).numpy()
        cap, _, _ = oalloc.allocate(imp, w.t, w.r_num, w.r_den, w.total_pages, w.min_pages, w.max_pages, w.page)
        self.cores = os.cpu_count() or 1
        self.n_heads = min(w.L * w.Hkv * w.B, max(self.cores, 16))
        picks = [(i * (w.L * w.Hkv) // self.n_heads) for i in range(self.n_heads)]
        gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
        self.twins = []
        for j, flat in enumerate(picks):
            l, h = divmod(flat, w.Hkv)
            C = int(cap[l, h]); n = C - 1
            K = synth.normal_bf16(w.seed, 40, (n, w.D), gen_dev, None, j << 24).double().cpu().numpy()
            V = synth.normal_bf16(w.seed, 41, (n, w.D), gen_dev, None, j << 24).double().cpu().numpy()
            sc = synth.uniform_f64(w.seed, 42, j << 20, n).numpy()
            hc = HeadCache(C, w.D, w.n_sink, w.recent_num, w.recent_den)
            hc.load(K, V, np.arange(n), sc)
            self.twins.append(hc)
        self.steps_done = 0
        self.limits = threadpoolctl.threadpool_limits

    def describe(self, steps):
        return "%d of %d heads x %d decode steps (fp64 numpy, one thread per head)" % (
            self.n_heads, self.w.L * self.w.Hkv * self.w.B, steps)

    def step(self, threads=None):
        """One oracle decode step over the sampled heads, one head per thread (`threads` = 1: one after another)."""
        from concurrent.futures import ThreadPoolExecutor

        from paper_2502_13176_b200 import synth
        w, s = self.w, self.steps_done
        feeds = [synth.normal_bf16(w.seed, 43, (w.g + 2, w.D), "cpu", None, (s * self.n_heads + j) * 4096).double().numpy()
                 for j in range(self.n_heads)]

        def one(args):
            hc, feed = args
            hc.step(feed[:w.g], feed[w.g], feed[w.g + 1], w.T + s)
            return hc.C * w.D * 4

        t0 = time.perf_counter()
        with self.limits(limits=1):
            if threads == 1:
                nbytes = sum(one(a) for a in zip(self.twins, feeds))
            else:
                with ThreadPoolExecutor(max_workers=self.cores) as pool:
                    nbytes = sum(pool.map(one, zip(self.twins, feeds)))
        self.steps_done += 1
        return nbytes, time.perf_counter() - t0


def oracle_sample(w, seconds_target=12.0, max_steps=128):
    """Time the CPU oracle's decode step on sampled heads of the workload.  Returns a cpu_baseline dict."""
    sample = OracleSample(w)
    total_bytes, total_s, steps = 0, 0.0, 0
    while steps < max_steps and total_s < seconds_target:
        nb, dt = sample.step()
        total_bytes += nb; total_s += dt; steps += 1
    one_bytes, one_s, one_steps = 0, 0.0, 0                # the same sample on one core
    while one_steps < max_steps and one_s < seconds_target / 2:
        nb, dt = sample.step(threads=1)
        one_bytes += nb; one_s += dt; one_steps += 1
    return {"value": total_bytes / total_s / 1e9, "unit": "GB/s", "cores": sample.cores, "kind": "oracle",
            "sample": sample.describe(steps), "seconds": total_s,
            "single_thread": {"value": one_bytes / one_s / 1e9, "unit": "GB/s", "cores": 1, "steps": one_steps}}


def run_reference(args, w):
    """The reference arm: the oracle as it stands on the host cores; one step = one oracle decode step over the
    bounded sample of heads (built once, untimed).  Rank 0 alone runs it."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = OracleSample(w)
    for _ in range(args.warmup):
        sample.step()
    total_bytes, total_s = 0, 0.0
    for _ in range(args.steps):
        nb, dt = sample.step()
        total_bytes += nb; total_s += dt
    v = total_bytes / total_s / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_s / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.L, "batch": w.B, "context": w.T, "budget": w.budget},
        "cpu_baseline": {"value": v, "unit": "GB/s", "cores": sample.cores, "kind": "oracle",
                         "sample": sample.describe(args.steps)},
        "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def timed_calls(dev, call, steps, warmup):
    """`warmup` untimed calls, then `steps` calls between two events; returns (ms per call, clocks summary)."""
    for _ in range(warmup):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    with ClockSampler(dev.index) as clocks:
        t_open = time.perf_counter()
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize(dev)
        t_close = time.perf_counter()
    return e0.elapsed_time(e1) / steps, clocks.summary(t_open, t_close)


def tensor_line(metric, workload, config, kernel, flop, ms, clocks, args, launches, dtype="bf16"):
    peak, peak_kind = measured_peaks("bf16_tflops", 1590.0)
    tf = flop / (ms * 1e-3) / 1e12
    # a timed region of a good part of a second runs under the power cap: the cuBLAS figure measured the same
    # way (back to back for seconds) is given beside the burst one
    sustained_peak, _ = measured_peaks("bf16_tflops_sustained", 1400.0)
    long_run = {"timed_seconds": ms * 1e-3 * args.steps, "peak_sustained": sustained_peak,
                "frac_of_sustained": tf / sustained_peak}
    return {"metric": metric, "value": tf, "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype,
            "data": "synthetic", "config": dict(workload=workload, **config),
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                         "traffic": ncu_traffic(workload, kernel), "peak_kind": peak_kind, "kernel": kernel,
                         **long_run},
            "ms_x_sm_ghz": None if not clocks.get("sm_mhz") else ms * clocks["sm_mhz"] * 1e-3,
            "gpu_launches": launches * args.steps, "clocks": clocks}


def run_profile_pass(args):
    """The one-time profiling pass (Algorithm 1 step 1) on the LLaMA-3-8B attention shape: one step = one
    layer's heads for all prompts.  Reported against the tensor roofline; not the headline benchmark."""
    from paper_2502_13176_b200 import binding as bk
    from paper_2502_13176_b200.engine import shape_of

    w = wl.LLAMA3_8B_32K
    P, T = args.prompts, args.prompt_tokens
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    shape = shape_of(w)
    parts = [wl.profile_inputs(w, p, 0, T, dev) for p in range(P)]
    q = torch.stack([x[0] for x in parts]); k = torch.stack([x[1] for x in parts]); v = torch.stack([x[2] for x in parts])
    del parts
    head_cos = torch.empty((P, w.Hq), dtype=torch.float32, device=dev)
    ws = torch.empty((bk.baklava_profile_workspace_size(shape, P, T),), dtype=torch.uint8, device=dev)
    ms, clocks = timed_calls(dev, lambda: bk.baklava_profile_heads(shape, q, k, v, None, P, T, head_cos, None, ws),
                             args.steps, args.warmup)
    assert bk.workspace_error(ws) == 0
    flop = P * w.Hq * 2.0 * T * T * w.D          # QK^T and PV under the causal mask: 2 * (T^2 / 2) * D * 2 each
    line = tensor_line("profiling-pass TFLOP/s (causal attention + cosine, one layer)", "profile-llama3-8b",
                       {"prompts": P, "prompt_tokens": T, "heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D},
                       "profile_pv_kernel", flop, ms, clocks, args, 4)
    # end to end: the layer's Q, K, V come from pinned host memory and the head means go back, every step
    host = [t.cpu().pin_memory() for t in (q, k, v)]
    back = torch.empty(head_cos.shape, dtype=head_cos.dtype).pin_memory()

    def e2e():
        for d, h in zip((q, k, v), host):
            d.copy_(h, non_blocking=True)
        bk.baklava_profile_heads(shape, q, k, v, None, P, T, head_cos, None, ws)
        back.copy_(head_cos, non_blocking=True)
    e2e_ms, _ = timed_calls(dev, e2e, max(1, args.steps // 4), 1)
    line["e2e"] = {"value": flop / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                   "h2d_bytes_per_step": sum(h.numel() * h.element_size() for h in host),
                   "d2h_bytes_per_step": back.numel() * back.element_size()}
    if not args.no_cpu_baseline:
        from oracle import profiling as oprof
        n, t0 = 0, time.perf_counter()
        while n < 4 and time.perf_counter() - t0 < 15.0:       # a few full (prompt, head) instances
            h = (n * 9) % w.Hq
            oprof.head_similarity(q[0, h].double().cpu().numpy(), k[0, h // w.g].double().cpu().numpy(),
                                  v[0, h // w.g].double().cpu().numpy(), T)
            n += 1
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n * 2.0 * T * T * w.D / dt / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(),
                                "kind": "oracle", "sample": "%d of %d (prompt, head) instances of %d tokens (fp64 numpy)" % (
                                    n, P * w.Hq, T)}
    print(json.dumps(line))


def run_prefill_scores(args):
    """Exact seeding of the heavy-hitter scores for one layer of a 32K prompt (two passes over Q K^T, or one
    when the caller already has the rows' log-sum-exp)."""
    from paper_2502_13176_b200 import binding as bk, synth
    from paper_2502_13176_b200.engine import shape_of

    w = wl.LLAMA3_8B_32K
    B, T = 1, args.prompt_tokens
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    shape = shape_of(w)
    q = synth.normal_bf16(w.seed, wl.T_PROFILE_Q, (B, w.Hq, T, w.D), dev)
    k = synth.normal_bf16(w.seed, wl.T_PROFILE_K, (B, w.Hkv, T, w.D), dev)
    score = torch.empty((B, w.Hkv, T), dtype=torch.float32, device=dev)
    ws = torch.empty((bk.baklava_prefill_workspace_size(shape, B, T),), dtype=torch.uint8, device=dev)
    lse = None
    if args.lse_given:
        # the rows' natural-log normaliser as a prefill attention kernel would leave it (set-up, not timed):
        # plain torch, a block of query rows at a time
        lse = torch.empty((B, w.Hq, T), dtype=torch.float32, device=dev)
        cols = torch.arange(T, device=dev)
        for b in range(B):
            for h in range(w.Hq):
                for r0 in range(0, T, 4096):
                    sc = (q[b, h, r0:r0 + 4096].float() @ k[b, h // w.g].float().T) / w.D ** 0.5
                    sc.masked_fill_(cols[None, :] > torch.arange(r0, min(T, r0 + 4096), device=dev)[:, None], float("-inf"))
                    lse[b, h, r0:r0 + 4096] = torch.logsumexp(sc, dim=1)
        del sc
    ms, clocks = timed_calls(dev, lambda: bk.baklava_prefill_scores(shape, q, k, None, B, T, score, ws, lse=lse),
                             args.steps, args.warmup)
    assert bk.workspace_error(ws) == 0
    passes = 1 if args.lse_given else 2
    flop = passes * B * w.Hq * 1.0 * T * T * w.D      # Q K^T under the causal mask, once per pass
    line = tensor_line("prompt-score seeding TFLOP/s (one layer)", "prefill-scores-llama3-8b",
                       {"batch": B, "prompt_tokens": T, "passes": passes,
                        "lse": "given by the caller" if args.lse_given else "computed by the first pass"},
                       "qk_pass_kernel", flop, ms, clocks, args, passes)
    host = [t.cpu().pin_memory() for t in (q, k)]
    back = torch.empty(score.shape, dtype=score.dtype).pin_memory()

    def e2e():
        for d, h in zip((q, k), host):
            d.copy_(h, non_blocking=True)
        bk.baklava_prefill_scores(shape, q, k, None, B, T, score, ws, lse=lse)
        back.copy_(score, non_blocking=True)
    e2e_ms, _ = timed_calls(dev, e2e, max(1, args.steps // 4), 1)
    line["e2e"] = {"value": flop / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                   "h2d_bytes_per_step": sum(h.numel() * h.element_size() for h in host),
                   "d2h_bytes_per_step": back.numel() * back.element_size()}
    if not args.no_cpu_baseline:
        from oracle.prefill import prefill_scores as oracle_scores
        Tc = min(T, 4096)                                  # the oracle forms a Tc x Tc matrix per query head
        t0 = time.perf_counter()
        oracle_scores(q[0, :w.g, :Tc].double().cpu().numpy(), k[0, 0, :Tc].double().cpu().numpy())
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 2 * w.g * 1.0 * Tc * Tc * w.D / dt / 1e12, "unit": "TFLOP/s",
                                "cores": os.cpu_count(), "kind": "oracle",
                                "sample": "one KV group (%d query heads) of the first %d tokens (fp64 numpy)" % (w.g, Tc)}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="llama", choices=sorted(WORKLOADS) + ["profile", "prefill"])
    ap.add_argument("--prompts", type=int, default=64, help="profile workload: prompts per step")
    ap.add_argument("--prompt-tokens", type=int, default=4096, help="profile workload: tokens per prompt")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="only the first LAYERS layers (for profiling a small case)")
    ap.add_argument("--chunk", type=int, default=0, help="force the plan's chunk length (tokens); 0 = automatic")
    ap.add_argument("--policy", default="heavy", choices=["heavy", "window"],
                    help="heavy: sinks + window + accumulated-attention heavy hitters (default); "
                         "window: the paper's evaluated sinks + window policy, run without scores")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"],
                    help="slab format: bf16 (the headline) or FP8 E4M3 with per-head scales (half the bytes per row)")
    ap.add_argument("--mixed-lengths", action="store_true",
                    help="prompts of different lengths (seeded, uniform in [T/8, T]) decoded at per-sequence "
                         "positions through baklava_decode_attn_varlen")
    ap.add_argument("--per-layer", default="off", choices=["off", "calls", "graph"],
                    help="one baklava_decode_attn_varlen call per layer instead of one call over all layers: "
                         "issued one by one (calls) or captured once in a CUDA graph and replayed (graph)")
    ap.add_argument("--lse-given", action="store_true",
                    help="prefill workload: hand the rows' log-sum-exp to baklava_prefill_scores (one pass instead of two)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="with --per-layer: do not let a layer's call start beside the previous layer's tail")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain-seconds", type=float, default=1.0,
                    help="after the K timed steps, keep stepping for at least this long (cycling the step inputs) "
                         "and report that region too, with the SM clock seen under it; 0 = skip")
    args = ap.parse_args()
    if args.workload == "profile":
        return run_profile_pass(args)
    if args.workload == "prefill":
        return run_prefill_scores(args)
    w = WORKLOADS[args.workload]
    if args.layers:
        w = wl.scaled(w, L=args.layers)
    if args.policy == "window":
        w = wl.scaled(w, name=w.name + "-window", recent_num=1, recent_den=1)
    if args.impl == "reference":
        return run_reference(args, w)

    from paper_2502_13176_b200 import binding as bk
    from paper_2502_13176_b200.engine import DecodeSession

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    bk.lib()                                             # fail now if the library is missing
    step_flags = bk.FLAG_NO_SCORE if args.policy == "window" else 0
    sess = DecodeSession(w, dev, chunk_tokens=args.chunk,
                         kv_dtype=bk.KV_FP8_E4M3 if args.kv == "fp8" else bk.KV_BF16)
    if args.kv == "fp8":
        w = wl.scaled(w, name=w.name + "-fp8")
    total = args.warmup + args.steps
    if args.mixed_lengths:
        from paper_2502_13176_b200 import synth
        u = synth.uniform_f64(w.seed, 50, 0, w.B).numpy()
        prompt_len = [int(w.T // 8 + x * (w.T - w.T // 8)) for x in u]
        sess.prefill_synthetic(prompt_len)
        # positions of every step, made ahead so that no other kernel runs between the steps
        t_steps = (sess.t_seq[None, :] + torch.arange(4 * total, device=dev, dtype=torch.int32)[:, None]).contiguous()
        counter = [0]

        def varlen_step(q, k, v, flags=0):
            i = counter[0]; counter[0] += 1
            return sess.step_varlen(q, k, v, t_steps[i], flags)
        sess.step = varlen_step
        w = wl.scaled(w, name=w.name + "-mixed")
    else:
        sess.prefill_synthetic()
    if args.per_layer != "off":
        # layer by layer, as a model calls attention; positions live on the device and advance there
        sess.per_layer_plans(args.chunk, overlap=not args.no_overlap)
        t_dev = torch.full((w.B,), w.T, dtype=torch.int32, device=dev)
        sq, sk, sv = (torch.empty_like(t) for t in wl.decode_inputs(w, 0, sess.scales, dev))

        def layer_calls():
            sess.step_layers(sq, sk, sv, t_dev, step_flags, overlap=not args.no_overlap)
            t_dev.add_(1)
        if args.per_layer == "graph":
            side = torch.cuda.Stream(dev)
            with torch.cuda.stream(side):
                layer_calls()                                # once outside capture: attributes, first-use set-up
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    layer_calls()
            torch.cuda.current_stream(dev).wait_stream(side)

        def layered_step(q, k, v, flags=0):
            sq.copy_(q, non_blocking=True); sk.copy_(k, non_blocking=True); sv.copy_(v, non_blocking=True)
            if args.per_layer == "graph":
                graph.replay()
            else:
                layer_calls()
            return sess.out
        sess.step = layered_step
        w = wl.scaled(w, name=w.name + "-per-layer-" + args.per_layer)
    feeds = [wl.decode_inputs(w, i, sess.scales, dev) for i in range(2 * total)]
    torch.cuda.synchronize(dev)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with ClockSampler(local) as clocks:
        for i in range(args.warmup):                       # load the GPU before the clock window opens
            sess.step(*feeds[i], flags=step_flags)
        barrier()
        rows_per_step = int(sess.cache.len.sum().item()) + sess.plan.info.n_units   # rows attended: retained + new
        t_open = time.perf_counter()
        ev[0].record()
        for i in range(args.steps):
            sess.step(*feeds[args.warmup + i], flags=step_flags)
        ev[1].record()
        torch.cuda.synchronize(dev)
        t_close = time.perf_counter()
    barrier()
    sess.check_status()
    elapsed_ms = ev[0].elapsed_time(ev[1])

    # ---- sustained: a second or more of continuous stepping, the clock the GPU settles at under it
    sustained = None
    if args.sustain_seconds > 0:
        est = max(elapsed_ms / args.steps, 1e-3)
        n_sus = int(args.sustain_seconds * 1e3 / est) + 1
        sv = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        with ClockSampler(local) as sus_clocks:
            s_open = time.perf_counter()
            sv[0].record()
            for i in range(n_sus):
                sess.step(*feeds[i % total], flags=step_flags)
            sv[1].record()
            torch.cuda.synchronize(dev)
            s_close = time.perf_counter()
        sus_ms = sv[0].elapsed_time(sv[1])
        sustained = {"steps": n_sus, "seconds": sus_ms * 1e-3, "ms_per_step": sus_ms / n_sus,
                     "clocks": sus_clocks.summary(s_open, s_close)}
        sess.check_status()

    # ---- per-step spread: the same steps again with an event after each (the events sit between the launches,
    # so these steps lose the overlap of one step's tail with the next step's start and run a few us longer)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    marks[0].record()
    for i in range(args.steps):
        sess.step(*feeds[args.warmup + i], flags=step_flags)
        marks[i + 1].record()
    torch.cuda.synchronize(dev)
    per_step_us = sorted(marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(args.steps))

    def pct(q):
        return per_step_us[min(len(per_step_us) - 1, int(q * len(per_step_us)))]

    # ---- end to end: host buffers in, host buffer out, every step.  A step's q / k_new / v_new travel as one
    # pinned buffer (one copy), the output comes back as one
    def packed(ts):
        flat = torch.cat([t.reshape(-1) for t in ts])
        return flat.cpu().pin_memory()
    host = [packed(feeds[total + i]) for i in range(total)]
    dev_in = torch.empty_like(host[0], device=dev)
    sizes = [t.numel() for t in feeds[0]]
    offs = [0, sizes[0], sizes[0] + sizes[1]]
    dq, dk, dv = (dev_in[o:o + n].view(t.shape) for o, n, t in zip(offs, sizes, feeds[0]))
    out_host = torch.empty(sess.out.shape, dtype=sess.out.dtype).pin_memory()
    h2d = host[0].numel() * host[0].element_size()
    d2h = out_host.numel() * out_host.element_size()

    def e2e_step(i):
        dev_in.copy_(host[i], non_blocking=True)
        out_host.copy_(sess.step(dq, dk, dv, flags=step_flags), non_blocking=True)

    for i in range(args.warmup):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        e2e_step(args.warmup + i)
    e1.record()
    torch.cuda.synchronize(dev)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    sess.check_status()

    elapsed_ms, e2e_ms = max_over_ranks([elapsed_ms, e2e_ms], dev)

    if rank == 0:
        bytes_per_step = rows_per_step * w.D * 2 * (1 if args.kv == "fp8" else 2)   # K and V rows, bf16 or one byte
        gbs = whole_job_rate(world, bytes_per_step, args.steps, elapsed_ms) / 1e9
        e2e_gbs = whole_job_rate(world, bytes_per_step, args.steps, e2e_ms) / 1e9
        peak, peak_kind = measured_peaks()
        kernel_ms = elapsed_ms / args.steps               # one step = one call = one kernel
        achieved = bytes_per_step / (kernel_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if args.kv == "bf16" else "fp8-e4m3 slabs, fp16 MMA",
            "data": "synthetic",
            "config": {"workload": w.name, "layers": w.L, "batch": w.B, "context": w.T, "budget": w.budget,
                       "kv_bytes_per_step": bytes_per_step, "l2": "inputs larger than L2 (no flush)",
                       "launch": ("one baklava_decode_attn_varlen call per layer (%s), %s" % (
                                      "CUDA graph replay" if args.per_layer == "graph" else "issued one by one",
                                      "each waiting for the one before it" if args.no_overlap else
                                      "layers after the first flagged BAKLAVA_FLAG_OVERLAP_PREV: every layer's inputs are "
                                      "ready before the first call, so a layer streams beside the tails of those before it"))
                       if args.per_layer != "off" else
                       "one baklava_decode_attn%s call per step covering all layers" % (
                           "_varlen" if args.mixed_lengths else ""), "policy": args.policy,
                       "replicas": world},
            "tokens_per_s": whole_job_rate(world, w.B, args.steps, elapsed_ms),
            "step_us_with_event_per_step": {"p10": pct(0.1), "median": pct(0.5), "p90": pct(0.9)},
            "pct_of_hbm_peak": 100.0 * gbs / world / peak,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": ncu_traffic(w.name, "decode_chunk_kernel"),
                         "peak_kind": peak_kind, "kernel": "decode_chunk_kernel",
                         "note": "events bracket one call = one kernel (attention, score update and eviction)"},
            "e2e": {"value": e2e_gbs, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": args.steps * (w.L if args.per_layer != "off" else 1),
            "clocks": clocks.summary(t_open, t_close),
        }
        mhz = line["clocks"].get("sm_mhz")
        line["us_x_sm_ghz"] = None if not mhz else kernel_ms * 1e3 * mhz * 1e-3      # clock-normalised step time
        if sustained:
            sustained["value"] = bytes_per_step / (sustained["ms_per_step"] * 1e-3) / 1e9
            sustained["unit"] = "GB/s"
            sustained["frac_of_peak"] = sustained["value"] / peak
            smhz = sustained["clocks"].get("sm_mhz")
            sustained["us_x_sm_ghz"] = None if not smhz else sustained["ms_per_step"] * 1e3 * smhz * 1e-3
            line["sustained"] = sustained
        if world == 1 and not args.no_cpu_baseline:
            cb = oracle_sample(w)
            cb.pop("seconds")
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
