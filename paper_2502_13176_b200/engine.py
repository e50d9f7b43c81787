"""Convenience layer over the binding: owns the device buffers of one budgeted cache and drives
allocate -> bulk evict -> decode steps.  Memory management and call sequencing only; every
computation happens inside libbaklava.so."""
import numpy as np
import torch

from . import binding as bk
from . import workloads as wl


def shape_of(w):
    return bk.make_shape(w.L, w.Hq, w.Hkv, w.D, w.page, w.n_sink, w.recent_num, w.recent_den)


class DecodeSession:
    def __init__(self, w, device="cuda", layers=None, chunk_tokens=0, uniform=False, alloc=None, importance=None,
                 total_tokens=None, kv_dtype=bk.KV_BF16):
        """`alloc` = (t, r_num, r_den) overrides the workload's Algorithm 2 parameters, `importance` its
        synthetic importances, `total_tokens` its budget (e.g. the dense length for a reference run)."""
        self.w, self.device = w, torch.device(device)
        self.shape = shape_of(w)
        self.scales = wl.kv_scales(w)
        self.importance = wl.importance(w).numpy() if importance is None else np.asarray(importance, dtype=np.float64)
        t, r_num, r_den = (w.t, w.r_num, w.r_den) if alloc is None else alloc
        total = w.total_pages * w.page if total_tokens is None else int(total_tokens)
        self.cap, self.off, self.stride = bk.baklava_allocate(
            self.shape, self.importance, t, 0 if uniform else r_num, r_den, total,
            w.min_pages * w.page, w.max_pages * w.page)
        self.kv_dtype = kv_dtype
        fp8_scales = wl.kv_fp8_scales(w, self.scales) if kv_dtype == bk.KV_FP8_E4M3 else None
        self.cache = bk.Cache(self.shape, self.cap, self.off, self.stride, w.B, self.device, kv_dtype=kv_dtype,
                              kv_scale=fp8_scales)
        self.lb, self.le = (0, w.L) if layers is None else layers
        n_sm = torch.cuda.get_device_properties(self.device).multi_processor_count
        self.plan = bk.baklava_decode_plan(self.shape, self.cap, w.B, self.lb, self.le, self.stride,
                                           chunk_tokens=chunk_tokens, n_sm=n_sm, kv_dtype=kv_dtype).to(self.device)
        self.ws = bk.decode_workspace(self.plan, self.device)
        nl = self.le - self.lb
        self.out = torch.zeros((nl, w.B, w.Hq, w.D), dtype=torch.bfloat16, device=self.device)
        self.lse = torch.zeros((nl, w.B, w.Hq), dtype=torch.float32, device=self.device)
        self.t = 0

    def prefill_synthetic(self, prompt_len=None, data=None):
        """Fill every head from the workload's dense synthetic prompt through baklava_evict, a layer at a time.
        `prompt_len` (B ints) keeps only that many tokens of each sequence's prompt; `data` is a copy of the
        workload with another seed (another prompt through the same heads)."""
        w = self.w if data is None else data
        ews = torch.empty((bk.baklava_evict_workspace_size(self.shape, w.B, 1, w.T),), dtype=torch.uint8,
                          device=self.device)
        plen = None if prompt_len is None else torch.tensor(list(prompt_len), dtype=torch.int32, device=self.device)
        for l in range(self.lb, self.le):
            k, v = wl.dense_kv_layer(w, l, self.scales, self.device)
            sc = wl.prefill_scores(w, l, self.device)
            bk.baklava_evict_varlen(self.shape, self.cache, l, l + 1, k, v, sc, w.T, plen, 0, w.Hkv * w.T, w.T, 1, ews)
            torch.cuda.synchronize(self.device)
        self.t = w.T
        self.t_seq = plen

    def step(self, q, k_new, v_new, flags=0):
        """One decode step for the session's layer range; returns the output tensor (device, bf16)."""
        bk.baklava_decode_attn(self.shape, self.cache, q, k_new, v_new, self.t, self.out, self.lse, flags,
                               self.plan, self.ws)
        if not (flags & bk.FLAG_NO_APPEND):
            self.t += 1
        return self.out

    def step_varlen(self, q, k_new, v_new, t_pos, flags=0):
        """One decode step with per-sequence positions `t_pos` (device int32 [B]; negative = idle)."""
        bk.baklava_decode_attn_varlen(self.shape, self.cache, q, k_new, v_new, t_pos, self.out, self.lse, flags,
                                      self.plan, self.ws)
        return self.out

    def per_layer_plans(self, chunk_tokens=0, overlap=True):
        """One plan and workspace per layer, for callers that run attention layer by layer (as a model does).
        With `overlap` (the calls after the first will carry BAKLAVA_FLAG_OVERLAP_PREV) and no chunk length given,
        chunks of 1024 tokens: consecutive layers' kernels then share the GPU, and what counts is the fixed cost
        per chunk, not that one layer's chunks fill one wave."""
        if overlap and chunk_tokens == 0:
            chunk_tokens = 1024
        n_sm = torch.cuda.get_device_properties(self.device).multi_processor_count
        self.layer_plans = []
        for l in range(self.lb, self.le):
            plan = bk.baklava_decode_plan(self.shape, self.cap, self.w.B, l, l + 1, self.stride, chunk_tokens=chunk_tokens,
                                          n_sm=n_sm, kv_dtype=self.kv_dtype).to(self.device)
            self.layer_plans.append((plan, bk.decode_workspace(plan, self.device)))

    def step_layers(self, q, k_new, v_new, t_pos, flags=0, overlap=True):
        """One decode step as one call per layer; t_pos: device int32 [B] (so that the sequence of calls can be
        captured in a CUDA graph and replayed with the positions advanced on the device).  q / k_new / v_new of
        every layer must be complete before the first call is enqueued when `overlap` is set."""
        for i, (plan, ws) in enumerate(self.layer_plans):
            # every layer has its own heads, inputs and workspace, and all inputs are complete before the first
            # call: from the second layer on a call may start beside the previous layer's tail
            fl = flags | (bk.FLAG_OVERLAP_PREV if overlap and i > 0 else 0)
            bk.baklava_decode_attn_varlen(self.shape, self.cache, q[i:i + 1], k_new[i:i + 1], v_new[i:i + 1], t_pos,
                                          self.out[i:i + 1], self.lse[i:i + 1], fl, plan, ws)
        return self.out

    def retained_kv_bytes(self):
        """Bytes of K and V in valid rows of the session's layers: what one step must read."""
        n = int(self.cache.len[:, self.lb:self.le].sum().item())
        return n * self.w.D * 2 * (1 if self.kv_dtype == bk.KV_FP8_E4M3 else 2)

    def check_status(self):
        code = int(self.cache.status.item())
        if code:
            raise RuntimeError("device status word = %d" % code)
