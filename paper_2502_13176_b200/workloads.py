"""The synthetic workloads: shapes, seeds and input recipes.  No arithmetic of the method lives here.

Each workload stands in for a model / context length the paper evaluates
(LLaMA-3-8B and Qwen2.5-7B attention shapes, 8K and 32K contexts): random
tensors of those shapes, not the models' activations.  Everything is produced
by `synth` from (seed, tensor_id, flat index), so any head can be regenerated
alone, on the host or on the device, with identical bits.
"""
from dataclasses import dataclass, replace

import torch

from . import synth

MASTER_SEED = 20250213

# tensor ids
T_K, T_V, T_Q, T_KNEW, T_VNEW, T_IMPORTANCE, T_KSCALE, T_OUTLIER, T_RMS, T_SCORE = range(10)
T_PROFILE_Q, T_PROFILE_K, T_PROFILE_V = 16, 17, 18


@dataclass(frozen=True)
class Workload:
    name: str
    L: int
    Hq: int
    Hkv: int
    D: int
    B: int
    T: int                    # prefilled context, tokens
    budget: float             # retained fraction of the dense cache
    steps: int
    importance_sigma: float
    kv_recipe: str            # "channel_lognormal" | "outlier" | "head_rms" | "plain"
    seed: int
    page: int = 16
    n_sink: int = 4
    recent_num: int = 1
    recent_den: int = 2
    t: float = 1.0            # Algorithm 2 threshold (median of lognormal importance)
    r_num: int = 1            # Algorithm 2 reduction r = r_num / r_den
    r_den: int = 2

    @property
    def g(self):
        return self.Hq // self.Hkv

    @property
    def base_pages(self):
        return int(self.budget * self.T / self.page + 1e-9)

    @property
    def total_pages(self):
        return self.base_pages * self.L * self.Hkv

    @property
    def min_pages(self):
        return -(-(self.n_sink + 2) // self.page)

    @property
    def max_pages(self):
        return -(-(self.T + self.steps) // self.page)


TINY = Workload("tiny", L=2, Hq=4, Hkv=2, D=64, B=1, T=512, budget=0.5, steps=8,
                importance_sigma=1.0, kv_recipe="channel_lognormal", seed=MASTER_SEED + 1)
LLAMA3_8B_32K = Workload("llama3-8b-32k-30pct", L=32, Hq=32, Hkv=8, D=128, B=1, T=32768, budget=0.3,
                         steps=64, importance_sigma=1.0, kv_recipe="outlier", seed=MASTER_SEED + 2)
QWEN25_7B_8K_B16 = Workload("qwen2.5-7b-8k-b16-30pct", L=28, Hq=28, Hkv=4, D=128, B=16, T=8192,
                            budget=0.3, steps=128, importance_sigma=1.5, kv_recipe="head_rms",
                            seed=MASTER_SEED + 3)


def sweep_point(B, T, budget):
    """One point of the long-context sweep (LLaMA-3-8B shape)."""
    return replace(LLAMA3_8B_32K, name=f"llama3-8b-b{B}-t{T}-{int(round(budget * 100))}pct",
                   B=B, T=T, budget=budget, steps=32, seed=MASTER_SEED + 5)


def scaled(w, **kw):
    """A smaller copy of a workload (fewer layers, shorter context) for parity tests."""
    return replace(w, **kw)


def importance(w):
    """[L, Hkv] float64, lognormal(0, sigma)."""
    return synth.lognormal_f64(w.seed, T_IMPORTANCE, w.L * w.Hkv, w.importance_sigma).reshape(w.L, w.Hkv)


def kv_scales(w):
    """(k_scale, v_scale), each fp32 [L, Hkv, D]."""
    shape = (w.L, w.Hkv, w.D)
    one = torch.ones(shape, dtype=torch.float32)
    if w.kv_recipe == "plain":
        return one, one.clone()
    if w.kv_recipe == "channel_lognormal":
        ks = synth.lognormal_f64(w.seed, T_KSCALE, w.L * w.Hkv * w.D, 0.5).reshape(shape).to(torch.float32)
        return ks, one
    if w.kv_recipe == "outlier":
        n_out = max(1, int(round(0.01 * w.D)))
        u = synth.uniform_f64(w.seed, T_OUTLIER, 0, w.L * w.Hkv * n_out).reshape(w.L, w.Hkv, n_out)
        ch = torch.clamp((u * w.D).to(torch.int64), max=w.D - 1)
        s = one.clone()
        s.scatter_(2, ch, 8.0)
        return s, s.clone()
    if w.kv_recipe == "head_rms":
        u = synth.uniform_f64(w.seed, T_RMS, 0, w.L * w.Hkv).reshape(w.L, w.Hkv, 1)
        s = (0.5 + 1.5 * u).to(torch.float32).expand(shape).contiguous()
        return s, s.clone()
    raise ValueError(w.kv_recipe)


def kv_fp8_scales(w, scales):
    """Per-head FP8 scales as float32 [L, Hkv, 4] = (K scale, 1 / K scale, V scale, 1 / V scale), the layout the
    library takes: six standard deviations of the head's widest channel map to the largest finite E4M3 value
    (448); the reciprocals are float32 divisions, rounded once, and are inputs like the scales themselves."""
    widest = torch.stack([scales[0].amax(dim=2), scales[1].amax(dim=2)], dim=2)      # [L, Hkv, 2]
    sc = (widest * (6.0 / 448.0)).to(torch.float32)
    one = torch.ones((), dtype=torch.float32)
    four = torch.stack([sc[..., 0], one / sc[..., 0], sc[..., 1], one / sc[..., 1]], dim=2)
    return four.numpy()


def dense_kv(w, l, b, h, scales, device="cpu", T=None):
    """Prefilled K and V of one (layer, sequence, KV head): two bf16 [T, D] tensors."""
    T = w.T if T is None else T
    start = (((l * w.B + b) * w.Hkv + h) * w.T) * w.D
    k = synth.normal_bf16(w.seed, T_K, (T, w.D), device, scales[0][l, h], start)
    v = synth.normal_bf16(w.seed, T_V, (T, w.D), device, scales[1][l, h], start)
    return k, v


def dense_kv_layer(w, l, scales, device="cpu"):
    """Prefilled K and V of one layer: bf16 [B, Hkv, T, D] each."""
    start = (l * w.B * w.Hkv * w.T) * w.D
    shape = (w.B, w.Hkv, w.T, w.D)
    ks = scales[0][l].reshape(1, w.Hkv, 1, w.D)
    vs = scales[1][l].reshape(1, w.Hkv, 1, w.D)
    return (synth.normal_bf16(w.seed, T_K, shape, device, ks, start),
            synth.normal_bf16(w.seed, T_V, shape, device, vs, start))


def prefill_scores(w, l, device="cpu"):
    """Stand-in for the attention mass each prompt token gathered during prefill:
    fp32 [B, Hkv, T], uniform in (0, 1)."""
    n = w.B * w.Hkv * w.T
    return synth.uniform_f64(w.seed, T_SCORE, l * n, n, device).to(torch.float32).reshape(w.B, w.Hkv, w.T)


def decode_inputs(w, step, scales, device="cpu", layers=None):
    """(q [L', B, Hq, D], k_new [L', B, Hkv, D], v_new [L', B, Hkv, D]) bf16 for one decode step,
    for the layer range `layers` = (begin, end) (default: all)."""
    lb, le = (0, w.L) if layers is None else layers
    nq, nk = w.B * w.Hq * w.D, w.B * w.Hkv * w.D
    q = synth.normal_bf16(w.seed, T_Q, (le - lb, w.B, w.Hq, w.D), device, None, (step * w.L + lb) * nq)
    ks = scales[0][lb:le].reshape(le - lb, 1, w.Hkv, w.D)
    vs = scales[1][lb:le].reshape(le - lb, 1, w.Hkv, w.D)
    kn = synth.normal_bf16(w.seed, T_KNEW, (le - lb, w.B, w.Hkv, w.D), device, ks, (step * w.L + lb) * nk)
    vn = synth.normal_bf16(w.seed, T_VNEW, (le - lb, w.B, w.Hkv, w.D), device, vs, (step * w.L + lb) * nk)
    return q, kn, vn


def profile_inputs(w, p, l, T, device="cpu"):
    """Q [Hq, T, D], K, V [Hkv, T, D] bf16 ~ N(0,1) of prompt p, layer l, for the profiling pass."""
    nq, nk = w.Hq * T * w.D, w.Hkv * T * w.D
    i = p * w.L + l
    return (synth.normal_bf16(w.seed, T_PROFILE_Q, (w.Hq, T, w.D), device, None, i * nq),
            synth.normal_bf16(w.seed, T_PROFILE_K, (w.Hkv, T, w.D), device, None, i * nk),
            synth.normal_bf16(w.seed, T_PROFILE_V, (w.Hkv, T, w.D), device, None, i * nk))
