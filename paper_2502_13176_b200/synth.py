"""Seeded synthetic inputs: a counter-based generator that gives the same bits on CPU and GPU.

This module holds no arithmetic of the method.  It only produces inputs, which
the CUDA library and the CPU oracle both receive.

Every value is a pure function of (seed, tensor_id, flat index), so any slice of
a large tensor can be regenerated on its own, on either device:

    key        = mix(seed + GOLDEN * (tensor_id + 1))
    word_j(i)  = mix(key + GOLDEN * (3 i + j + 1))          j = 0, 1, 2

with mix the splitmix64 output function (Steele, Lea, Flood 2014).  A standard
normal deviate is the Irwin-Hall sum of the twelve 16-bit fields of the three
words, (sum - 6 * 65535) / 65536: integer arithmetic plus one exact int -> fp32
conversion and an exact power-of-two scaling, hence bit-identical everywhere.
Its variance is 1 - 2^-32 and its range +-6.
"""
import math

import torch

_MASK = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_CHUNK = 1 << 22


def _s64(x):
    """Python int -> the same 64 bits as a signed value."""
    x &= _MASK
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x, s):
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x):
    x = (x ^ _lsr(x, 30)) * _s64(_C1)
    x = (x ^ _lsr(x, 27)) * _s64(_C2)
    return x ^ _lsr(x, 31)


def _mix_int(x):
    x &= _MASK
    x = ((x ^ (x >> 30)) * _C1) & _MASK
    x = ((x ^ (x >> 27)) * _C2) & _MASK
    return x ^ (x >> 31)


def stream_key(seed, tensor_id):
    return _mix_int(int(seed) + _GOLDEN * (int(tensor_id) + 1))


def _words(key, idx, j):
    """word_j for an int64 tensor of flat indices."""
    ctr = idx * 3 + (j + 1)
    return _mix(ctr * _s64(_GOLDEN) + _s64(key))


def normal_f32(seed, tensor_id, start, count, device="cpu"):
    """`count` approximately N(0,1) fp32 values for flat indices start .. start+count-1."""
    key = stream_key(seed, tensor_id)
    out = torch.empty(count, dtype=torch.float32, device=device)
    for c0 in range(0, count, _CHUNK):
        c1 = min(count, c0 + _CHUNK)
        idx = torch.arange(start + c0, start + c1, dtype=torch.int64, device=device)
        total = torch.zeros(c1 - c0, dtype=torch.int64, device=device)
        for j in range(3):
            w = _words(key, idx, j)
            for f in range(4):
                total += _lsr(w, 16 * f) & 0xFFFF
        out[c0:c1] = (total - 6 * 65535).to(torch.float32) / 65536.0
    return out


def uniform_f64(seed, tensor_id, start, count, device="cpu"):
    """`count` float64 values in (0, 1): (top 53 bits of word_0 + 0.5) / 2^53."""
    key = stream_key(seed, tensor_id)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    w = _lsr(_words(key, idx, 0), 11)
    return (w.to(torch.float64) + 0.5) / float(1 << 53)


def normal_f64(seed, tensor_id, start, count):
    """Box-Muller normals in float64 on the host, for small parameter arrays."""
    u = uniform_f64(seed, tensor_id, 2 * start, 2 * count)
    u1, u2 = u[0::2], u[1::2]
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)


def lognormal_f64(seed, tensor_id, count, sigma, start=0):
    return torch.exp(sigma * normal_f64(seed, tensor_id, start, count))


def normal_bf16(seed, tensor_id, shape, device="cpu", scale=None, start=0):
    """A bf16 tensor of `shape`: N(0,1) deviates times an optional fp32 `scale`
    (broadcast against `shape`), rounded to bf16 once.  `start` is the flat index
    of the first element inside the logical tensor this slice belongs to."""
    count = 1
    for s in shape:
        count *= int(s)
    z = normal_f32(seed, tensor_id, start, count, device).reshape(shape)
    if scale is not None:
        z = z * scale.to(device=device, dtype=torch.float32)
    return z.to(torch.bfloat16)
