"""ctypes binding of libbaklava.so: argument marshalling only.

Function names and argument order follow include/baklava.h.  Device buffers are
torch tensors (torch is used for device memory and streams, nothing else); every
step of the method runs inside the library.  If the library is missing the
first call raises: there is no other path.
"""
import ctypes
import os
from ctypes import POINTER, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_uint32, c_void_p

import numpy as np
import torch

OK = 0
FLAG_NO_APPEND, FLAG_NO_SCORE, FLAG_NO_EVICT = 1, 2, 4
FLAG_OVERLAP_PREV = 8
FLAG_TEST_STALL = 256
SCOPE_LAYER, SCOPE_MODEL = 0, 1
STATUS_OVERFLOW, STATUS_BAD_STATE, STATUS_TIMEOUT = 1, 2, 4
KV_BF16, KV_FP8_E4M3 = 0, 1

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbaklava.so")
_lib = None


class BaklavaError(RuntimeError):
    def __init__(self, code, what):
        super().__init__("%s failed: %s (%d)" % (what, strerror(code), code))
        self.code = code


class Shape(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("L", "Hq", "Hkv", "D", "page", "n_sink", "recent_num", "recent_den")]

    @property
    def g(self):
        return self.Hq // self.Hkv


class CacheStruct(ctypes.Structure):
    _fields_ = [("k_slab", c_void_p), ("v_slab", c_void_p), ("pos", c_void_p), ("score", c_void_p),
                ("len", c_void_p), ("free_slot", c_void_p), ("cap", c_void_p), ("slab_off", c_void_p),
                ("seq_stride_tokens", c_int64), ("B", c_int32), ("status", c_void_p), ("kv_dtype", c_int32),
                ("kv_scale", c_void_p)]


class AllocParams(ctypes.Structure):
    _fields_ = [("t", c_double), ("r_num", c_int32), ("r_den", c_int32), ("scope", c_int32),
                ("min_tokens", c_int32), ("max_tokens", c_int32), ("layer_importance", POINTER(c_double)),
                ("t_layer", c_double), ("rl_num", c_int32), ("rl_den", c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("n_items", c_int32), ("n_score_items", c_int32), ("n_units", c_int32), ("chunk_tokens", c_int32),
                ("layer_begin", c_int32), ("layer_end", c_int32), ("B", c_int32), ("ws_bytes", c_int64)]


def lib():
    """The loaded library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libbaklava.so is not built (run `python -m paper_2502_13176_b200.build`); "
                               "there is no fallback path")
        L = ctypes.CDLL(_LIB_PATH)
        L.baklava_strerror.restype = c_char_p
        L.baklava_strerror.argtypes = [ctypes.c_int]
        L.baklava_importance.argtypes = [POINTER(Shape), POINTER(c_float), c_int32, POINTER(c_double)]
        L.baklava_allocate.argtypes = [POINTER(Shape), POINTER(c_double), POINTER(AllocParams), c_int64,
                                       POINTER(c_int32), POINTER(c_int64), POINTER(c_int64)]
        L.baklava_decode_plan.argtypes = [POINTER(Shape), POINTER(c_int32), c_int32, c_int32, c_int32, c_int32,
                                          c_int32, c_int32, c_int64, POINTER(c_int32), c_int64, POINTER(PlanInfo)]
        L.baklava_decode_attn.argtypes = [POINTER(Shape), POINTER(CacheStruct), c_void_p, c_void_p, c_void_p, c_int32,
                                          c_void_p, c_void_p, c_uint32, c_void_p, POINTER(PlanInfo),
                                          c_void_p, c_size_t, c_void_p]
        L.baklava_decode_attn_varlen.argtypes = [POINTER(Shape), POINTER(CacheStruct), c_void_p, c_void_p, c_void_p,
                                                 c_void_p, c_void_p, c_void_p, c_uint32, c_void_p, POINTER(PlanInfo),
                                                 c_void_p, c_size_t, c_void_p]
        L.baklava_evict_varlen.argtypes = [POINTER(Shape), POINTER(CacheStruct), c_int32, c_int32, c_void_p, c_void_p,
                                           c_void_p, c_int32, c_void_p, c_int64, c_int64, c_int64, c_int32, c_void_p,
                                           c_size_t, c_void_p]
        L.baklava_evict.argtypes = [POINTER(Shape), POINTER(CacheStruct), c_int32, c_int32, c_void_p, c_void_p,
                                    c_void_p, c_int32, c_int64, c_int64, c_int64, c_int32, c_void_p, c_size_t, c_void_p]
        L.baklava_evict_workspace_size.restype = c_size_t
        L.baklava_evict_workspace_size.argtypes = [POINTER(Shape), c_int32, c_int32, c_int32]
        L.baklava_evict_static.argtypes = [POINTER(Shape), POINTER(CacheStruct), c_int32, c_int32, c_void_p, c_void_p,
                                           c_void_p, c_int32, c_int64, c_int64, c_int64, c_int32, c_void_p]
        L.baklava_profile_heads.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                            c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.baklava_prefill_scores.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                             c_void_p, c_void_p, c_size_t, c_void_p]
        L.baklava_prefill_workspace_size.restype = c_size_t
        L.baklava_prefill_workspace_size.argtypes = [POINTER(Shape), c_int32, c_int32]
        L.baklava_output_error.argtypes = [c_void_p, c_void_p, c_int64, c_int32, c_void_p, c_void_p, c_size_t, c_void_p]
        L.baklava_output_error_workspace_size.restype = c_size_t
        L.baklava_output_error_workspace_size.argtypes = [c_int64]
        L.baklava_search_pick.argtypes = [POINTER(c_double), c_int32, POINTER(c_int32)]
        L.baklava_set_wait_limit.argtypes = [c_int64]
        L.baklava_profile_workspace_size.restype = c_size_t
        L.baklava_profile_workspace_size.argtypes = [POINTER(Shape), c_int32, c_int32]
        _lib = L
    return _lib


def strerror(code):
    return lib().baklava_strerror(int(code)).decode()


def _check(rc, what):
    if rc != OK:
        raise BaklavaError(rc, what)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def make_shape(L, Hq, Hkv, D, page=16, n_sink=4, recent_num=1, recent_den=2):
    return Shape(L, Hq, Hkv, D, page, n_sink, recent_num, recent_den)


# ------------------------------------------------------------------ host entry points
def baklava_importance(shape, head_cos):
    """head_cos: float32 array [P, L, Hq] -> float64 array [L, Hkv]."""
    hc = np.ascontiguousarray(head_cos, dtype=np.float32)
    P = hc.shape[0]
    assert hc.shape == (P, shape.L, shape.Hq)
    out = np.empty((shape.L, shape.Hkv), dtype=np.float64)
    _check(lib().baklava_importance(ctypes.byref(shape), hc.ctypes.data_as(POINTER(c_float)), P,
                                    out.ctypes.data_as(POINTER(c_double))), "baklava_importance")
    return out


def baklava_allocate(shape, kv_importance, t, r_num, r_den, total_tokens, min_tokens, max_tokens,
                     scope=SCOPE_LAYER, layer_importance=None, t_layer=0.0, rl_num=0, rl_den=1):
    """Returns (cap int32 [L, Hkv], slab_off int64 [L, Hkv], seq_stride int)."""
    imp = np.ascontiguousarray(kv_importance, dtype=np.float64).reshape(shape.L, shape.Hkv)
    li = None if layer_importance is None else np.ascontiguousarray(layer_importance, dtype=np.float64)
    params = AllocParams(t, r_num, r_den, scope, min_tokens, max_tokens,
                         None if li is None else li.ctypes.data_as(POINTER(c_double)), t_layer, rl_num, rl_den)
    cap = np.empty((shape.L, shape.Hkv), dtype=np.int32)
    off = np.empty((shape.L, shape.Hkv), dtype=np.int64)
    stride = c_int64(0)
    _check(lib().baklava_allocate(ctypes.byref(shape), imp.ctypes.data_as(POINTER(c_double)), ctypes.byref(params),
                                  int(total_tokens), cap.ctypes.data_as(POINTER(c_int32)),
                                  off.ctypes.data_as(POINTER(c_int64)), ctypes.byref(stride)), "baklava_allocate")
    return cap, off, int(stride.value)


class Plan:
    """The decode work plan: `items` (int32 [n_items + n_score_items, 4], host) and `info`; `items_dev` after `.to(device)`."""

    def __init__(self, items, info):
        self.items, self.info, self.items_dev = items, info, None

    def to(self, device):
        self.items_dev = torch.from_numpy(self.items).to(device)
        return self


def baklava_decode_plan(shape, cap, B, layer_begin, layer_end, seq_stride_tokens, chunk_tokens=0, n_sm=148, kv_dtype=0):
    cap = np.ascontiguousarray(cap, dtype=np.int32).reshape(shape.L, shape.Hkv)
    info = PlanInfo()
    capp = cap.ctypes.data_as(POINTER(c_int32))
    _check(lib().baklava_decode_plan(ctypes.byref(shape), capp, B, layer_begin, layer_end, chunk_tokens, n_sm, kv_dtype,
                                     int(seq_stride_tokens), None, 0, ctypes.byref(info)), "baklava_decode_plan")
    total = info.n_items + info.n_score_items
    items = np.empty((total, 4), dtype=np.int32)
    _check(lib().baklava_decode_plan(ctypes.byref(shape), capp, B, layer_begin, layer_end, chunk_tokens, n_sm, kv_dtype,
                                     int(seq_stride_tokens), items.ctypes.data_as(POINTER(c_int32)), total,
                                     ctypes.byref(info)), "baklava_decode_plan")
    return Plan(items, info)


# ------------------------------------------------------------------ device state
class Cache:
    """Device buffers of a budgeted cache plus the struct the library reads.  Memory only."""

    def __init__(self, shape, cap, slab_off, seq_stride, B, device="cuda", kv_dtype=KV_BF16, kv_scale=None):
        """kv_scale: float32 array [L, Hkv, 4] = (K scale, 1 / K scale, V scale, 1 / V scale) per head, for FP8
        slabs; passed to the library as given."""
        self.shape, self.B, self.seq_stride = shape, int(B), int(seq_stride)
        self.kv_dtype = int(kv_dtype)
        self.cap_host = np.ascontiguousarray(cap, dtype=np.int32).reshape(shape.L, shape.Hkv)
        self.off_host = np.ascontiguousarray(slab_off, dtype=np.int64).reshape(shape.L, shape.Hkv)
        rows = self.B * self.seq_stride
        slab_type = torch.uint8 if self.kv_dtype == KV_FP8_E4M3 else torch.bfloat16
        self.k_slab = torch.empty((rows, shape.D), dtype=slab_type, device=device)
        self.v_slab = torch.empty((rows, shape.D), dtype=slab_type, device=device)
        self.kv_scale = None
        if self.kv_dtype == KV_FP8_E4M3:
            self.kv_scale_host = np.ascontiguousarray(kv_scale, dtype=np.float32).reshape(shape.L, shape.Hkv, 4).copy()
            self.kv_scale = torch.from_numpy(self.kv_scale_host).to(device)
        self.pos = torch.full((rows,), -1, dtype=torch.int32, device=device)
        self.score = torch.zeros((rows,), dtype=torch.float32, device=device)
        self.len = torch.zeros((self.B, shape.L, shape.Hkv), dtype=torch.int32, device=device)
        self.free_slot = torch.zeros((self.B, shape.L, shape.Hkv), dtype=torch.int32, device=device)
        self.cap = torch.from_numpy(self.cap_host).to(device)
        self.slab_off = torch.from_numpy(self.off_host).to(device)
        self.status = torch.zeros((1,), dtype=torch.int32, device=device)
        self.struct = CacheStruct(self.k_slab.data_ptr(), self.v_slab.data_ptr(), self.pos.data_ptr(),
                                  self.score.data_ptr(), self.len.data_ptr(), self.free_slot.data_ptr(),
                                  self.cap.data_ptr(), self.slab_off.data_ptr(), self.seq_stride, self.B,
                                  self.status.data_ptr(), self.kv_dtype,
                                  None if self.kv_scale is None else self.kv_scale.data_ptr())

    def reset(self):
        self.len.zero_()
        self.free_slot.zero_()
        self.status.zero_()

    def rows(self, b, l, h):
        """Row range [lo, hi) of head (l, h) of sequence b inside the slabs."""
        lo = b * self.seq_stride + int(self.off_host[l, h])
        return lo, lo + int(self.cap_host[l, h])

    def kv_bytes_retained(self):
        """Bytes of K and V rows currently valid (the metric's numerator for one step)."""
        return int(self.len.sum().item()) * self.shape.D * 2 * (1 if self.kv_dtype == KV_FP8_E4M3 else 2)


def decode_workspace(plan, device="cuda"):
    return torch.zeros((int(plan.info.ws_bytes),), dtype=torch.uint8, device=device)


def baklava_decode_attn(shape, cache, q, k_new, v_new, t_pos, out, lse, flags, plan, ws, stream=None):
    _check(lib().baklava_decode_attn(ctypes.byref(shape), ctypes.byref(cache.struct), _ptr(q), _ptr(k_new), _ptr(v_new),
                                     int(t_pos), _ptr(out), _ptr(lse), int(flags), _ptr(plan.items_dev),
                                     ctypes.byref(plan.info), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "baklava_decode_attn")


def baklava_decode_attn_varlen(shape, cache, q, k_new, v_new, t_pos, out, lse, flags, plan, ws, stream=None):
    """t_pos: device int32 [B]; a negative entry idles that sequence for the step."""
    assert t_pos.dtype == torch.int32 and t_pos.numel() == cache.B and t_pos.is_cuda
    _check(lib().baklava_decode_attn_varlen(ctypes.byref(shape), ctypes.byref(cache.struct), _ptr(q), _ptr(k_new),
                                            _ptr(v_new), _ptr(t_pos), _ptr(out), _ptr(lse), int(flags),
                                            _ptr(plan.items_dev), ctypes.byref(plan.info), _ptr(ws),
                                            ws.numel() * ws.element_size(), _stream(stream)),
           "baklava_decode_attn_varlen")


def baklava_set_wait_limit(sm_cycles):
    _check(lib().baklava_set_wait_limit(int(sm_cycles)), "baklava_set_wait_limit")


def workspace_error(ws):
    """The error word baklava_profile_heads / baklava_prefill_scores leave in their workspace (0 = none);
    synchronises."""
    return int(ws[:4].view(torch.int32).item())


def baklava_evict_workspace_size(shape, B, layers, T):
    return int(lib().baklava_evict_workspace_size(ctypes.byref(shape), B, layers, T))


def baklava_evict(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T,
                  stride_layer, stride_seq, stride_head, reserve, ws, stream=None):
    _check(lib().baklava_evict(ctypes.byref(shape), ctypes.byref(cache.struct), layer_begin, layer_end,
                               _ptr(k_dense), _ptr(v_dense), _ptr(score_dense), int(T), int(stride_layer),
                               int(stride_seq), int(stride_head), int(reserve), _ptr(ws),
                               ws.numel() * ws.element_size(), _stream(stream)), "baklava_evict")


def baklava_evict_varlen(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T, prompt_len,
                         stride_layer, stride_seq, stride_head, reserve, ws, stream=None):
    """prompt_len: device int32 [B] or None."""
    _check(lib().baklava_evict_varlen(ctypes.byref(shape), ctypes.byref(cache.struct), layer_begin, layer_end,
                                      _ptr(k_dense), _ptr(v_dense), _ptr(score_dense), int(T), _ptr(prompt_len),
                                      int(stride_layer), int(stride_seq), int(stride_head), int(reserve), _ptr(ws),
                                      ws.numel() * ws.element_size(), _stream(stream)), "baklava_evict_varlen")


EVICT_STATIC_MAX_ENTRIES = 1 << 20


def baklava_evict_static(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T,
                         stride_layer, stride_seq, stride_head, reserve, stream=None):
    """baklava_evict for callers that cannot allocate a workspace: the kept-row list lives in a
    fixed 4 MiB array inside the library.  Calls on one device must not overlap in time."""
    _check(lib().baklava_evict_static(ctypes.byref(shape), ctypes.byref(cache.struct), layer_begin, layer_end,
                                      _ptr(k_dense), _ptr(v_dense), _ptr(score_dense), int(T), int(stride_layer),
                                      int(stride_seq), int(stride_head), int(reserve), _stream(stream)),
           "baklava_evict_static")


def baklava_profile_workspace_size(shape, P, T):
    return int(lib().baklava_profile_workspace_size(ctypes.byref(shape), P, T))


def baklava_profile_heads(shape, q, k, v, prompt_len, P, T, head_cos, token_cos, ws, stream=None):
    _check(lib().baklava_profile_heads(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(prompt_len), P, T,
                                       _ptr(head_cos), _ptr(token_cos), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "baklava_profile_heads")


def baklava_prefill_workspace_size(shape, B, T):
    return int(lib().baklava_prefill_workspace_size(ctypes.byref(shape), B, T))


def baklava_prefill_scores(shape, q, k, prompt_len, B, T, score, ws, stream=None, lse=None):
    _check(lib().baklava_prefill_scores(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(prompt_len), _ptr(lse), B, T, _ptr(score),
                                        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "baklava_prefill_scores")


def baklava_output_error(out, ref, loss, ws, stream=None):
    """out, ref: bf16 tensors of the same shape [..., D]; loss: float64 tensor [1] (device), overwritten."""
    assert out.shape == ref.shape and out.dtype == torch.bfloat16 and ref.dtype == torch.bfloat16
    assert out.is_contiguous() and ref.is_contiguous() and loss.dtype == torch.float64
    D = out.shape[-1]
    rows = out.numel() // D
    _check(lib().baklava_output_error(_ptr(out), _ptr(ref), rows, D, _ptr(loss), _ptr(ws),
                                      ws.numel() * ws.element_size(), _stream(stream)), "baklava_output_error")


def baklava_output_error_workspace_size(rows):
    return int(lib().baklava_output_error_workspace_size(int(rows)))


def baklava_search_pick(avg_loss):
    a = np.ascontiguousarray(avg_loss, dtype=np.float64)
    best = c_int32(-2)
    _check(lib().baklava_search_pick(a.ctypes.data_as(POINTER(c_double)), len(a), ctypes.byref(best)),
           "baklava_search_pick")
    return int(best.value)
