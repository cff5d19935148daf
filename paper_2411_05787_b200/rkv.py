"""Thin ctypes binding of librkv.so: argument marshalling only.

Every step of the RefreshKV decode path runs inside the CUDA library; this
module turns torch tensors into device pointers and checks status codes.
torch is used for device memory and streams only.  There is no fallback: if
the shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "librkv.so")

RKV_OK = 0
AGG_MAX, AGG_MEAN, AGG_FIRST = 0, 1, 2
DEV_APPEND_OVERFLOW, DEV_LEN_CLAMPED, DEV_NONFINITE, DEV_BAD_INDEX, DEV_TIMEOUT = 1, 2, 4, 8, 16

EXPORTS = ["rkv_create", "rkv_destroy", "rkv_workspace_bytes", "rkv_full_step", "rkv_gather_small",
           "rkv_small_step", "rkv_append", "rkv_should_refresh", "rkv_get_device_status",
           "rkv_status_string", "rkv_last_cuda_error", "rkv_launch_count", "rkv_set_profiling", "rkv_get_profile",
           "rkv_set_option", "rkv_small_step_noalloc", "rkv_append_small_step", "rkv_score_step",
           "rkv_gather_small_evict", "rkv_append_small_step_evict", "rkv_full_attention", "rkv_select_topk",
           "rkv_append_full_attention", "rkv_get_option", "rkv_score_keys"]
NOALLOC_MAX_PROBLEMS, NOALLOC_MAX_LEN = 32, 65536
OPT_SMALL_MIN_CHUNK, OPT_DEPENDENT_LAUNCH, OPT_SMALL_CLUSTER, OPT_EARLY_CACHE_READ, OPT_INTERLEAVE_TILES = 1, 2, 3, 4, 5
OPT_SELECT_KEYS_PER_CTA = 6
OPT_SCORE_SLICE = 7
KERNEL_NAMES = ["attn_full", "select", "attn_small", "gather", "append", "trigger", "fold", "score"]


class RkvConfig(ctypes.Structure):
    _fields_ = [("n_seq", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("max_len", ctypes.c_int32), ("max_small", ctypes.c_int32),
                ("agg", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("softmax_scale", ctypes.c_float)]


class RkvCache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("n_rows", ctypes.c_int64),
                ("row_offset", ctypes.c_void_p), ("cap", ctypes.c_void_p), ("len", ctypes.c_void_p)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it first (python -m paper_2411_05787_b200.build); "
                          "there is no CPU or PyTorch fallback for this library")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    cfgp, cachep = ctypes.POINTER(RkvConfig), ctypes.POINTER(RkvCache)
    lib.rkv_create.argtypes = [cfgp, ctypes.POINTER(vp)]
    lib.rkv_destroy.argtypes = [vp]
    lib.rkv_workspace_bytes.argtypes = [cfgp]
    lib.rkv_workspace_bytes.restype = ctypes.c_size_t
    lib.rkv_full_step.argtypes = [vp, vp, cachep, vp, i32, vp, vp, vp, i64, vp, vp, i32, vp]
    lib.rkv_gather_small_evict.argtypes = [vp, vp, vp, i32, cachep, cachep, vp, vp, vp, i32, vp]
    lib.rkv_gather_small_evict.restype = i32
    lib.rkv_append_small_step_evict.argtypes = [vp, vp, vp, vp, cachep, cachep, vp, vp, vp, vp, vp, i32, i32, vp]
    lib.rkv_append_small_step_evict.restype = i32
    lib.rkv_score_step.argtypes = [vp, vp, cachep, vp, i32, vp, vp, i64, vp, vp, i32, vp]
    lib.rkv_score_step.restype = i32
    lib.rkv_full_attention.argtypes = [vp, vp, cachep, vp, vp, i32, vp]
    lib.rkv_full_attention.restype = i32
    lib.rkv_append_full_attention.argtypes = [vp, vp, vp, vp, cachep, vp, vp, i32, vp]
    lib.rkv_append_full_attention.restype = i32
    lib.rkv_select_topk.argtypes = [vp, vp, cachep, vp, i32, vp, vp, i64, vp, vp, vp]
    lib.rkv_select_topk.restype = i32
    lib.rkv_score_keys.argtypes = [vp, vp, cachep, vp, i32, vp, vp, i64, vp, vp]
    lib.rkv_score_keys.restype = i32
    lib.rkv_gather_small.argtypes = [vp, vp, vp, i32, cachep, cachep, vp, vp]
    lib.rkv_small_step.argtypes = [vp, vp, cachep, vp, vp, i32, vp]
    lib.rkv_append.argtypes = [vp, vp, vp, cachep, cachep, vp]
    lib.rkv_append_small_step.argtypes = [vp, vp, vp, vp, cachep, cachep, vp, vp, i32, vp]
    lib.rkv_append_small_step.restype = i32
    lib.rkv_should_refresh.argtypes = [vp, vp, vp, f32, vp, vp, vp, vp]
    lib.rkv_get_device_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    lib.rkv_status_string.argtypes = [i32]
    lib.rkv_status_string.restype = ctypes.c_char_p
    lib.rkv_last_cuda_error.argtypes = [vp]
    lib.rkv_last_cuda_error.restype = ctypes.c_char_p
    lib.rkv_launch_count.argtypes = [vp]
    lib.rkv_launch_count.restype = i64
    lib.rkv_set_option.argtypes = [vp, i32, i32]
    lib.rkv_set_option.restype = i32
    lib.rkv_get_option.argtypes = [vp, i32, ctypes.POINTER(i32)]
    lib.rkv_get_option.restype = i32
    lib.rkv_set_profiling.argtypes = [vp, i32]
    lib.rkv_set_profiling.restype = i32
    lib.rkv_get_profile.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    lib.rkv_get_profile.restype = i32
    lib.rkv_small_step_noalloc.argtypes = [cfgp, vp, cachep, vp, vp, i32, vp, vp, ctypes.c_char_p, ctypes.c_size_t]
    lib.rkv_small_step_noalloc.restype = i32
    for name in ("rkv_create", "rkv_destroy", "rkv_full_step", "rkv_gather_small", "rkv_small_step",
                 "rkv_append", "rkv_should_refresh", "rkv_get_device_status"):
        getattr(lib, name).restype = i32
    return lib


lib = _load()


class RkvError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        msg = lib.rkv_status_string(code).decode()
        super().__init__(f"rkv status {code} ({msg}){': ' + detail if detail else ''}")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("librkv takes device tensors")
    if not t.is_contiguous():
        raise ValueError("librkv takes contiguous tensors")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def cache_struct(k, v, row_offset, cap, length) -> RkvCache:
    """Describe a packed K/V cache (see include/rkv.h).  The caller keeps the tensors alive."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.shape == v.shape and k.shape[-1] == 128
    assert row_offset.dtype == torch.int64 and cap.dtype == torch.int32 and length.dtype == torch.int32
    return RkvCache(_ptr(k), _ptr(v), k.numel() // 128, _ptr(row_offset), _ptr(cap), _ptr(length))


def small_step_noalloc(cfg: RkvConfig, q, small: RkvCache, out, active=None, max_len_hint=0, device_status=None,
                       stream=None):
    """Partial step for callers that may not allocate device memory (no context; see include/rkv.h).

    Raises RkvError carrying the library's one-line reason, e.g. when a size exceeds the static scratch."""
    msg = ctypes.create_string_buffer(256)
    rc = lib.rkv_small_step_noalloc(ctypes.byref(cfg), _ptr(q), ctypes.byref(small), _ptr(active), _ptr(out),
                                    max_len_hint, _ptr(device_status), _stream(stream), msg, len(msg))
    if rc != RKV_OK:
        raise RkvError(rc, msg.value.decode())


class Context:
    """Owns one rkv_ctx (its scratch workspace).  Calls on one context share one stream."""

    def __init__(self, n_seq, n_q_heads, n_kv_heads, max_len, max_small, agg=AGG_MAX, pool_kernel=1,
                 softmax_scale=0.0, head_dim=128):
        self.cfg = RkvConfig(n_seq, n_q_heads, n_kv_heads, head_dim, max_len, max_small, agg, pool_kernel,
                             softmax_scale)
        handle = ctypes.c_void_p()
        rc = lib.rkv_create(ctypes.byref(self.cfg), ctypes.byref(handle))
        if rc != RKV_OK:
            raise RkvError(rc)
        self._h = handle

    def close(self):
        if getattr(self, "_h", None):
            lib.rkv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != RKV_OK:
            raise RkvError(rc, lib.rkv_last_cuda_error(self._h).decode())

    @property
    def workspace_bytes(self) -> int:
        return lib.rkv_workspace_bytes(ctypes.byref(self.cfg))

    @property
    def launch_count(self) -> int:
        return lib.rkv_launch_count(self._h)

    def full_step(self, q, full: RkvCache, k_small, k_max, out, topk_idx, active=None, scores=None,
                  q_last_full=None, max_len_hint=0, stream=None):
        stride = scores.shape[-1] if scores is not None else 0
        self._check(lib.rkv_full_step(self._h, _ptr(q), ctypes.byref(full), _ptr(k_small), k_max, _ptr(active),
                                      _ptr(out), _ptr(scores), stride, _ptr(topk_idx), _ptr(q_last_full),
                                      max_len_hint, _stream(stream)))

    def score_step(self, q, full: RkvCache, k_small, k_max, topk_idx, active=None, scores=None, q_last_full=None,
                   max_len_hint=0, stream=None):
        stride = scores.shape[-1] if scores is not None else 0
        self._check(lib.rkv_score_step(self._h, _ptr(q), ctypes.byref(full), _ptr(k_small), k_max, _ptr(active),
                                       _ptr(scores), stride, _ptr(topk_idx), _ptr(q_last_full), max_len_hint,
                                       _stream(stream)))

    def full_attention(self, q, full: RkvCache, out, active=None, max_len_hint=0, stream=None):
        self._check(lib.rkv_full_attention(self._h, _ptr(q), ctypes.byref(full), _ptr(active), _ptr(out),
                                           max_len_hint, _stream(stream)))

    def append_full_attention(self, q, k_new, v_new, full: RkvCache, out, active=None, max_len_hint=0, stream=None):
        self._check(lib.rkv_append_full_attention(self._h, _ptr(q), _ptr(k_new), _ptr(v_new), ctypes.byref(full),
                                                  _ptr(active), _ptr(out), max_len_hint, _stream(stream)))

    def select_topk(self, q, full: RkvCache, k_small, k_max, topk_idx, active=None, scores=None, q_last_full=None,
                    stream=None):
        stride = scores.shape[-1] if scores is not None else 0
        self._check(lib.rkv_select_topk(self._h, _ptr(q), ctypes.byref(full), _ptr(k_small), k_max, _ptr(active),
                                        _ptr(scores), stride, _ptr(topk_idx), _ptr(q_last_full), _stream(stream)))

    def score_keys(self, q, full: RkvCache, k_small, k_max, active=None, scores=None, q_last_full=None, stream=None):
        """The score pass alone; the next select_topk (scores=None, q_last_full=None) launches the selection alone."""
        stride = scores.shape[-1] if scores is not None else 0
        self._check(lib.rkv_score_keys(self._h, _ptr(q), ctypes.byref(full), _ptr(k_small), k_max, _ptr(active),
                                       _ptr(scores), stride, _ptr(q_last_full), _stream(stream)))

    def gather_small(self, topk_idx, k_small, k_max, full: RkvCache, small: RkvCache, active=None, stream=None):
        self._check(lib.rkv_gather_small(self._h, _ptr(topk_idx), _ptr(k_small), k_max, ctypes.byref(full),
                                         ctypes.byref(small), _ptr(active), _stream(stream)))

    def small_step(self, q, small: RkvCache, out, active=None, max_len_hint=0, stream=None):
        self._check(lib.rkv_small_step(self._h, _ptr(q), ctypes.byref(small), _ptr(active), _ptr(out),
                                       max_len_hint, _stream(stream)))

    def append(self, k_new, v_new, full: RkvCache | None, small: RkvCache | None, stream=None):
        self._check(lib.rkv_append(self._h, _ptr(k_new), _ptr(v_new),
                                   ctypes.byref(full) if full is not None else None,
                                   ctypes.byref(small) if small is not None else None, _stream(stream)))

    def append_small_step(self, q, k_new, v_new, full: RkvCache | None, small: RkvCache, out, active=None,
                          max_len_hint=0, stream=None):
        self._check(lib.rkv_append_small_step(self._h, _ptr(q), _ptr(k_new), _ptr(v_new),
                                              ctypes.byref(full) if full is not None else None, ctypes.byref(small),
                                              _ptr(active), _ptr(out), max_len_hint, _stream(stream)))

    def gather_small_evict(self, topk_idx, k_small, k_max, full: RkvCache, small: RkvCache, evict_order, evict_count,
                           active=None, stream=None):
        self._check(lib.rkv_gather_small_evict(self._h, _ptr(topk_idx), _ptr(k_small), k_max, ctypes.byref(full),
                                               ctypes.byref(small), _ptr(active), _ptr(evict_order), _ptr(evict_count),
                                               evict_order.shape[-1], _stream(stream)))

    def append_small_step_evict(self, q, k_new, v_new, full: RkvCache | None, small: RkvCache, k_small, out,
                                evict_order, evict_count, active=None, max_len_hint=0, stream=None):
        self._check(lib.rkv_append_small_step_evict(self._h, _ptr(q), _ptr(k_new), _ptr(v_new),
                                                    ctypes.byref(full) if full is not None else None,
                                                    ctypes.byref(small), _ptr(k_small), _ptr(active), _ptr(out),
                                                    _ptr(evict_order), _ptr(evict_count), evict_order.shape[-1],
                                                    max_len_hint, _stream(stream)))

    def should_refresh(self, q_now, q_last_full, threshold, flag, sim=None, keep=None, stream=None):
        self._check(lib.rkv_should_refresh(self._h, _ptr(q_now), _ptr(q_last_full), float(threshold), _ptr(flag),
                                           _ptr(keep), _ptr(sim), _stream(stream)))

    def set_option(self, option: int, value: int):
        self._check(lib.rkv_set_option(self._h, option, value))

    def get_option(self, option: int) -> int:
        value = ctypes.c_int32(0)
        self._check(lib.rkv_get_option(self._h, option, ctypes.byref(value)))
        return value.value

    def set_profiling(self, on: bool):
        self._check(lib.rkv_set_profiling(self._h, 1 if on else 0))

    def get_profile(self) -> dict:
        """{kernel name: (total microseconds, launches)} since the last call; waits for the recorded events."""
        us = (ctypes.c_double * len(KERNEL_NAMES))()
        cnt = (ctypes.c_int64 * len(KERNEL_NAMES))()
        self._check(lib.rkv_get_profile(self._h, us, cnt))
        return {n: (us[i], cnt[i]) for i, n in enumerate(KERNEL_NAMES)}

    def device_status(self, stream=None) -> int:
        """Synchronises the stream; returns and clears the sticky device status bits."""
        bits = ctypes.c_int32(0)
        rc = lib.rkv_get_device_status(self._h, ctypes.byref(bits), _stream(stream))
        if rc not in (RKV_OK, 5):
            raise RkvError(rc, lib.rkv_last_cuda_error(self._h).decode())
        return bits.value
