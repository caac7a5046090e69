"""Thin ctypes binding of libmeda.so: same names as include/meda.h, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every step of the pass runs in
the library's kernels.  There is no fallback: if the library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .workloads import Workload

_LIB = None

MEDA_OK = 0
MEDA_ERR_INVALID_ARG = -1
MEDA_ERR_SHAPE = -2
MEDA_ERR_BUDGET_INFEASIBLE = -3
MEDA_ERR_WORKSPACE = -4
MEDA_ERR_CUDA = -5
MEDA_ERR_UNSUPPORTED = -6
MEDA_ERR_TIMEOUT = -7

N_KERNEL_CLASSES = 12
NEAREST_SMALL_MAX_S = 384   # kNearestSmallMaxS: layers keeping at most this many slots take the streaming arg-max kernel

MEDA_BF16 = 0
MEDA_F32 = 1


class MedaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class meda_span(ctypes.Structure):
    _fields_ = [("begin", ctypes.c_int32), ("end", ctypes.c_int32), ("modality", ctypes.c_int32)]


class meda_config(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("n_tokens", ctypes.c_int32), ("window", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("global_budget", ctypes.c_int64),
        ("beta_recent", ctypes.c_int32), ("beta_important", ctypes.c_int32),
        ("min_budget", ctypes.c_int32), ("entropy_mode", ctypes.c_int32),
        ("alloc_mode", ctypes.c_int32), ("merge_mode", ctypes.c_int32),
    ]


EXPORTS = {
    # name: (restype, argtypes)
    "meda_create": (ctypes.c_int, [ctypes.POINTER(meda_config), ctypes.POINTER(meda_span), ctypes.c_int32,
                                   ctypes.POINTER(ctypes.c_void_p)]),
    "meda_destroy": (None, [ctypes.c_void_p]),
    "meda_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "meda_workspace_bytes": (ctypes.c_int64, [ctypes.c_void_p]),
    "meda_poll_status": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "meda_kernel_class_name": (ctypes.c_char_p, [ctypes.c_int32]),
    "meda_profile_enable": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32]),
    "meda_profile_read": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]),
    "meda_launch_count": (ctypes.c_int64, [ctypes.c_void_p]),
    "meda_profile_dropped": (ctypes.c_int64, [ctypes.c_void_p]),
    "meda_selftest_wait_timeout": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]),
    "meda_window_scores": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 6),
    "meda_window_scores_from_stats": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 6),
    "meda_prompt_scores_scratch_bytes": (ctypes.c_int64, [ctypes.c_void_p]),
    "meda_prompt_scores": (ctypes.c_int, [ctypes.c_void_p] * 5 + [ctypes.c_int64, ctypes.c_void_p]),
    "meda_layer_entropy": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 5 +
                           [ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]),
    "meda_decode_attention": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 4 +
                              [ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]),
    "meda_row_stats_static": (ctypes.c_int, [ctypes.c_void_p] * 3 + [ctypes.c_int32] * 6 + [ctypes.c_void_p] * 2),
    "meda_allocate_budgets": (ctypes.c_int, [ctypes.c_void_p] * 4),
    "meda_select_topk": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 4 +
                         [ctypes.c_int32, ctypes.c_void_p]),
    "meda_merge_kv": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 9 +
                      [ctypes.c_int32, ctypes.c_void_p]),
    "meda_compress_layer": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 8 +
                            [ctypes.c_int32, ctypes.c_void_p]),
}


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmeda.so")


def load_library():
    """Loads libmeda.so (once).  Raises if it has not been built: there is no other code path."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2502_17599_b200.build` "
                               "(or __graft_entry__.build()); there is no fallback implementation")
        lib = ctypes.CDLL(path)
        for name, (restype, argtypes) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = restype
            fn.argtypes = argtypes
        _LIB = lib
    return _LIB


def status_string(status: int) -> str:
    return load_library().meda_status_string(int(status)).decode()


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device pointers must come from contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != MEDA_OK:
        raise MedaError(status, where)


STATIC_STATS_MAX_ROWS = 4096


def row_stats_static(q_win, k, modality, row_stats, stream=None):
    """meda_row_stats_static: the window rows' softmax normalisers without a context and without
    any device allocation, for callers that cannot call cudaMalloc (all of device memory already
    belongs to their own pool, or they are inside a section that must not synchronise the device).
    Shapes are read from the tensors: q_win [Hq, w, d], k [Hkv, n, d], modality uint8 [n],
    row_stats fp32 [Hq, w, 4].  Calls that overlap on one GPU race on the library's fixed scratch
    array; the first call on a device should come before any stream capture."""
    hq, w, d = q_win.shape
    hkv, n, _ = k.shape
    dtype = MEDA_F32 if q_win.dtype == torch.float32 else MEDA_BF16
    _check(load_library().meda_row_stats_static(_ptr(q_win), _ptr(k), _ptr(modality), hq, hkv, d, n, w, dtype,
                                                _ptr(row_stats), _stream(stream)), "meda_row_stats_static")


class Context:
    """Owns one meda_ctx.  Method names and argument order follow include/meda.h."""

    def __init__(self, *, n_layers, n_q_heads, n_kv_heads, head_dim, n_tokens, window, dtype, global_budget,
                 spans, beta_recent=3, beta_important=1, min_budget=None, entropy_mode=0, alloc_mode=0,
                 merge_mode=0):
        lib = load_library()
        self.cfg = meda_config(n_layers, n_q_heads, n_kv_heads, head_dim, n_tokens, window,
                               MEDA_F32 if dtype in ("f32", torch.float32) else MEDA_BF16,
                               int(global_budget), beta_recent, beta_important,
                               int(window if min_budget is None else min_budget), entropy_mode, alloc_mode, merge_mode)
        arr = (meda_span * len(spans))(*[meda_span(int(b), int(e), int(m)) for b, e, m in spans])
        handle = ctypes.c_void_p()
        self._h = None
        _check(lib.meda_create(ctypes.byref(self.cfg), arr, len(spans), ctypes.byref(handle)), "meda_create")
        self._h = handle
        self._lib = lib

    @classmethod
    def for_workload(cls, wl: Workload, **overrides) -> "Context":
        kw = dict(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                  n_tokens=wl.n_tokens, window=wl.window, dtype=wl.dtype, global_budget=wl.global_budget,
                  spans=wl.spans, min_budget=wl.min_budget)
        kw.update(overrides)
        return cls(**kw)

    def close(self):
        if self._h is not None:
            self._lib.meda_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self) -> int:
        return int(self._lib.meda_workspace_bytes(self._h))

    def launch_count(self) -> int:
        return int(self._lib.meda_launch_count(self._h))

    def profile_enable(self, enable: bool = True):
        _check(self._lib.meda_profile_enable(self._h, 1 if enable else 0), "meda_profile_enable")

    def profile_read(self) -> dict:
        """{kernel class name: (summed ms, timed launches)} since the last read."""
        n = N_KERNEL_CLASSES
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int32 * n)()
        _check(self._lib.meda_profile_read(self._h, ms, cnt), "meda_profile_read")
        return {self._lib.meda_kernel_class_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

    def profile_dropped(self) -> int:
        """Launches since the last profile_read that went untimed because the event pool was full."""
        return int(self._lib.meda_profile_dropped(self._h))

    def selftest_wait_timeout(self, wait_cycles: int = 20000, stream=None):
        _check(self._lib.meda_selftest_wait_timeout(self._h, int(wait_cycles), _stream(stream)),
               "meda_selftest_wait_timeout")

    def poll_status(self, stream=None) -> int:
        return int(self._lib.meda_poll_status(self._h, _stream(stream)))

    def check(self, stream=None):
        _check(self.poll_status(stream), "device status")

    def window_scores(self, layer, q_win, k, row_stats, scores, entropy=None, stream=None):
        _check(self._lib.meda_window_scores(self._h, layer, _ptr(q_win), _ptr(k), _ptr(row_stats), _ptr(scores),
                                            _ptr(entropy), _stream(stream)), "meda_window_scores")

    def window_scores_from_stats(self, layer, q_win, k, row_stats, scores, entropy=None, stream=None):
        _check(self._lib.meda_window_scores_from_stats(self._h, layer, _ptr(q_win), _ptr(k), _ptr(row_stats),
                                                       _ptr(scores), _ptr(entropy), _stream(stream)),
               "meda_window_scores_from_stats")

    def prompt_scores_scratch_bytes(self) -> int:
        return int(self._lib.meda_prompt_scores_scratch_bytes(self._h))

    def prompt_scores(self, q_all, k, scores, scratch=None, stream=None):
        """Eq. 8 over every prompt row.  `scratch`: a uint8 device tensor of at least
        prompt_scores_scratch_bytes() bytes (None only when that is 0)."""
        nbytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
        _check(self._lib.meda_prompt_scores(self._h, _ptr(q_all), _ptr(k), _ptr(scores), _ptr(scratch), nbytes,
                                            _stream(stream)), "meda_prompt_scores")

    def layer_entropy(self, layer, q_win, k, row_stats, entropy, q_vis=None, q_vis_pos=None, n_vis_rows=0, stream=None):
        _check(self._lib.meda_layer_entropy(self._h, layer, _ptr(q_win), _ptr(k), _ptr(row_stats), _ptr(q_vis),
                                            _ptr(q_vis_pos), n_vis_rows, _ptr(entropy), _stream(stream)),
               "meda_layer_entropy")

    def allocate_budgets(self, entropy, budgets, stream=None):
        _check(self._lib.meda_allocate_budgets(self._h, _ptr(entropy), _ptr(budgets), _stream(stream)),
               "meda_allocate_budgets")

    def select_topk(self, layer, scores, budgets, idx_conserved, idx_less, out_capacity, stream=None):
        _check(self._lib.meda_select_topk(self._h, layer, _ptr(scores), _ptr(budgets), _ptr(idx_conserved),
                                          _ptr(idx_less), out_capacity, _stream(stream)), "meda_select_topk")

    def merge_kv(self, layer, k, v, budgets, idx_conserved, idx_less, k_out, v_out, counts, target, out_capacity,
                 stream=None):
        _check(self._lib.meda_merge_kv(self._h, layer, _ptr(k), _ptr(v), _ptr(budgets), _ptr(idx_conserved),
                                       _ptr(idx_less), _ptr(k_out), _ptr(v_out), _ptr(counts), _ptr(target),
                                       out_capacity, _stream(stream)), "meda_merge_kv")

    def compress_layer(self, layer, k, v, scores, budgets, k_out, v_out, counts, idx_conserved, out_capacity,
                       stream=None):
        _check(self._lib.meda_compress_layer(self._h, layer, _ptr(k), _ptr(v), _ptr(scores), _ptr(budgets),
                                             _ptr(k_out), _ptr(v_out), _ptr(counts), _ptr(idx_conserved),
                                             out_capacity, _stream(stream)), "meda_compress_layer")

    def decode_attention(self, layer, q, k_cache, v_cache, out, budgets=None, n_rows=0, capacity=None, stream=None):
        cap = k_cache.shape[1] if capacity is None else capacity
        _check(self._lib.meda_decode_attention(self._h, layer, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(budgets),
                                               int(n_rows), int(cap), _ptr(out), _stream(stream)), "meda_decode_attention")

