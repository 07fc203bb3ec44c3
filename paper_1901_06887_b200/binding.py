"""Thin ctypes binding of libmt.so: the same entry points as include/mt.h, argument marshalling only.

Every step of the inference path runs inside the CUDA library.  There is no fallback: if libmt.so has
not been built (``python -m paper_1901_06887_b200.build``) importing a function from here raises.
torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmt.so")

MT_OK = 0
STATUS_NAMES = {0: "MT_OK", 1: "MT_ERR_INVALID_ARG", 2: "MT_ERR_BAD_MODEL_ID", 3: "MT_ERR_SHAPE",
                4: "MT_ERR_UNSUPPORTED", 5: "MT_ERR_OOM", 6: "MT_ERR_CUDA", 7: "MT_ERR_ARCH",
                8: "MT_ERR_TIMEOUT", 9: "MT_ERR_NOT_INIT", 10: "MT_ERR_NOT_RESIDENT"}

EXPORTS = ["mt_init", "mt_shutdown", "mt_register_model", "mt_infer", "mt_infer_host", "mt_infer_host_async", "mt_release",
           "mt_get_async_status", "mt_status_string", "mt_debug_last_bucketing", "mt_set_kernel_timing",
           "mt_get_kernel_times", "mt_bucket_noalloc", "mt_debug_wait_timeout", "mt_debug_launch_count", "mt_debug_set_option", "mt_debug_empty_launches", "mt_debug_item_cost",
           "mt_debug_schedule_balance", "mt_set_cache_bytes", "mt_prefetch", "mt_get_cache_stats", "mt_cache_sim_create",
           "mt_cache_sim_access", "mt_cache_sim_release", "mt_cache_sim_stats", "mt_cache_sim_destroy", "mt_output_elems", "mt_input_elems"]


class MtError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__("%s failed: %s (%d)" % (where, STATUS_NAMES.get(int(code), "?"), int(code)))


class CacheStats(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint64) for k in ("capacity_bytes", "resident_bytes", "tenant_hits", "tenant_misses",
                                               "request_hits", "request_misses", "evictions", "bytes_loaded")]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class LayerDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("in_ch", ctypes.c_int32), ("out_ch", ctypes.c_int32),
                ("h", ctypes.c_int32), ("w", ctypes.c_int32), ("relu", ctypes.c_int32), ("residual", ctypes.c_int32),
                ("weight", ctypes.c_void_p), ("bias", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libmt.so (once).  Raises if it is missing: there is no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s not built; run `python -m paper_1901_06887_b200.build`" % LIB_PATH)
        l = ctypes.CDLL(LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        l.mt_init.argtypes = [i32, i32, i32]
        l.mt_shutdown.argtypes = []
        l.mt_register_model.argtypes = [ctypes.POINTER(LayerDesc), i32, ctypes.POINTER(i32)]
        l.mt_infer.argtypes = [vp, vp, i32, vp, vp]
        l.mt_infer_host.argtypes = [vp, vp, i32, vp, vp]
        l.mt_infer_host_async.argtypes = [vp, vp, i32, vp, vp]
        l.mt_release.argtypes = [i32]
        l.mt_get_async_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        l.mt_status_string.argtypes = [i32]
        l.mt_status_string.restype = ctypes.c_char_p
        l.mt_debug_last_bucketing.argtypes = [vp] * 4 + [ctypes.POINTER(i32)]
        l.mt_set_kernel_timing.argtypes = [i32]
        l.mt_get_kernel_times.argtypes = [ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_double),
                                          ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
        l.mt_bucket_noalloc.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
        l.mt_debug_wait_timeout.argtypes = [i32, vp]
        l.mt_debug_launch_count.argtypes = [ctypes.POINTER(ctypes.c_int64)]
        l.mt_debug_set_option.argtypes = [ctypes.c_char_p, i32]
        l.mt_debug_empty_launches.argtypes = [i32, vp]
        l.mt_output_elems.argtypes = [ctypes.POINTER(i32)]
        l.mt_input_elems.argtypes = [ctypes.POINTER(i32)]
        l.mt_set_cache_bytes.argtypes = [ctypes.c_size_t]
        l.mt_prefetch.argtypes = [vp, i32, vp]
        l.mt_get_cache_stats.argtypes = [ctypes.POINTER(CacheStats), i32]
        l.mt_cache_sim_create.argtypes = [ctypes.c_size_t, ctypes.POINTER(vp)]
        l.mt_cache_sim_access.argtypes = [vp, i32, ctypes.c_size_t, ctypes.c_uint64, ctypes.POINTER(i32),
                                          ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
        l.mt_cache_sim_release.argtypes = [vp, i32]
        l.mt_cache_sim_stats.argtypes = [vp, ctypes.POINTER(CacheStats)]
        l.mt_cache_sim_destroy.argtypes = [vp]
        l.mt_debug_item_cost.argtypes = [i32, i32, i32, ctypes.POINTER(ctypes.c_double)]
        l.mt_debug_schedule_balance.argtypes = [i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        for name in EXPORTS:
            if name != "mt_status_string":
                getattr(l, name).restype = ctypes.c_int
        _lib = l
    return _lib


def _check(code: int, where: str) -> None:
    if code != MT_OK:
        raise MtError(code, where)


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor (device or host), a numpy array, or None."""
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def mt_init(device: int = 0, max_models: int = 1024, max_batch: int = 0) -> None:
    _check(lib().mt_init(device, max_models, max_batch), "mt_init")


def mt_shutdown() -> None:
    _check(lib().mt_shutdown(), "mt_shutdown")


def mt_register_model(layers: Sequence) -> int:
    """layers: objects with kind, in_ch, out_ch, h, w, relu, weight, bias and optionally residual (weight: uint16 numpy array of bf16
    bit patterns or a torch bf16 tensor, host or device; bias: float32 or None).  Returns the model id."""
    arr = (LayerDesc * len(layers))()
    keep = []
    for i, l in enumerate(layers):
        w, b = l.weight, l.bias
        if isinstance(w, np.ndarray):
            w = np.ascontiguousarray(w, dtype=np.uint16)
        if isinstance(b, np.ndarray):
            b = np.ascontiguousarray(b, dtype=np.float32)
        keep += [w, b]
        arr[i] = LayerDesc(int(l.kind), int(l.in_ch), int(l.out_ch), int(l.h), int(l.w), int(l.relu), int(getattr(l, "residual", 0)),
                           _ptr(w), _ptr(b))
    mid = ctypes.c_int32(-1)
    _check(lib().mt_register_model(arr, len(layers), ctypes.byref(mid)), "mt_register_model")
    return int(mid.value)


def mt_release(model_id: int) -> None:
    _check(lib().mt_release(int(model_id)), "mt_release")


def mt_infer(inputs, model_ids, n: int, outputs, stream=None) -> None:
    """inputs: device bf16 [n, in_elems]; model_ids: device int32 [n]; outputs: device fp32 [n, out_elems]."""
    _check(lib().mt_infer(_ptr(inputs), _ptr(model_ids), int(n), _ptr(outputs), _stream_handle(stream)), "mt_infer")


def mt_infer_host(inputs, model_ids, n: int, outputs, stream=None) -> None:
    """Same with host buffers (pinned torch tensors or numpy arrays); returns after the outputs have landed."""
    _check(lib().mt_infer_host(_ptr(inputs), _ptr(model_ids), int(n), _ptr(outputs), _stream_handle(stream)),
           "mt_infer_host")


def mt_infer_host_async(inputs, model_ids, n: int, outputs, stream=None) -> None:
    """mt_infer_host without the final synchronisation: pinned host buffers, everything enqueued on `stream`.
    Alternate between two streams to overlap one batch's copies with the next batch's kernels; synchronise the
    stream before reading `outputs`."""
    _check(lib().mt_infer_host_async(_ptr(inputs), _ptr(model_ids), int(n), _ptr(outputs), _stream_handle(stream)),
           "mt_infer_host_async")


def mt_get_async_status(stream=None) -> Tuple[int, int]:
    st, bad = ctypes.c_int32(0), ctypes.c_int32(-1)
    _check(lib().mt_get_async_status(_stream_handle(stream), ctypes.byref(st), ctypes.byref(bad)), "mt_get_async_status")
    return int(st.value), int(bad.value)


def mt_status_string(code: int) -> str:
    return lib().mt_status_string(int(code)).decode()


def mt_debug_last_bucketing(n: int):
    """Copies of (counts[T], offsets[T+2], perm[n], inv[n]) of the last mt_infer (batch size n) as numpy int32."""
    T = ctypes.c_int32(0)
    _check(lib().mt_debug_last_bucketing(None, None, None, None, ctypes.byref(T)), "mt_debug_last_bucketing")
    arrs = [np.zeros(T.value, np.int32), np.zeros(T.value + 2, np.int32), np.zeros(n, np.int32), np.zeros(n, np.int32)]
    _check(lib().mt_debug_last_bucketing(*[a.ctypes.data for a in arrs], None), "mt_debug_last_bucketing")
    return tuple(arrs)


def mt_debug_wait_timeout(limit_ms: int = 20, stream=None) -> None:
    """Enqueue the bounded-wait self-test (a wait nothing satisfies); mt_get_async_status then reports MT_ERR_TIMEOUT."""
    _check(lib().mt_debug_wait_timeout(int(limit_ms), _stream_handle(stream)), "mt_debug_wait_timeout")


def mt_debug_launch_count() -> int:
    """Kernels enqueued by mt_infer / mt_infer_host since the library was loaded."""
    c = ctypes.c_int64(0)
    _check(lib().mt_debug_launch_count(ctypes.byref(c)), "mt_debug_launch_count")
    return int(c.value)


def mt_output_elems() -> int:
    """Row stride (elements) of mt_infer's output buffer: the widest registered model's output width."""
    v = ctypes.c_int32(0)
    _check(lib().mt_output_elems(ctypes.byref(v)), "mt_output_elems")
    return int(v.value)


def mt_input_elems() -> int:
    """Row stride (elements) of mt_infer's input buffer: the widest registered model's input width."""
    v = ctypes.c_int32(0)
    _check(lib().mt_input_elems(ctypes.byref(v)), "mt_input_elems")
    return int(v.value)


def mt_set_cache_bytes(device_bytes: int) -> None:
    """Switch to a weight cache of this many device bytes (0: every model resident).  Only while no model is registered."""
    _check(lib().mt_set_cache_bytes(int(device_bytes)), "mt_set_cache_bytes")


def mt_prefetch(model_ids, stream=None) -> None:
    """Make these tenants (host ints) resident for work enqueued on `stream` afterwards."""
    ids = np.ascontiguousarray(model_ids, dtype=np.int32)
    _check(lib().mt_prefetch(ids.ctypes.data, int(ids.size), _stream_handle(stream)), "mt_prefetch")


def mt_get_cache_stats(reset: bool = False) -> dict:
    st = CacheStats()
    _check(lib().mt_get_cache_stats(ctypes.byref(st), int(bool(reset))), "mt_get_cache_stats")
    return st.as_dict()


def mt_cache_sim_create(capacity_bytes: int):
    """A stand-alone instance of the cache's policy (host code of the library; needs no GPU).  Returns its handle."""
    h = ctypes.c_void_p()
    _check(lib().mt_cache_sim_create(int(capacity_bytes), ctypes.byref(h)), "mt_cache_sim_create")
    return h


def mt_cache_sim_access(sim, model_id: int, nbytes: int, tick: int):
    """Returns (result, offset, evicted ids): result 0 hit, 1 placed, -1 no room."""
    res, off, n = ctypes.c_int32(0), ctypes.c_int64(0), ctypes.c_int32(0)
    ev = (ctypes.c_int32 * 4096)()
    _check(lib().mt_cache_sim_access(sim, int(model_id), int(nbytes), int(tick), ctypes.byref(res), ctypes.byref(off),
                                     ev, 4096, ctypes.byref(n)), "mt_cache_sim_access")
    return int(res.value), int(off.value), [int(ev[i]) for i in range(min(n.value, 4096))]


def mt_cache_sim_release(sim, model_id: int) -> None:
    _check(lib().mt_cache_sim_release(sim, int(model_id)), "mt_cache_sim_release")


def mt_cache_sim_stats(sim) -> dict:
    st = CacheStats()
    _check(lib().mt_cache_sim_stats(sim, ctypes.byref(st)), "mt_cache_sim_stats")
    return st.as_dict()


def mt_cache_sim_destroy(sim) -> None:
    _check(lib().mt_cache_sim_destroy(sim), "mt_cache_sim_destroy")


def mt_debug_item_cost(k_blocks: int, n_cols: int, rows: int) -> float:
    """Modelled SM cycles of one dense work item (host code only; needs no GPU)."""
    c = ctypes.c_double(0.0)
    _check(lib().mt_debug_item_cost(int(k_blocks), int(n_cols), int(rows), ctypes.byref(c)), "mt_debug_item_cost")
    return float(c.value)


def mt_debug_schedule_balance(layer: int) -> Tuple[float, int, int]:
    """(heaviest CTA's modelled cost / mean, work items, CTAs) of a dense layer of the last mt_infer."""
    r, n, g = ctypes.c_double(0.0), ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().mt_debug_schedule_balance(int(layer), ctypes.byref(r), ctypes.byref(n), ctypes.byref(g)),
           "mt_debug_schedule_balance")
    return float(r.value), int(n.value), int(g.value)


def mt_debug_empty_launches(count: int, stream=None) -> None:
    """Enqueue `count` empty kernels chained like the kernels of the path (to time the launch floor)."""
    _check(lib().mt_debug_empty_launches(int(count), _stream_handle(stream)), "mt_debug_empty_launches")


def mt_debug_set_option(name: str, value: int) -> None:
    """Switch an executor choice ("fused", "pair", "conv_pair", "pool_head") on or off for the calls that follow."""
    _check(lib().mt_debug_set_option(name.encode(), int(value)), "mt_debug_set_option")


def mt_set_kernel_timing(enable) -> None:
    """0/False off, 1/True every kernel, 2 only the grouped layer executors, 3 the same on every fourth call."""
    _check(lib().mt_set_kernel_timing(int(enable)), "mt_set_kernel_timing")


def mt_get_kernel_times() -> List[Tuple[str, float, int]]:
    cap = 16
    names = (ctypes.c_char_p * cap)()
    ms = (ctypes.c_double * cap)()
    cnt = (ctypes.c_int32 * cap)()
    n = ctypes.c_int32(0)
    _check(lib().mt_get_kernel_times(names, ms, cnt, cap, ctypes.byref(n)), "mt_get_kernel_times")
    return [(names[i].decode(), float(ms[i]), int(cnt[i])) for i in range(n.value)]


def mt_bucket_noalloc(model_ids, n: int, n_models: int, counts_out, offsets_out, perm_out, inv_out, stream=None) -> None:
    """Stable bucketing of a batch by model id for callers that must not allocate device memory (allocator
    hooks, frozen-memory serving loops): all six buffers are the caller's device tensors, the scratch is a
    fixed array inside the library.  Limits: n <= 65536, n_models <= 1024 (else MtError MT_ERR_UNSUPPORTED).
    Calls that overlap on the GPU share that scratch and race."""
    _check(lib().mt_bucket_noalloc(_ptr(model_ids), int(n), int(n_models), _ptr(counts_out), _ptr(offsets_out),
                                   _ptr(perm_out), _ptr(inv_out), _stream_handle(stream)), "mt_bucket_noalloc")
