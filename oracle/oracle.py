"""ctypes front end of the plain-C fp64 oracle in ``mt_oracle.c`` (test infrastructure only).

Models are passed as lists of layer objects with the attributes ``kind, in_ch, out_ch, h, w, relu,
weight, bias`` and optionally ``residual`` (weight: uint16 array of bf16 bit patterns or None; bias: float32
array or None).
Nothing here computes: it only marshals arrays into the C routines.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mt_oracle.c")
_SO = os.path.join(_HERE, "libmt_oracle.so")
_lock = threading.Lock()
_lib = None


def lib_path() -> str:
    return _SO


def build(force: bool = False) -> str:
    """Compile mt_oracle.c with gcc (-O2, OpenMP, no fast-math) next to its source."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
                   "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


class _CLayer(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("in_ch", ctypes.c_int32), ("out_ch", ctypes.c_int32),
                ("h", ctypes.c_int32), ("w", ctypes.c_int32), ("relu", ctypes.c_int32),
                ("residual", ctypes.c_int32), ("weight", ctypes.c_void_p), ("bias", ctypes.c_void_p)]


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        lib.orc_bucket.restype = ctypes.c_int
        lib.orc_bucket.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32] + [ctypes.c_void_p] * 4
        lib.orc_forward_one.restype = ctypes.c_int
        lib.orc_forward_one.argtypes = [ctypes.POINTER(_CLayer), ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        lib.orc_forward_batch.restype = ctypes.c_int
        lib.orc_forward_batch.argtypes = [ctypes.POINTER(ctypes.POINTER(_CLayer)), ctypes.c_void_p, ctypes.c_int32,
                                          ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64,
                                          ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32]
        lib.orc_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().orc_max_threads())


def _pack_model(layers: Sequence, keep: list):
    arr = (_CLayer * len(layers))()
    for i, l in enumerate(layers):
        w = b = None
        if l.weight is not None:
            w = np.ascontiguousarray(l.weight, dtype=np.uint16)
            keep.append(w)
        if l.bias is not None:
            b = np.ascontiguousarray(l.bias, dtype=np.float32)
            keep.append(b)
        arr[i] = _CLayer(int(l.kind), int(l.in_ch), int(l.out_ch), int(l.h), int(l.w), int(l.relu),
                         int(getattr(l, "residual", 0)), w.ctypes.data if w is not None else None,
                         b.ctypes.data if b is not None else None)
    keep.append(arr)
    return arr


def _out_elems(l) -> int:
    return int(l.out_ch) * (int(l.h) * int(l.w) if int(l.kind) in (1, 3) else 1)      # conv3x3 and conv1x1 keep the image


def bucket(model_ids: np.ndarray, n_tenants: int):
    """Stable counting sort: returns (counts[T], offsets[T+1], perm[n], inv[n]) as int32 arrays."""
    ids = np.ascontiguousarray(model_ids, dtype=np.int32)
    n = int(ids.shape[0])
    counts = np.zeros(n_tenants, np.int32)
    offsets = np.zeros(n_tenants + 1, np.int32)
    perm = np.zeros(n, np.int32)
    inv = np.zeros(n, np.int32)
    rc = _load().orc_bucket(ids.ctypes.data, n, n_tenants, counts.ctypes.data, offsets.ctypes.data,
                            perm.ctypes.data, inv.ctypes.data)
    if rc != 0:
        raise ValueError("oracle bucket: model id outside [0, T) (rc=%d)" % rc)
    return counts, offsets, perm, inv


def forward_one(layers: Sequence, x_bf16_bits: np.ndarray) -> np.ndarray:
    """One request through one model; returns float64 [out_elems]."""
    keep: list = []
    arr = _pack_model(layers, keep)
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16).reshape(-1)
    out = np.zeros(_out_elems(layers[-1]), np.float64)
    rc = _load().orc_forward_one(arr, len(layers), x.ctypes.data, out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle forward_one failed (rc=%d)" % rc)
    return out


def forward(models: List[Sequence], model_ids: np.ndarray, inputs_bf16_bits: np.ndarray,
            n_threads: int = 0) -> np.ndarray:
    """The mixed batch, one request at a time: returns float64 [n, out_elems] in arrival order."""
    keep: list = []
    T = len(models)
    ptrs = (ctypes.POINTER(_CLayer) * T)()
    nl = np.zeros(T, np.int32)
    for t, m in enumerate(models):
        ptrs[t] = ctypes.cast(_pack_model(m, keep), ctypes.POINTER(_CLayer))
        nl[t] = len(m)
    ids = np.ascontiguousarray(model_ids, dtype=np.int32)
    n = int(ids.shape[0])
    x = np.ascontiguousarray(inputs_bf16_bits, dtype=np.uint16).reshape(n, -1) if n else \
        np.zeros((0, 0), np.uint16)
    in_elems = int(x.shape[1]) if n else 0
    out_elems = _out_elems(models[0][-1])
    out = np.zeros((n, out_elems), np.float64)
    if n == 0:
        return out
    rc = _load().orc_forward_batch(ptrs, nl.ctypes.data, T, ids.ctypes.data, n, x.ctypes.data, in_elems,
                                   out.ctypes.data, out_elems, int(n_threads))
    if rc != 0:
        raise ValueError("oracle forward failed (rc=%d): bad id or shape" % rc)
    return out
