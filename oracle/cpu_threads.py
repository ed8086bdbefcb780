"""Python face of the multi-core fp32 CPU baseline.  TEST INFRASTRUCTURE ONLY.

``densify_threads`` calls the column-parallel loop in ``dst_cpu_threads.c``: the scatter-sum of the
paper's Section 4 (Listing 1) followed by the reduction of Algorithm 1, in fp32, one thread per block
of columns.  The benchmark times it beside the fp64 oracle as "a plain CPU loop on every core"; the
CUDA library and its binding never import this module, and it never imports them.

Pin: ``tests/test_cpu_threads.py`` (against the fp64 oracle; bit-exact on small-integer data).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dst_cpu_threads.c")
_LIB = os.path.join(_HERE, "libdst_cpu_threads.so")
_lib = None


def build_cpu_threads_library(force: bool = False) -> str:
    """Compile ``dst_cpu_threads.c`` with gcc (no fast-math: the sum keeps input order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Slice(ctypes.Structure):
    _fields_ = [("indices", ctypes.c_void_p), ("values", ctypes.c_void_p), ("n_rows", ctypes.c_int64)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_cpu_threads_library())
        lib.dst_cpu_threads_densify.restype = ctypes.c_int
        lib.dst_cpu_threads_densify.argtypes = [
            ctypes.POINTER(_Slice), ctypes.c_int32, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        _lib = lib
    return _lib


def host_cores() -> int:
    """Cores this process may run on."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def densify_threads(indices: Sequence[np.ndarray], values: Sequence[np.ndarray], d: int, vocab: int,
                    dense_in: Optional[np.ndarray] = None, *, value_dtype: str = "f32", out_dtype: str = "f32",
                    n_threads: Optional[int] = None) -> Tuple[np.ndarray, int, int]:
    """Returns (out [vocab, d] in the output dtype (float32 / uint16 bf16 bits), rows out of range, threads used)."""
    lib = _load()
    R = len(indices)
    assert len(values) == R
    idx_dtype = np.dtype(indices[0].dtype) if R else np.dtype(np.int64)
    assert idx_dtype in (np.dtype(np.int32), np.dtype(np.int64))
    vdt = np.float32 if value_dtype == "f32" else np.uint16
    odt = np.float32 if out_dtype == "f32" else np.uint16
    keep = []
    arr = (_Slice * max(R, 1))()
    for r in range(R):
        ix = np.ascontiguousarray(indices[r], dtype=idx_dtype)
        va = np.ascontiguousarray(values[r], dtype=vdt)
        assert va.size == ix.shape[0] * d, "values[%d] must be [n_rows, d]" % r
        keep += [ix, va]
        arr[r].indices = ix.ctypes.data
        arr[r].values = va.ctypes.data
        arr[r].n_rows = ix.shape[0]
    dn = None
    if dense_in is not None:
        dn = np.ascontiguousarray(dense_in, dtype=odt)
        assert dn.size == vocab * d
    out = np.empty((vocab, d), odt)
    scratch = np.empty((vocab, d), np.float32) if out_dtype == "bf16" else None
    n_bad = ctypes.c_int64(0)
    used = lib.dst_cpu_threads_densify(arr, R, int(idx_dtype == np.dtype(np.int64)), int(value_dtype == "bf16"),
                                       int(out_dtype == "bf16"), d, vocab,
                                       dn.ctypes.data if dn is not None else None, out.ctypes.data,
                                       scratch.ctypes.data if scratch is not None else None,
                                       int(n_threads or host_cores()), ctypes.byref(n_bad))
    if used < 0:
        raise ValueError("dst_cpu_threads_densify rejected its arguments")
    return out, int(n_bad.value), int(used)
