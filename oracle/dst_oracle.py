"""Python face of the CPU oracle.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
this module; the CUDA library and its binding never do, and this module never
imports them.

``densify`` calls the plain C loop in ``dst_oracle.c`` (the definition of the
operation of the paper's Section 4 / Listing 1 followed by the reduction of
Algorithm 1) and derives ``unique_rows`` / ``counts`` by a linear scan of the
per-row counters.  ``bytes_report`` is the footprint comparison of Section 4
(Fig. 5a): what a gather of IndexedSlices holds against the fixed dense tensor.

Pins: see ``tests/test_oracle_pins.py`` and ``tests/test_bytes_report.py``.
Not pinned: nothing -- every function here has at least one independent check.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dst_oracle.c")
_LIB = os.path.join(_HERE, "libdst_oracle.so")
_lib = None


def build_oracle_library(force: bool = False) -> str:
    """Compile ``dst_oracle.c`` with gcc (no fast-math: fp64 semantics matter)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Slice(ctypes.Structure):
    _fields_ = [("indices", ctypes.c_void_p), ("values", ctypes.c_void_p), ("n_rows", ctypes.c_int64)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_oracle_library())
        lib.dst_oracle_densify.restype = ctypes.c_int
        lib.dst_oracle_densify.argtypes = [
            ctypes.POINTER(_Slice), ctypes.c_int32, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64)]
        lib.dst_oracle_round_bf16.restype = ctypes.c_uint16
        lib.dst_oracle_round_bf16.argtypes = [ctypes.c_double]
        lib.dst_oracle_widen_bf16.restype = ctypes.c_double
        lib.dst_oracle_widen_bf16.argtypes = [ctypes.c_uint16]
        _lib = lib
    return _lib


@dataclasses.dataclass
class OracleResult:
    acc: np.ndarray          # [vocab, d] float64, unrounded sums
    mag: np.ndarray          # [vocab, d] float64, sum of |terms| (tolerance scale)
    out: np.ndarray          # [vocab, d] rounded once to the output dtype (float32 / uint16 bf16 bits)
    cnt: np.ndarray          # [vocab] int64 occurrences of each row
    unique_rows: np.ndarray  # ascending rows with cnt > 0, in the index dtype
    counts: np.ndarray       # int32 occurrences of those rows
    n_unique: int
    n_out_of_range: int
    max_segment: int


def densify(indices: Sequence[np.ndarray], values: Sequence[np.ndarray], d: int, vocab: int,
            dense_in: Optional[np.ndarray] = None, *, value_dtype: str = "f32",
            out_dtype: str = "f32") -> OracleResult:
    """Scatter-sum R slices into a dense [vocab, d] tensor plus ``dense_in``.

    ``indices[r]`` is int32 or int64 (all slices alike); ``values[r]`` is
    float32, or uint16 bf16 bit patterns when ``value_dtype == "bf16"``;
    ``dense_in`` has the output dtype.
    """
    lib = _load()
    R = len(indices)
    assert len(values) == R
    idx_dtype = np.dtype(indices[0].dtype) if R else np.dtype(np.int64)
    assert idx_dtype in (np.dtype(np.int32), np.dtype(np.int64))
    vdt = np.float32 if value_dtype == "f32" else np.uint16
    odt = np.float32 if out_dtype == "f32" else np.uint16
    keep: List[np.ndarray] = []
    arr = (_Slice * max(R, 1))()
    for r in range(R):
        ix = np.ascontiguousarray(indices[r], dtype=idx_dtype)
        va = np.ascontiguousarray(values[r], dtype=vdt)
        n = ix.shape[0]
        assert va.size == n * d, "values[%d] must be [n_rows, d]" % r
        keep += [ix, va]
        arr[r].indices = ix.ctypes.data
        arr[r].values = va.ctypes.data
        arr[r].n_rows = n
    dn = None
    if dense_in is not None:
        dn = np.ascontiguousarray(dense_in, dtype=odt)
        assert dn.size == vocab * d
    acc = np.empty((vocab, d), np.float64)
    mag = np.empty((vocab, d), np.float64)
    out = np.empty((vocab, d), odt)
    cnt = np.empty((vocab,), np.int64)
    n_bad = ctypes.c_int64(0)
    rc = lib.dst_oracle_densify(arr, R, int(idx_dtype == np.dtype(np.int64)), int(value_dtype == "bf16"),
                                int(out_dtype == "bf16"), d, vocab,
                                dn.ctypes.data if dn is not None else None,
                                acc.ctypes.data, mag.ctypes.data, out.ctypes.data, cnt.ctypes.data,
                                ctypes.byref(n_bad))
    if rc != 0:
        raise ValueError("dst_oracle_densify rejected its arguments")
    unique_rows = np.nonzero(cnt)[0]
    counts = cnt[unique_rows].astype(np.int32)
    return OracleResult(acc, mag, out, cnt, unique_rows.astype(idx_dtype), counts, int(unique_rows.shape[0]),
                        int(n_bad.value), int(cnt.max()) if vocab else 0)


@dataclasses.dataclass
class SgdResult:
    weight: np.ndarray       # [vocab, d] float64: the updated weight, unrounded
    mag: np.ndarray          # [vocab, d] float64: |w| + lr * sum of |gradient terms| (tolerance scale)
    out: np.ndarray          # [vocab, d] float32: rounded once
    grad: OracleResult       # the dense gradient that was applied


def apply_sgd(indices: Sequence[np.ndarray], values: Sequence[np.ndarray], d: int, vocab: int,
              dense_in: Optional[np.ndarray], weight: np.ndarray, lr: float) -> SgdResult:
    """The step that follows accumulation in the paper's training loop (Section 4: the optimizer the
    distributed wrapper hands the accumulated gradients to), for plain SGD on the tied weight:

        weight[v, c] <- weight[v, c] - lr * (dense_in[v, c] + sum of the value rows naming v)

    Written as exactly that: the pinned scatter-sum of ``densify`` in fp64, then one fp64 multiply-subtract
    per element.  fp32 tensors only."""
    g = densify(indices, values, d, vocab, dense_in)
    w = np.asarray(weight, np.float32).reshape(vocab, d).astype(np.float64)
    new = w - float(lr) * g.acc
    return SgdResult(new, np.abs(w) + abs(float(lr)) * g.mag, new.astype(np.float32), g)


def round_bf16(x: float) -> int:
    return int(_load().dst_oracle_round_bf16(float(x)))


def widen_bf16(bits: int) -> float:
    return float(_load().dst_oracle_widen_bf16(int(bits)))


_SIZEOF = {"f32": 4, "bf16": 2, "i32": 4, "i64": 8}


def bytes_report(n_rows_per_slice: Sequence[int], d: int, vocab: int, *, index_dtype: str = "i64",
                 value_dtype: str = "f32", out_dtype: str = "f32") -> dict:
    """Footprint of accumulating by gather against accumulating by reduction.

    Section 4 compares the buffer a gather of IndexedSlices needs (11.4 GB at
    64 processes) with the fixed dense tensor a reduction needs (139 MB).

    ``sparse_*``: what the R concatenated slices hold -- every value row and
    every index.  ``dense_bytes``: one [vocab, d] tensor.  ``gather_all_*``:
    the accounting that reproduces the paper's printed figure: under
    Algorithm 1's gather branch the dense projection gradient is itself turned
    into ``vocab`` slices on every rank, so each rank ships ``vocab + n_r``
    value rows.
    """
    sv, si, so = _SIZEOF[value_dtype], _SIZEOF[index_dtype], _SIZEOF[out_dtype]
    R = len(n_rows_per_slice)
    n_total = 0
    for n in n_rows_per_slice:
        n_total += int(n)
    sparse_value_bytes = n_total * d * sv
    sparse_index_bytes = n_total * si
    dense_bytes = vocab * d * so
    gather_all_value_bytes = 0
    for n in n_rows_per_slice:
        gather_all_value_bytes += (vocab + int(n)) * d * sv
    def ratio(a, b):
        return (a / b) if b else 0.0
    return {
        "R": R,
        "n_rows_total": n_total,
        "sparse_value_bytes": sparse_value_bytes,
        "sparse_index_bytes": sparse_index_bytes,
        "sparse_bytes": sparse_value_bytes + sparse_index_bytes,
        "dense_bytes": dense_bytes,
        "gather_all_value_bytes": gather_all_value_bytes,
        "sparse_over_dense": ratio(sparse_value_bytes + sparse_index_bytes, dense_bytes),
        "gather_all_over_dense": ratio(gather_all_value_bytes, dense_bytes),
    }
