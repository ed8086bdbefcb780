"""ctypes marshalling for ``libdst_b200.so`` (see ``include/dst.h`` for the contract)."""
from __future__ import annotations

import contextlib
import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdst_b200.so")
_lib = None

DST_STATUS = {
    0: "DST_OK", 1: "DST_ERR_INVALID_ARG", 2: "DST_ERR_UNSUPPORTED", 3: "DST_ERR_WORKSPACE_TOO_SMALL",
    4: "DST_ERR_INDEX_OUT_OF_RANGE", 5: "DST_ERR_TIMEOUT", 6: "DST_ERR_CUDA",
}
DST_I32, DST_I64 = 0, 1
DST_F32, DST_BF16 = 0, 1


class DstError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%s)" % (where, DST_STATUS.get(status, status), dst_status_string(status)))


class _Opts(ctypes.Structure):
    _fields_ = [("index_type", ctypes.c_int32), ("value_type", ctypes.c_int32), ("out_type", ctypes.c_int32),
                ("flags", ctypes.c_uint32)]


class _Slice(ctypes.Structure):
    _fields_ = [("indices", ctypes.c_void_p), ("values", ctypes.c_void_p), ("n_rows", ctypes.c_int64)]


class _Result(ctypes.Structure):
    _fields_ = [("status", ctypes.c_int32), ("n_unique", ctypes.c_int32), ("n_out_of_range", ctypes.c_int64),
                ("max_segment", ctypes.c_int64)]


class _BytesReport(ctypes.Structure):
    _fields_ = [("n_rows_total", ctypes.c_int64), ("sparse_value_bytes", ctypes.c_int64),
                ("sparse_index_bytes", ctypes.c_int64), ("sparse_bytes", ctypes.c_int64),
                ("dense_bytes", ctypes.c_int64), ("gather_all_value_bytes", ctypes.c_int64),
                ("sparse_over_dense", ctypes.c_double), ("gather_all_over_dense", ctypes.c_double)]


class _Optimizer(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("step", ctypes.c_int32), ("lr", ctypes.c_float), ("momentum", ctypes.c_float),
                ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("grad_scale", ctypes.c_float), ("state1", ctypes.c_void_p), ("state2", ctypes.c_void_p)]


class _RankGrads(ctypes.Structure):
    _fields_ = [("dense", ctypes.c_void_p), ("slices", ctypes.POINTER(_Slice)), ("n_slices", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


class _Grad(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("reserved", ctypes.c_int32), ("indices", ctypes.c_void_p),
                ("values", ctypes.c_void_p), ("n_rows", ctypes.c_int64)]


class _AccumPlan(ctypes.Structure):
    _fields_ = [("branch", ctypes.c_int32), ("out_kind", ctypes.c_int32), ("out_rows", ctypes.c_int64),
                ("out_bytes", ctypes.c_int64), ("n_dense", ctypes.c_int32), ("n_slices", ctypes.c_int32),
                ("n_slice_rows", ctypes.c_int64), ("converts", ctypes.c_int32), ("reserved", ctypes.c_int32)]


RESULT_BYTES = ctypes.sizeof(_Result)
DST_GRAD_DENSE, DST_GRAD_SLICES = 0, 1
DST_ACC_STOCK, DST_ACC_PROPOSED, DST_ACC_SPARSE_AS_DENSE = 0, 1, 2
DST_OPT_SGD, DST_OPT_MOMENTUM, DST_OPT_ADAM = 0, 1, 2
DST_BRANCH = {0: "empty", 1: "pass-through", 2: "reduce", 3: "convert+reduce", 4: "gather"}

# name -> (restype, argtypes); also the list of symbols the header declares
_vp, _i64, _i32, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
SYMBOLS = {
    "dst_version": (ctypes.c_int, []),
    "dst_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "dst_workspace_bytes": (_sz, [_i64, _i32, _i64, _i64, ctypes.POINTER(_Opts)]),
    "dst_densify": (ctypes.c_int, [_vp, _vp, _i64, _i64, _i64, _vp, _vp, _vp, ctypes.POINTER(_Opts), _vp, _sz,
                                   _vp, _vp, _vp]),
    "dst_densify_concat": (ctypes.c_int, [ctypes.POINTER(_Slice), _i32, _i64, _i64, _vp, _vp, _vp,
                                          ctypes.POINTER(_Opts), _vp, _sz, _vp, _vp, _vp]),
    "dst_densify_apply_sgd": (ctypes.c_int, [ctypes.POINTER(_Slice), _i32, _i64, _i64, _vp, _vp, ctypes.c_float, _vp,
                                             ctypes.POINTER(_Opts), _vp, _sz, _vp, _vp, _vp]),
    "dst_densify_apply": (ctypes.c_int, [ctypes.POINTER(_Slice), _i32, _i64, _i64, _vp, _vp, ctypes.POINTER(_Optimizer), _vp,
                                         ctypes.POINTER(_Opts), _vp, _sz, _vp, _vp, _vp]),
    "dst_densify_batch": (ctypes.c_int, [ctypes.POINTER(_RankGrads), _i32, _i64, _i64, _vp, _vp, ctypes.POINTER(_Opts),
                                         _vp, _sz, _vp, _vp, _vp]),
    "dst_densify_static": (ctypes.c_int, [_vp, _vp, _i64, _i64, _i64, _vp, _vp, _vp, ctypes.POINTER(_Opts),
                                          _vp, _vp, _vp]),
    "dst_host_staging_bytes": (_sz, [_i64, _i64, _i64, ctypes.POINTER(_Opts)]),
    "dst_densify_concat_host": (ctypes.c_int, [ctypes.POINTER(_Slice), _i32, _i64, _i64, _vp, _vp, _vp,
                                               ctypes.POINTER(_Opts), _vp, _sz, _vp, _sz, _vp]),
    "dst_selftest_wait_limit": (ctypes.c_int, [_i64, _vp, _sz, _vp, _vp]),
    "dst_profile_events": (None, [_vp, _vp]),
    "dst_kernel_launches": (ctypes.c_int64, []),
    "dst_profile_ranges": (None, [ctypes.c_int]),
    "dst_bytes_report": (ctypes.c_int, [ctypes.POINTER(_i64), _i32, _i64, _i64, ctypes.POINTER(_Opts),
                                        ctypes.POINTER(_BytesReport)]),
    "dst_accumulate_plan": (ctypes.c_int, [ctypes.POINTER(_Grad), _i32, _i64, _i64, _i32, ctypes.POINTER(_Opts),
                                           ctypes.POINTER(_AccumPlan)]),
    "dst_accumulate": (ctypes.c_int, [ctypes.POINTER(_Grad), _i32, _i64, _i64, _i32, _vp, _vp, _vp, _i64, _vp,
                                      ctypes.POINTER(_Opts), _vp, _sz, _vp, ctypes.POINTER(_AccumPlan)]),
}


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                "%s is missing: build it with `python -m paper_1905_04035_b200.build` "
                "(nvcc, sm_100a). There is no CPU fallback." % _LIB_PATH)
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _index_type(t: torch.dtype) -> int:
    if t == torch.int64:
        return DST_I64
    if t == torch.int32:
        return DST_I32
    raise TypeError("indices must be int32 or int64, got %s" % t)


def _dtype(t: torch.dtype) -> int:
    if t == torch.float32:
        return DST_F32
    if t == torch.bfloat16:
        return DST_BF16
    raise TypeError("values / dense tensors must be float32 or bfloat16, got %s" % t)


def _opts(index_dtype, value_dtype, out_dtype) -> _Opts:
    return _Opts(_index_type(index_dtype), _dtype(value_dtype), _dtype(out_dtype), 0)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_handle(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def dst_version() -> int:
    return int(load_library().dst_version())


def dst_status_string(status: int) -> str:
    return load_library().dst_status_string(int(status)).decode()


def dst_profile_events(before=None, after=None) -> None:
    """Record two ``torch.cuda.Event`` objects around the row-reduction kernel of later calls
    made from this thread; ``None, None`` switches it off.  The events must have been recorded
    once already (torch creates the CUDA event lazily)."""
    def handle(ev):
        return None if ev is None else ctypes.c_void_p(ev.cuda_event)
    load_library().dst_profile_events(handle(before), handle(after))


def dst_kernel_launches() -> int:
    return int(load_library().dst_kernel_launches())


def dst_profile_ranges(on: bool) -> None:
    """NVTX ranges around the phases of later calls (off by default)."""
    load_library().dst_profile_ranges(1 if on else 0)


def dst_selftest_wait_limit(limit_cycles: int, workspace: torch.Tensor, result: Optional[torch.Tensor] = None,
                            stream=None) -> None:
    """Run the give-up path of the library's bounded device-side waits on its own (see ``include/dst.h``)."""
    rc = load_library().dst_selftest_wait_limit(int(limit_cycles), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                _stream_handle(stream), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_selftest_wait_limit")


def dst_workspace_bytes(n_rows_total: int, R: int, d: int, vocab: int, index_dtype=torch.int64,
                        value_dtype=torch.float32, out_dtype=torch.float32) -> int:
    o = _opts(index_dtype, value_dtype, out_dtype)
    return int(load_library().dst_workspace_bytes(n_rows_total, R, d, vocab, ctypes.byref(o)))


def dst_host_staging_bytes(n_rows_total: int, d: int, vocab: int, index_dtype=torch.int64,
                           value_dtype=torch.float32, out_dtype=torch.float32) -> int:
    o = _opts(index_dtype, value_dtype, out_dtype)
    return int(load_library().dst_host_staging_bytes(n_rows_total, d, vocab, ctypes.byref(o)))


def dst_bytes_report(n_rows_per_slice: Sequence[int], d: int, vocab: int, index_dtype=torch.int64,
                     value_dtype=torch.float32, out_dtype=torch.float32) -> dict:
    o = _opts(index_dtype, value_dtype, out_dtype)
    R = len(n_rows_per_slice)
    arr = (ctypes.c_int64 * max(R, 1))(*[int(n) for n in n_rows_per_slice])
    rep = _BytesReport()
    rc = load_library().dst_bytes_report(arr, R, d, vocab, ctypes.byref(o), ctypes.byref(rep))
    if rc != 0:
        raise DstError(rc, "dst_bytes_report")
    out = {name: getattr(rep, name) for name, _ in _BytesReport._fields_}
    out["R"] = R
    return out


def _check_slice(idx: torch.Tensor, val: torch.Tensor, d: int, device) -> None:
    if idx.dim() != 1 or not idx.is_contiguous() or not val.is_contiguous():
        raise ValueError("indices must be 1-D contiguous and values contiguous")
    if val.numel() != idx.shape[0] * d:
        raise ValueError("values must be [n_rows, d]")
    if idx.device != device or val.device != device:
        raise ValueError("all tensors must live on the same device")


def dst_densify_concat(slices: Sequence[Tuple[torch.Tensor, torch.Tensor]], d: int, vocab: int,
                       dense_in: Optional[torch.Tensor], out: torch.Tensor, workspace: torch.Tensor,
                       unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                       result: Optional[torch.Tensor] = None, stream=None,
                       index_dtype: Optional[torch.dtype] = None, value_dtype: Optional[torch.dtype] = None) -> None:
    """Enqueue ``dst_densify_concat`` (include/dst.h).  All tensors are CUDA tensors owned by the caller.

    ``result``: an int32/uint8 CUDA (or pinned) tensor of at least 24 bytes that receives ``dst_result_t``.
    """
    lib = load_library()
    R = len(slices)
    if R:
        index_dtype, value_dtype = slices[0][0].dtype, slices[0][1].dtype
    elif index_dtype is None or value_dtype is None:
        index_dtype, value_dtype = index_dtype or torch.int64, value_dtype or out.dtype
    arr = (_Slice * max(R, 1))()
    for r, (idx, val) in enumerate(slices):
        if idx.dtype != index_dtype or val.dtype != value_dtype:
            raise TypeError("all slices must share index and value dtypes")
        _check_slice(idx, val, d, out.device)
        arr[r].indices, arr[r].values, arr[r].n_rows = idx.data_ptr(), val.data_ptr(), idx.shape[0]
    if out.numel() != vocab * d or not out.is_contiguous():
        raise ValueError("out must be contiguous [vocab, d]")
    if dense_in is not None and (dense_in.dtype != out.dtype or dense_in.numel() != vocab * d
                                 or not dense_in.is_contiguous()):
        raise ValueError("dense_in must be contiguous [vocab, d] in out's dtype")
    o = _opts(index_dtype, value_dtype, out.dtype)
    with torch.cuda.device(out.device):
        rc = lib.dst_densify_concat(arr, R, d, vocab, _ptr(dense_in), _ptr(out), _stream_handle(stream),
                                    ctypes.byref(o), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _ptr(unique_rows), _ptr(counts), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify_concat")


def dst_densify_apply_sgd(slices: Sequence[Tuple[torch.Tensor, torch.Tensor]], d: int, vocab: int,
                          dense_in: Optional[torch.Tensor], weight: torch.Tensor, lr: float, workspace: torch.Tensor,
                          unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                          result: Optional[torch.Tensor] = None, stream=None,
                          index_dtype: Optional[torch.dtype] = None) -> None:
    """Enqueue ``dst_densify_apply_sgd`` (include/dst.h): weight -= lr * (dense_in + densified slices), fp32."""
    lib = load_library()
    R = len(slices)
    index_dtype = slices[0][0].dtype if R else (index_dtype or torch.int64)
    arr = (_Slice * max(R, 1))()
    for r, (idx, val) in enumerate(slices):
        if idx.dtype != index_dtype or val.dtype != torch.float32:
            raise TypeError("all slices must share the index dtype and hold float32 values")
        _check_slice(idx, val, d, weight.device)
        arr[r].indices, arr[r].values, arr[r].n_rows = idx.data_ptr(), val.data_ptr(), idx.shape[0]
    if weight.dtype != torch.float32 or weight.numel() != vocab * d or not weight.is_contiguous():
        raise ValueError("weight must be contiguous float32 [vocab, d]")
    if dense_in is not None and (dense_in.dtype != torch.float32 or dense_in.numel() != vocab * d
                                 or not dense_in.is_contiguous()):
        raise ValueError("dense_in must be contiguous float32 [vocab, d]")
    o = _opts(index_dtype, torch.float32, torch.float32)
    with torch.cuda.device(weight.device):
        rc = lib.dst_densify_apply_sgd(arr, R, d, vocab, _ptr(dense_in), _ptr(weight), float(lr), _stream_handle(stream),
                                       ctypes.byref(o), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                       _ptr(unique_rows), _ptr(counts), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify_apply_sgd")


def dst_densify_batch(ranks, d: int, vocab: int, out: torch.Tensor, workspace: torch.Tensor,
                      unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                      result: Optional[torch.Tensor] = None, stream=None, index_dtype: Optional[torch.dtype] = None,
                      value_dtype: Optional[torch.dtype] = None) -> None:
    """Enqueue ``dst_densify_batch`` (include/dst.h).  ``ranks``: a list of (dense or None, [(indices, values), ...])."""
    lib = load_library()
    R = len(ranks)
    arr = (_RankGrads * max(R, 1))()
    keep = []
    for r, (dense, slices) in enumerate(ranks):
        if dense is not None and (dense.dtype != out.dtype or dense.numel() != vocab * d or not dense.is_contiguous()):
            raise ValueError("a rank's dense tensor must be contiguous [vocab, d] in out's dtype")
        sl = (_Slice * max(len(slices), 1))()
        for q, (idx, val) in enumerate(slices):
            index_dtype = index_dtype or idx.dtype
            value_dtype = value_dtype or val.dtype
            if idx.dtype != index_dtype or val.dtype != value_dtype:
                raise TypeError("all slices must share index and value dtypes")
            _check_slice(idx, val, d, out.device)
            sl[q].indices, sl[q].values, sl[q].n_rows = idx.data_ptr(), val.data_ptr(), idx.shape[0]
        keep.append(sl)
        arr[r].dense = dense.data_ptr() if dense is not None else None
        arr[r].slices = ctypes.cast(sl, ctypes.POINTER(_Slice))
        arr[r].n_slices = len(slices)
    o = _opts(index_dtype or torch.int64, value_dtype or torch.float32, out.dtype)
    with torch.cuda.device(out.device):
        rc = lib.dst_densify_batch(arr, R, d, vocab, _ptr(out), _stream_handle(stream), ctypes.byref(o), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _ptr(unique_rows), _ptr(counts), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify_batch")


def dst_densify_apply(slices: Sequence[Tuple[torch.Tensor, torch.Tensor]], d: int, vocab: int,
                      dense_in: Optional[torch.Tensor], weight: torch.Tensor, workspace: torch.Tensor, *,
                      kind: int = DST_OPT_SGD, lr: float, momentum: float = 0.0, beta1: float = 0.9,
                      beta2: float = 0.999, eps: float = 1e-8, step: int = 1, grad_scale: float = 1.0,
                      state1: Optional[torch.Tensor] = None, state2: Optional[torch.Tensor] = None,
                      unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                      result: Optional[torch.Tensor] = None, stream=None,
                      index_dtype: Optional[torch.dtype] = None, grad_dtype: Optional[torch.dtype] = None) -> None:
    """Enqueue ``dst_densify_apply`` (include/dst.h): the optimizer step (SGD, momentum, Adam) on the fp32
    ``weight`` with the gradient grad_scale * (dense_in + densified slices), fp32 or bf16 gradients."""
    lib = load_library()
    R = len(slices)
    index_dtype = slices[0][0].dtype if R else (index_dtype or torch.int64)
    grad_dtype = slices[0][1].dtype if R else (grad_dtype or (dense_in.dtype if dense_in is not None else torch.float32))
    arr = (_Slice * max(R, 1))()
    for r, (idx, val) in enumerate(slices):
        if idx.dtype != index_dtype or val.dtype != grad_dtype:
            raise TypeError("all slices must share the index dtype and the gradient dtype")
        _check_slice(idx, val, d, weight.device)
        arr[r].indices, arr[r].values, arr[r].n_rows = idx.data_ptr(), val.data_ptr(), idx.shape[0]
    for name, t in (("weight", weight), ("state1", state1), ("state2", state2)):
        if t is not None and (t.dtype != torch.float32 or t.numel() != vocab * d or not t.is_contiguous()):
            raise ValueError("%s must be contiguous float32 [vocab, d]" % name)
    if dense_in is not None and (dense_in.dtype != grad_dtype or dense_in.numel() != vocab * d
                                 or not dense_in.is_contiguous()):
        raise ValueError("dense_in must be contiguous [vocab, d] in the gradient dtype")
    o = _opts(index_dtype, grad_dtype, grad_dtype)
    opt = _Optimizer(int(kind), int(step), float(lr), float(momentum), float(beta1), float(beta2), float(eps),
                     float(grad_scale), state1.data_ptr() if state1 is not None else None,
                     state2.data_ptr() if state2 is not None else None)
    with torch.cuda.device(weight.device):
        rc = lib.dst_densify_apply(arr, R, d, vocab, _ptr(dense_in), _ptr(weight), ctypes.byref(opt), _stream_handle(stream),
                                   ctypes.byref(o), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _ptr(unique_rows), _ptr(counts), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify_apply")


def dst_densify(indices: torch.Tensor, values: torch.Tensor, d: int, vocab: int,
                dense_in: Optional[torch.Tensor], out: torch.Tensor, workspace: torch.Tensor,
                unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                result: Optional[torch.Tensor] = None, stream=None) -> None:
    """Enqueue ``dst_densify`` (include/dst.h) for one IndexedSlices gradient."""
    lib = load_library()
    _check_slice(indices, values, d, out.device)
    if out.numel() != vocab * d or not out.is_contiguous():
        raise ValueError("out must be contiguous [vocab, d]")
    if dense_in is not None and (dense_in.dtype != out.dtype or dense_in.numel() != vocab * d
                                 or not dense_in.is_contiguous()):
        raise ValueError("dense_in must be contiguous [vocab, d] in out's dtype")
    o = _opts(indices.dtype, values.dtype, out.dtype)
    with torch.cuda.device(out.device):
        rc = lib.dst_densify(_ptr(indices), _ptr(values), indices.shape[0], d, vocab, _ptr(dense_in), _ptr(out),
                             _stream_handle(stream), ctypes.byref(o), _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _ptr(unique_rows), _ptr(counts),
                             _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify")


STATIC_WORKSPACE_BYTES = 4 << 20   # DST_STATIC_WORKSPACE_BYTES of include/dst.h


def dst_densify_static(indices: torch.Tensor, values: torch.Tensor, d: int, vocab: int,
                       dense_in: Optional[torch.Tensor], out: torch.Tensor,
                       unique_rows: Optional[torch.Tensor] = None, counts: Optional[torch.Tensor] = None,
                       result: Optional[torch.Tensor] = None, stream=None) -> None:
    """Enqueue ``dst_densify_static`` (include/dst.h): ``dst_densify`` for callers that cannot hand
    over a workspace because they must not allocate device memory where they call from.  The scratch
    is an array inside the library (``STATIC_WORKSPACE_BYTES`` per GPU), so shapes that need more raise
    ``DstError`` (workspace too small), and calls that may overlap on the GPU must be ordered by the
    caller.  Make the first call on a device outside stream capture."""
    lib = load_library()
    _check_slice(indices, values, d, out.device)
    if out.numel() != vocab * d or not out.is_contiguous():
        raise ValueError("out must be contiguous [vocab, d]")
    if dense_in is not None and (dense_in.dtype != out.dtype or dense_in.numel() != vocab * d
                                 or not dense_in.is_contiguous()):
        raise ValueError("dense_in must be contiguous [vocab, d] in out's dtype")
    o = _opts(indices.dtype, values.dtype, out.dtype)
    with torch.cuda.device(out.device):
        rc = lib.dst_densify_static(_ptr(indices), _ptr(values), indices.shape[0], d, vocab, _ptr(dense_in),
                                    _ptr(out), _stream_handle(stream), ctypes.byref(o), _ptr(unique_rows),
                                    _ptr(counts), _ptr(result))
    if rc != 0:
        raise DstError(rc, "dst_densify_static")


def dst_densify_concat_host(slices: Sequence[Tuple[torch.Tensor, torch.Tensor]], d: int, vocab: int,
                            host_dense_in: Optional[torch.Tensor], host_out: torch.Tensor, staging: torch.Tensor,
                            workspace: torch.Tensor, host_result: Optional[torch.Tensor] = None, stream=None) -> None:
    """Enqueue ``dst_densify_concat_host``: slices, dense_in and out are HOST (ideally pinned) tensors;
    ``staging`` and ``workspace`` are CUDA tensors.  host_out is valid after the stream has drained."""
    lib = load_library()
    R = len(slices)
    if R == 0:
        raise ValueError("need at least one slice")
    index_dtype, value_dtype = slices[0][0].dtype, slices[0][1].dtype
    arr = (_Slice * R)()
    for r, (idx, val) in enumerate(slices):
        if idx.is_cuda or val.is_cuda:
            raise ValueError("host entry point: slices must be CPU tensors")
        if idx.dtype != index_dtype or val.dtype != value_dtype:
            raise TypeError("all slices must share index and value dtypes")
        _check_slice(idx, val, d, torch.device("cpu"))
        arr[r].indices, arr[r].values, arr[r].n_rows = idx.data_ptr(), val.data_ptr(), idx.shape[0]
    o = _opts(index_dtype, value_dtype, host_out.dtype)
    with torch.cuda.device(staging.device):
        rc = lib.dst_densify_concat_host(arr, R, d, vocab, _ptr(host_dense_in), _ptr(host_out),
                                         _stream_handle(stream), ctypes.byref(o), _ptr(staging),
                                         staging.numel() * staging.element_size(), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _ptr(host_result))
    if rc != 0:
        raise DstError(rc, "dst_densify_concat_host")


def _marshal_grads(grads, d: int, vocab: int, index_dtype, value_dtype, out_dtype):
    """``grads``: a dense gradient is a [vocab, d] tensor, IndexedSlices are an (indices, values) pair."""
    arr = (_Grad * max(len(grads), 1))()
    for k, g in enumerate(grads):
        if isinstance(g, torch.Tensor):
            if g.numel() != vocab * d or not g.is_contiguous():
                raise ValueError("a dense gradient must be contiguous [vocab, d]")
            out_dtype = out_dtype or g.dtype
            if g.dtype != out_dtype:
                raise TypeError("all dense gradients must share one dtype")
            arr[k].kind, arr[k].indices, arr[k].values, arr[k].n_rows = DST_GRAD_DENSE, None, g.data_ptr(), 0
        else:
            idx, val = g
            index_dtype, value_dtype = index_dtype or idx.dtype, value_dtype or val.dtype
            if idx.dtype != index_dtype or val.dtype != value_dtype:
                raise TypeError("all IndexedSlices must share index and value dtypes")
            _check_slice(idx, val, d, val.device)
            arr[k].kind, arr[k].indices, arr[k].values, arr[k].n_rows = (DST_GRAD_SLICES, idx.data_ptr(),
                                                                         val.data_ptr(), idx.shape[0])
    return arr, index_dtype or torch.int64, value_dtype or out_dtype or torch.float32, out_dtype or value_dtype or torch.float32


def _plan_dict(p: _AccumPlan) -> dict:
    return {"branch": DST_BRANCH[p.branch], "out_kind": {0: "dense", 1: "slices", -1: None}[p.out_kind],
            "out_rows": p.out_rows, "out_bytes": p.out_bytes, "n_dense": p.n_dense, "n_slices": p.n_slices,
            "n_slice_rows": p.n_slice_rows, "converts": bool(p.converts)}


def dst_accumulate_plan(grads, d: int, vocab: int, strategy: int = DST_ACC_PROPOSED, index_dtype=None,
                        value_dtype=None, out_dtype=None) -> dict:
    """``dst_accumulate_plan`` (include/dst.h): which branch of Algorithm 1 / Algorithm 2 / Listing 1 the list takes."""
    lib = load_library()
    arr, it, vt, ot = _marshal_grads(grads, d, vocab, index_dtype, value_dtype, out_dtype)
    o = _opts(it, vt, ot)
    p = _AccumPlan()
    rc = lib.dst_accumulate_plan(arr, len(grads), d, vocab, strategy, ctypes.byref(o), ctypes.byref(p))
    if rc != 0:
        raise DstError(rc, "dst_accumulate_plan")
    return _plan_dict(p)


def dst_accumulate(grads, d: int, vocab: int, strategy: int = DST_ACC_PROPOSED, *,
                   out_dense: Optional[torch.Tensor] = None, out_indices: Optional[torch.Tensor] = None,
                   out_values: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   result: Optional[torch.Tensor] = None, stream=None, index_dtype=None, value_dtype=None,
                   out_dtype=None) -> dict:
    """Enqueue ``dst_accumulate`` (include/dst.h).  Output buffers are the caller's; returns the plan."""
    lib = load_library()
    if out_dense is not None:
        out_dtype = out_dtype or out_dense.dtype
    arr, it, vt, ot = _marshal_grads(grads, d, vocab, index_dtype, value_dtype, out_dtype)
    if out_dense is not None and (out_dense.dtype != ot or out_dense.numel() != vocab * d or not out_dense.is_contiguous()):
        raise ValueError("out_dense must be contiguous [vocab, d] in the dense gradients' dtype")
    cap = 0
    if out_indices is not None and out_values is not None:
        if out_indices.dtype != it or out_values.dtype != vt or not out_indices.is_contiguous() or not out_values.is_contiguous():
            raise ValueError("out_indices / out_values must be contiguous and of the slices' dtypes")
        cap = min(out_indices.shape[0], out_values.numel() // d if d else out_indices.shape[0])
    o = _opts(it, vt, ot)
    p = _AccumPlan()
    dev = next((t.device for t in (out_dense, out_values, workspace) if t is not None), None)
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with torch.cuda.device(dev) if dev is not None else contextlib.nullcontext():
        rc = lib.dst_accumulate(arr, len(grads), d, vocab, strategy, _ptr(out_dense), _ptr(out_indices),
                                _ptr(out_values), cap, _stream_handle(stream), ctypes.byref(o), _ptr(workspace),
                                ws_bytes, _ptr(result), ctypes.byref(p))
    if rc != 0:
        raise DstError(rc, "dst_accumulate")
    return _plan_dict(p)


class Densifier:
    """Owns the caller-side buffers (workspace, result block, optional unique/count arrays) for
    repeated calls on one shape; the arithmetic stays in the library."""

    def __init__(self, n_rows_total: int, R: int, d: int, vocab: int, *, index_dtype=torch.int64,
                 value_dtype=torch.float32, out_dtype=torch.float32, device="cuda", want_unique: bool = True):
        self.n_rows_total, self.R, self.d, self.vocab = n_rows_total, R, d, vocab
        self.index_dtype, self.value_dtype, self.out_dtype = index_dtype, value_dtype, out_dtype
        self.device = torch.device(device)
        nbytes = dst_workspace_bytes(n_rows_total, R, d, vocab, index_dtype, value_dtype, out_dtype)
        if nbytes == 0 and vocab and d:
            raise DstError(2, "dst_workspace_bytes")
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        self.result = torch.zeros(RESULT_BYTES // 4, dtype=torch.int32, device=self.device)
        cap = max(1, min(n_rows_total, vocab))
        self.unique_rows = torch.empty(cap, dtype=index_dtype, device=self.device) if want_unique else None
        self.counts = torch.empty(cap, dtype=torch.int32, device=self.device) if want_unique else None

    def __call__(self, slices, dense_in, out, stream=None):
        dst_densify_concat(slices, self.d, self.vocab, dense_in, out, self.workspace, self.unique_rows,
                           self.counts, self.result, stream, self.index_dtype, self.value_dtype)
        return out

    def densify(self, indices, values, dense_in, out, stream=None):
        dst_densify(indices, values, self.d, self.vocab, dense_in, out, self.workspace, self.unique_rows,
                    self.counts, self.result, stream)
        return out

    def read_result(self) -> dict:
        """Synchronising read of the dst_result_t the last call wrote."""
        raw = self.result.cpu().numpy().tobytes()
        r = _Result.from_buffer_copy(raw)
        return {"status": r.status, "n_unique": r.n_unique, "n_out_of_range": r.n_out_of_range,
                "max_segment": r.max_segment}
