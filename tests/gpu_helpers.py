"""Shared helpers for the GPU parity tests: move a Workload to the device, run the
library through its binding, and compare with the CPU oracle."""
import numpy as np
import torch

import oracle
import paper_1905_04035_b200 as dst

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32, "i64": torch.int64}


def to_device(arr: np.ndarray, kind: str, device="cuda") -> torch.Tensor:
    """NumPy array (uint16 bit patterns for bf16) -> CUDA tensor of the real dtype."""
    if kind == "bf16":
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)


def to_numpy_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        bits = t.view(torch.int16).cpu().numpy().view(np.uint16)
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


def raw_bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy().view(np.uint32)


class GpuRun:
    def __init__(self, out, unique_rows, counts, result):
        self.out, self.unique_rows, self.counts, self.result = out, unique_rows, counts, result


def run_library(w, *, mode="concat", in_place=False, device="cuda") -> GpuRun:
    """mode: 'concat' -> dst_densify_concat on the R slices; 'single' -> dst_densify on the physical concatenation."""
    idt, vdt, odt = TORCH_DT[w.index_dtype], TORCH_DT[w.value_dtype], TORCH_DT[w.out_dtype]
    dense = to_device(w.dense_in, w.out_dtype, device) if w.dense_in is not None else None
    if in_place and dense is not None:
        out = dense
    else:
        out = torch.full((w.vocab, w.d), float("nan"), dtype=odt, device=device)
    if mode == "concat":
        slices = [(to_device(i, w.index_dtype, device), to_device(v, w.value_dtype, device))
                  for i, v in zip(w.indices, w.values)]
        R = len(slices)
    else:
        ci, cv = w.concatenated()
        slices = [(to_device(ci, w.index_dtype, device), to_device(cv, w.value_dtype, device))]
        R = 1
    eng = dst.Densifier(w.n_rows_total, R, w.d, w.vocab, index_dtype=idt, value_dtype=vdt, out_dtype=odt,
                        device=device)
    if mode == "concat":
        eng(slices, dense, out)
    else:
        eng.densify(slices[0][0], slices[0][1], dense, out)
    torch.cuda.synchronize()
    res = eng.read_result()
    nu = res["n_unique"]
    return GpuRun(out, eng.unique_rows[:nu].cpu().numpy(), eng.counts[:nu].cpu().numpy(), res)


def oracle_of(w):
    return oracle.densify(w.indices, w.values, w.d, w.vocab, w.dense_in, value_dtype=w.value_dtype,
                          out_dtype=w.out_dtype)


def tolerance(w, orc) -> np.ndarray:
    """Per-element bound on |gpu - exact sum|.

    fp32 values: 1e-5 * sum|terms| + 1e-7.  bf16 values with fp32 accumulation: 4e-3 * sum|terms|
    (covers the final rounding to bf16: half an ulp is 2^-8 = 3.9e-3 of the value).  fp32 values
    rounded to a bf16 output get the fp32 bound plus that rounding."""
    if w.value_dtype == "bf16":
        return 4e-3 * orc.mag
    tol = 1e-5 * orc.mag + 1e-7
    if w.out_dtype == "bf16":
        tol = tol + 2.0 ** -8 * np.abs(orc.acc)
    return tol


def assert_parity(w, run: GpuRun, orc=None):
    orc = orc or oracle_of(w)
    got = to_numpy_f64(run.out)
    assert not np.isnan(got).any(), "output rows were left unwritten"
    err = np.abs(got - orc.acc)
    tol = tolerance(w, orc)
    bad = err > tol
    assert not bad.any(), "%d elements out of tolerance, worst err/tol %.3g at %s" % (
        int(bad.sum()), float((err / np.maximum(tol, 1e-300)).max()), np.argwhere(bad)[:4].tolist())
    # integer outputs: bit-exact
    assert run.result["n_unique"] == orc.n_unique
    assert run.result["n_out_of_range"] == orc.n_out_of_range
    assert run.result["max_segment"] == orc.max_segment
    assert run.result["status"] == (4 if orc.n_out_of_range else 0)
    assert run.unique_rows.dtype == orc.unique_rows.dtype
    assert np.array_equal(run.unique_rows, orc.unique_rows)
    assert np.array_equal(run.counts, orc.counts)
    # rows nobody names are the dense partner (or zero) bit for bit
    untouched = orc.cnt == 0
    if w.dense_in is not None:
        want = w.dense_in.view(np.uint32 if w.out_dtype == "f32" else np.uint16)
        assert np.array_equal(raw_bits(run.out)[untouched], want[untouched])
    else:
        assert not raw_bits(run.out)[untouched].any()
    return orc
