"""Seeded synthetic IndexedSlices workloads.

This module only draws random inputs; it holds none of the densify arithmetic
and is the one piece of code that both the CPU oracle's tests and the CUDA
path's tests/benchmark share.  Everything is produced on the host as NumPy
arrays so that the very same bytes can be handed to either side.

An ``IndexedSlices`` gradient (paper Section 3) is a vector of row indices
plus a ``[n_rows, d]`` block of value rows.  The generators here stand in for
the sub-word token batches of the paper's WMT-17 English-German runs
(Section 5): token ids follow a bounded Zipf law, value rows are small
Gaussians like early-training embedding gradients.

bfloat16 arrays are carried as ``uint16`` bit patterns (NumPy has no bf16).
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np

__all__ = [
    "Workload",
    "zipf_indices",
    "to_bf16_bits",
    "make_workload",
    "CONFIG_NAMES",
    "SWEEP_DISTRIBUTIONS",
]

CONFIG_NAMES = ("tiny", "base", "big", "r64", "sweep_uniform", "sweep_zipf", "sweep_same")
SWEEP_DISTRIBUTIONS = ("uniform", "zipf", "same")


@dataclasses.dataclass
class Workload:
    """One densify problem: R slices, an optional dense partner, and dtypes."""

    name: str
    vocab: int
    d: int
    indices: List[np.ndarray]          # R arrays, int64 or int32, shape [n_r]
    values: List[np.ndarray]           # R arrays, float32 or uint16(bf16 bits), shape [n_r, d]
    dense_in: Optional[np.ndarray]     # [vocab, d] in the output dtype, or None
    index_dtype: str                   # "i64" | "i32"
    value_dtype: str                   # "f32" | "bf16"
    out_dtype: str                     # "f32" | "bf16"
    seed: int
    recipe: str                        # human-readable description of the draw

    @property
    def R(self) -> int:
        return len(self.indices)

    @property
    def n_rows_total(self) -> int:
        return int(sum(int(i.shape[0]) for i in self.indices))

    def concatenated(self):
        """Physical concatenation of all slices (what a sparse gather would hold)."""
        if self.R == 0:
            idt = np.int64 if self.index_dtype == "i64" else np.int32
            vdt = np.float32 if self.value_dtype == "f32" else np.uint16
            return np.zeros((0,), idt), np.zeros((0, self.d), vdt)
        return np.concatenate(self.indices), np.concatenate(self.values, axis=0)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 samples to bfloat16 (round-to-nearest-even), as uint16 bits.

    Input preparation only: it decides which bf16 numbers the random inputs
    are.  Done with integer arithmetic on the fp32 bit pattern.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    out = np.empty(u.shape, dtype=np.uint16)
    flat_u = u.reshape(-1)
    flat_o = out.reshape(-1)
    step = 1 << 24
    for s in range(0, flat_u.shape[0], step):
        w = flat_u[s:s + step]
        lsb = (w >> np.uint32(16)) & np.uint32(1)
        # finite samples only: the add cannot wrap below the NaN patterns
        r = (w + (lsb + np.uint32(0x7FFF))) >> np.uint32(16)
        flat_o[s:s + step] = r.astype(np.uint16)
    return out


_ZIPF_CDF_CACHE = {}


def _zipf_cdf(vocab: int, s: float) -> np.ndarray:
    key = (int(vocab), float(s))
    cdf = _ZIPF_CDF_CACHE.get(key)
    if cdf is None:
        w = np.arange(1, vocab + 1, dtype=np.float64) ** (-float(s))
        cdf = np.cumsum(w)
        cdf /= cdf[-1]
        _ZIPF_CDF_CACHE[key] = cdf
    return cdf


def zipf_indices(rng: np.random.Generator, n: int, vocab: int, s: float, dtype) -> np.ndarray:
    """Bounded Zipf: P(index = k) proportional to (k+1)^-s for k in [0, vocab).

    Sampled by inverting the normalised cumulative table; index 0 is the most
    frequent token.
    """
    cdf = _zipf_cdf(vocab, s)
    u = rng.random(n)
    k = np.searchsorted(cdf, u, side="right")
    np.minimum(k, vocab - 1, out=k)
    return k.astype(dtype)


def _normal_f32(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def _build(name, vocab, d, slice_rows, index_dtype, value_dtype, out_dtype, std,
           with_dense, seed, dist, zipf_s, permute_vocab, recipe):
    idt = np.int64 if index_dtype == "i64" else np.int32
    indices, values = [], []
    perm = None
    if permute_vocab:
        perm = np.random.default_rng(seed + 7919).permutation(vocab).astype(idt)
    for r, n in enumerate(slice_rows):
        # One generator per slice: slice r of a multi-slice workload is what
        # "rank r" would have drawn on its own.  Indices first, then values.
        rng = np.random.default_rng(seed + 1 + r)
        if dist == "zipf":
            idx = zipf_indices(rng, n, vocab, zipf_s, idt)
        elif dist == "uniform":
            idx = rng.integers(0, vocab, size=n, dtype=np.int64).astype(idt)
        elif dist == "same":
            idx = np.full((n,), int(rng.integers(0, vocab)), dtype=idt)
        else:
            raise ValueError(dist)
        if perm is not None:
            idx = perm[idx]
        v = _normal_f32(rng, (n, d), std)
        if value_dtype == "bf16":
            v = to_bf16_bits(v)
        indices.append(idx)
        values.append(v)
    dense_in = None
    if with_dense:
        rng = np.random.default_rng(seed + 1000003)
        dense_in = _normal_f32(rng, (vocab, d), std)
        if out_dtype == "bf16":
            dense_in = to_bf16_bits(dense_in)
    return Workload(name, vocab, d, indices, values, dense_in, index_dtype, value_dtype,
                    out_dtype, seed, recipe)


def make_workload(name: str, seed: int = 0, scale: float = 1.0, *, permute_vocab: bool = False,
                  out_dtype: Optional[str] = None, with_dense: Optional[bool] = None) -> Workload:
    """Build one of the named configurations.

    ``scale`` < 1 shrinks the number of rows per slice (never vocab or d) so
    that CPU tests can run a shape-alike case quickly.  ``permute_vocab``
    relabels token ids with a seeded permutation so that the frequent rows are
    not the low row numbers.

    Names
      tiny           vocab 1000,  d 64,   1 x 512 int64 Zipf(1.1), fp32 N(0,1), dense partner N(0,1)
      base           vocab 33708, d 512,  2 x 4096 int64 Zipf(1.1), fp32 N(0,0.02), dense partner
      big            vocab 33708, d 1024, 2 x 12800 int64 Zipf(1.1), fp32 N(0,0.02), dense partner
      r64            vocab 33708, d 1024, 64 x 10240 int64 Zipf(1.1), per-slice seed, dense partner
      sweep_uniform  vocab 65536, d 1024, 1 x 1048576 int32 uniform, bf16 N(0,1), no dense partner
      sweep_zipf     same, Zipf(1.2)
      sweep_same     same, every index equal
    """
    def rows(n):
        return max(1, int(round(n * scale))) if scale != 1.0 else n

    if name == "tiny":
        return _build(name, 1000, 64, [rows(512)], "i64", "f32", out_dtype or "f32", 1.0,
                      True if with_dense is None else with_dense, seed, "zipf", 1.1, permute_vocab,
                      "512 int64 ~ bounded Zipf(1.1) over [0,1000); values N(0,1) fp32 [512,64]; dense N(0,1)")
    if name == "base":
        return _build(name, 33708, 512, [rows(4096)] * 2, "i64", "f32", out_dtype or "f32", 0.02,
                      True if with_dense is None else with_dense, seed, "zipf", 1.1, permute_vocab,
                      "2 x 4096 int64 ~ bounded Zipf(1.1) over [0,33708); values N(0,0.02) fp32; dense N(0,0.02)")
    if name == "big":
        return _build(name, 33708, 1024, [rows(12800)] * 2, "i64", "f32", out_dtype or "f32", 0.02,
                      True if with_dense is None else with_dense, seed, "zipf", 1.1, permute_vocab,
                      "2 x 12800 int64 ~ bounded Zipf(1.1) over [0,33708); values N(0,0.02) fp32; dense N(0,0.02)")
    if name == "r64":
        return _build(name, 33708, 1024, [rows(10240)] * 64, "i64", "f32", out_dtype or "f32", 0.02,
                      True if with_dense is None else with_dense, seed, "zipf", 1.1, permute_vocab,
                      "64 x 10240 int64, slice r ~ bounded Zipf(1.1) with seed base+1+r; values N(0,0.02) fp32; dense N(0,0.02)")
    if name.startswith("sweep_"):
        dist = name.split("_", 1)[1]
        if dist not in SWEEP_DISTRIBUTIONS:
            raise ValueError(name)
        return _build(name, 65536, 1024, [rows(1048576)], "i32", "bf16", out_dtype or "bf16", 1.0,
                      False if with_dense is None else with_dense, seed, dist, 1.2, permute_vocab,
                      "1 x 1048576 int32 ~ %s over [0,65536); values N(0,1) bf16; no dense partner" % (
                          {"uniform": "uniform", "zipf": "bounded Zipf(1.2)", "same": "one repeated index"}[dist]))
    raise ValueError("unknown workload %r" % (name,))
