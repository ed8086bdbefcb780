"""Oracle for the gradient-accumulation strategies of the paper.  TEST INFRASTRUCTURE ONLY.

What a list of gradients of one variable accumulates to, in NumPy, with fp64 sums:

* the stock rule (Section 3, Algorithm 1): a list of fewer than two gradients is handed on unchanged;
  a list of dense tensors only is summed; any other list is turned into IndexedSlices (a dense
  [vocab, d] tensor becomes ``vocab`` slices, row v carrying index v, as Section 3 describes) and
  concatenated -- a gather;
* the proposed rule (Section 6, Algorithm 2): the same, except that a mixed list holding at least one
  dense tensor is converted to dense tensors and summed instead of gathered;
* Horovod's ``sparse_as_dense`` (Section 4, Listing 1): every IndexedSlices gradient is made dense
  before the stock rule sees the list, which can then only pass through or sum.

Making IndexedSlices dense is the scatter-sum of ``oracle.densify`` (duplicates add up).  Nothing here
is imported by the CUDA library or its binding.

Pins: ``tests/test_accumulate_oracle.py`` (hand-worked example, strategy-independence of the
accumulated value, the paper's row counts, pass-through identity, library sum).
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np

from . import dst_oracle

STOCK, PROPOSED, SPARSE_AS_DENSE = "stock", "proposed", "sparse_as_dense"
PASS_THROUGH, REDUCE, CONVERT_AND_REDUCE, GATHER = "pass-through", "reduce", "convert+reduce", "gather"


@dataclasses.dataclass
class Grad:
    """A gradient: dense ([vocab, d] array in ``values``) or IndexedSlices (``indices`` + [n, d] ``values``)."""
    values: np.ndarray
    indices: Optional[np.ndarray] = None

    @property
    def is_dense(self) -> bool:
        return self.indices is None


@dataclasses.dataclass
class Accumulated:
    branch: str               # which rule produced it
    grad: Optional[Grad]      # None for an empty input; dense values are float64 sums


def densified(g: Grad, d: int, vocab: int) -> np.ndarray:
    """The gradient as a dense fp64 [vocab, d] array: a dense tensor is itself, IndexedSlices are scatter-summed."""
    if g.is_dense:
        return np.asarray(g.values, np.float64).reshape(vocab, d)
    return dst_oracle.densify([np.asarray(g.indices)], [np.asarray(g.values, np.float32)], d, vocab).acc


def as_slices(g: Grad, d: int, vocab: int, index_dtype) -> Grad:
    """The gradient as IndexedSlices: a dense tensor names every row once (Section 3)."""
    if not g.is_dense:
        return g
    return Grad(np.asarray(g.values).reshape(vocab, d), np.arange(vocab, dtype=index_dtype))


def rule(n: int, n_dense: int, strategy: str) -> str:
    """Which rule a list of ``n`` gradients, ``n_dense`` of them dense, falls under."""
    if n < 2:
        return PASS_THROUGH
    if n_dense == n:
        return REDUCE
    if strategy == PROPOSED and n_dense > 0:
        return CONVERT_AND_REDUCE
    return GATHER


def accumulate(grads: Sequence[Grad], d: int, vocab: int, strategy: str = PROPOSED,
               index_dtype=np.int64) -> Accumulated:
    if strategy not in (STOCK, PROPOSED, SPARSE_AS_DENSE):
        raise ValueError(strategy)
    grads = list(grads)
    if strategy == SPARSE_AS_DENSE:
        grads = [g if g.is_dense else Grad(densified(g, d, vocab)) for g in grads]
    how = rule(len(grads), sum(g.is_dense for g in grads), strategy)
    if how == PASS_THROUGH:
        return Accumulated(how, grads[0] if grads else None)
    if how in (REDUCE, CONVERT_AND_REDUCE):
        total = np.zeros((vocab, d), np.float64)
        for g in grads:
            total += densified(g, d, vocab)
        return Accumulated(how, Grad(total))
    # gather: the concatenation of the IndexedSlices forms, in the order given
    parts: List[Grad] = [as_slices(g, d, vocab, index_dtype) for g in grads]
    indices = np.concatenate([np.asarray(p.indices).astype(index_dtype) for p in parts])
    values = np.concatenate([np.asarray(p.values).reshape(-1, d) for p in parts], axis=0)
    return Accumulated(GATHER, Grad(values, indices))
