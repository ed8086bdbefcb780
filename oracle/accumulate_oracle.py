"""Oracle for the gradient-accumulation strategies of the paper.  TEST INFRASTRUCTURE ONLY.

Follows the paper's two algorithms step by step, in NumPy, with fp64 sums:

* Algorithm 1 (Section 3), the stock strategy: fewer than two gradients pass through; all-dense
  gradients are summed; anything else is turned into IndexedSlices (a dense [vocab, d] tensor becomes
  ``vocab`` slices, row v carrying index v, as Section 3 describes) and concatenated -- a gather.
* Algorithm 2 (Section 6), the proposed strategy: one more branch before the gather -- if at least
  one gradient is dense, every gradient is converted to a dense tensor and the tensors are summed.
* Listing 1 (Section 4), Horovod's ``sparse_as_dense``: every IndexedSlices gradient is converted to a
  dense tensor before accumulation, after which Algorithm 1 only ever sees dense tensors.

``conv_to_tensor`` of an IndexedSlices gradient is the scatter-sum of ``oracle.densify`` (duplicates
add up).  Nothing here is imported by the CUDA library or its binding.

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
    branch: str               # which line of the algorithm produced it
    grad: Optional[Grad]      # None for an empty input; dense values are float64 sums


def conv_to_tensor(g: Grad, d: int, vocab: int) -> np.ndarray:
    """``tf.convert_to_tensor`` of Listing 1: a dense tensor is itself, IndexedSlices are scatter-summed."""
    if g.is_dense:
        return np.asarray(g.values, np.float64).reshape(vocab, d)
    return dst_oracle.densify([np.asarray(g.indices)], [np.asarray(g.values, np.float32)], d, vocab).acc


def as_slices(g: Grad, d: int, vocab: int, index_dtype) -> Grad:
    """Algorithm 1's gather branch sees everything as IndexedSlices: a dense tensor names every row once."""
    if not g.is_dense:
        return g
    return Grad(np.asarray(g.values).reshape(vocab, d), np.arange(vocab, dtype=index_dtype))


def accumulate(grads: Sequence[Grad], d: int, vocab: int, strategy: str = PROPOSED,
               index_dtype=np.int64) -> Accumulated:
    grads = list(grads)
    if strategy == SPARSE_AS_DENSE:
        # Listing 1: convert each IndexedSlices gradient first, then the stock algorithm runs
        grads = [g if g.is_dense else Grad(conv_to_tensor(g, d, vocab)) for g in grads]
    elif strategy not in (STOCK, PROPOSED):
        raise ValueError(strategy)
    # line 1-2 of both algorithms
    if len(grads) < 2:
        return Accumulated(PASS_THROUGH, grads[0] if grads else None)
    # line 3-4 of both algorithms
    if all(g.is_dense for g in grads):
        total = np.zeros((vocab, d), np.float64)
        for g in grads:
            total += np.asarray(g.values, np.float64).reshape(vocab, d)
        return Accumulated(REDUCE, Grad(total))
    # Algorithm 2 only: any dense gradient -> convert all, reduce
    if strategy == PROPOSED and any(g.is_dense for g in grads):
        total = np.zeros((vocab, d), np.float64)
        for g in grads:
            total += conv_to_tensor(g, d, vocab)
        return Accumulated(CONVERT_AND_REDUCE, Grad(total))
    # last branch of both: gather (concatenation of IndexedSlices in the order given)
    parts: List[Grad] = [as_slices(g, d, vocab, index_dtype) for g in grads]
    indices = np.concatenate([np.asarray(p.indices).astype(index_dtype) for p in parts])
    values = np.concatenate([np.asarray(p.values).reshape(-1, d) for p in parts], axis=0)
    return Accumulated(GATHER, Grad(values, indices))
