"""The exchange step that follows the local densify in data-parallel training: a sum all-reduce of the
fixed-size dense [vocab, d] gradient (the paper's Fig. 3b "reduce" and Section 4: 139 MB whatever the
number of ranks), in place of the gather of IndexedSlices whose buffers grow with the rank count.

Plumbing only: ``torch.distributed`` does the collective (NCCL over NVLink on GPUs; any backend works,
which is how the CPU tests drive it).  The local densify writes straight into the tensor that is then
reduced, so no staging copy sits between the two.  No kernel of this package touches another GPU's memory.
"""
from __future__ import annotations

from typing import Callable, Optional


def reduce_dense(out, dist, group=None, average: bool = False, async_op: bool = False):
    """All-reduce ``out`` (sum over ranks) in place.  ``average=True`` divides by the number of ranks
    afterwards, as Horovod's allreduce does; the densify calls themselves never scale.
    Returns the work handle when ``async_op`` (the division is then the caller's), else None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return None
    work = dist.all_reduce(out, op=dist.ReduceOp.SUM, group=group, async_op=async_op)
    if async_op:
        return work
    if average:
        out.div_(dist.get_world_size(group))
    return None


def densify_then_reduce(densify_local: Callable[[], None], out, dist, group=None, average: bool = False):
    """One accumulation step of a rank: ``densify_local()`` enqueues this rank's densify into ``out``
    (e.g. ``lambda: engine(slices, dense_in, out)``), then ``out`` is summed over the ranks.  Both run on
    the current stream, in order; with the NCCL backend nothing synchronises with the host."""
    densify_local()
    reduce_dense(out, dist, group=group, average=average)
    return out


def exchange_bytes(vocab: int, d: int, elem_size: int, n_rows_per_rank: int, index_size: int, world: int) -> dict:
    """What each rank has to receive per step either way (Section 4): the dense tensor once, against every
    other rank's IndexedSlices when they are gathered with the dense partner turned into slices too."""
    dense = vocab * d * elem_size
    gathered = (world - 1) * (vocab + n_rows_per_rank) * (d * elem_size + index_size)
    return {"dense_reduce_bytes": dense, "sparse_gather_bytes": gathered, "ratio": gathered / dense if dense else 0.0}
