"""Host-side bookkeeping for running the densify path as independent replicas.

The path has no exchange step between GPUs: each data-parallel rank densifies its own
slices (paper Section 4); the all-reduce that follows in training is not part of it.
With N processes, whole-job throughput is the work of all ranks over the slowest rank's time.
"""
from __future__ import annotations

from typing import Optional


def combine_over_ranks(ms_per_step: float, bytes_per_step: int, rows_per_step: int, dist=None, device=None) -> dict:
    """max over ranks of the step time, sum over ranks of the work.  ``dist`` is an initialised
    ``torch.distributed`` module (any backend) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        t, b, r, n = float(ms_per_step), float(bytes_per_step), float(rows_per_step), 1
    else:
        import torch
        dev = device if (device is not None and dist.get_backend() == "nccl") else "cpu"
        tmax = torch.tensor([ms_per_step], dtype=torch.float64, device=dev)
        work = torch.tensor([bytes_per_step, rows_per_step], dtype=torch.float64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        dist.all_reduce(work, op=dist.ReduceOp.SUM)
        t, b, r, n = float(tmax.item()), float(work[0].item()), float(work[1].item()), dist.get_world_size()
    return {"ms_per_step": t, "gbs": b / t / 1e6 if t > 0 else 0.0, "rows_per_s": r / t * 1e3 if t > 0 else 0.0,
            "replicas": n}


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own slices, as each training rank would."""
    return int(base_seed) + 1000 * int(rank)
