"""N > 1 runs are independent replicas; their host-side aggregation is tested with gloo on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_04035_b200.replicas import combine_over_ranks, replica_seed


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 2.0 if rank == 0 else 5.0          # rank 1 is the slow one
    out = combine_over_ranks(ms, 1000 * (rank + 1), 10 * (rank + 1), dist)
    dist.barrier()
    q.put((rank, out))
    dist.destroy_process_group()


def test_two_replicas_max_time_sum_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in (0, 1):
        assert got[r]["ms_per_step"] == 5.0
        assert got[r]["replicas"] == 2
        assert abs(got[r]["gbs"] - 3000 / 5.0 / 1e6) < 1e-15
        assert abs(got[r]["rows_per_s"] - 30 / 5.0 * 1e3) < 1e-9


def test_single_process():
    out = combine_over_ranks(4.0, 8_000_000, 100)
    assert out == {"ms_per_step": 4.0, "gbs": 2.0, "rows_per_s": 25000.0, "replicas": 1}
    assert replica_seed(3, 0) == 3 and replica_seed(3, 2) == 2003
