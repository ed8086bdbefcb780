"""The dense all-reduce that follows the local densify, driven with two gloo ranks on CPU tensors.  The local
densify is stood in for by the CPU oracle here (this is a test): what is under test is the exchange."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_04035_b200.reduce import densify_then_reduce, exchange_bytes, reduce_dense


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_inputs(rank, vocab, d, n):
    rng = np.random.default_rng(100 + rank)
    return (rng.integers(0, vocab, size=n), rng.integers(-4, 5, size=(n, d)).astype(np.float32),
            rng.integers(-4, 5, size=(vocab, d)).astype(np.float32))


def _worker(rank, world, port, q):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    vocab, d, n = 50, 4, 300
    idx, val, dense = _rank_inputs(rank, vocab, d, n)
    out = torch.empty(vocab, d)

    def local():
        out.copy_(torch.from_numpy(oracle.densify([idx], [val], d, vocab, dense).acc.astype(np.float32)))

    densify_then_reduce(local, out, dist)
    summed = out.clone()
    densify_then_reduce(local, out, dist, average=True)
    q.put((rank, summed.numpy(), out.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_sum_their_dense_gradients():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {r: (s, a) for r, s, a in (q.get(timeout=180) for _ in range(2))}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    vocab, d, n = 50, 4, 300
    want = np.zeros((vocab, d))
    for r in range(2):
        idx, val, dense = _rank_inputs(r, vocab, d, n)
        want += dense
        np.add.at(want, idx, val.astype(np.float64))
    for r in range(2):
        assert np.array_equal(got[r][0], want)              # small integers: exact; every rank holds the sum
        assert np.array_equal(got[r][1], want / 2)


def test_single_process_is_a_no_op_and_the_sizes_are_the_papers():
    t = torch.ones(3, 2)
    assert reduce_dense(t, None) is None and bool((t == 1).all())
    b = exchange_bytes(33708, 1024, 4, 10000, 0, 64)
    assert b["dense_reduce_bytes"] == 138067968
    assert abs(b["sparse_gather_bytes"] / 1e9 - 63 * 43708 * 4096 / 1e9) < 1e-9
