"""The entry point for callers that cannot allocate device memory (``dst_densify_static``).

Such a caller -- a plugin that may not re-enter its host framework's allocator, a callback that
cannot afford cudaMalloc's device-wide synchronisation, a process whose memory pool is already
spoken for -- has no workspace to pass, so the library lends its own fixed array.  The result must
not depend on that: it is compared here with ``dst_densify`` on a caller-owned workspace, twice in
a row (the second call finds the array as the first one left it), on different shapes.

This file sorts last on purpose, so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

import paper_1905_04035_b200 as dst
from paper_1905_04035_b200 import binding
from paper_1905_04035_b200.workloads import make_workload

from gpu_helpers import raw_bits, to_device

pytestmark = pytest.mark.gpu


def _both(w):
    idx, val = to_device(w.indices[0], w.index_dtype), to_device(w.values[0], w.value_dtype)
    dense = to_device(w.dense_in, w.out_dtype) if w.dense_in is not None else None
    n, cap = w.n_rows_total, max(1, min(w.n_rows_total, w.vocab))
    outs = []
    for static in (False, True):
        out = torch.full((w.vocab, w.d), float("nan"), device="cuda")
        uniq = torch.full((cap,), -1, dtype=torch.int64, device="cuda")
        cnt = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
        res = torch.zeros(6, dtype=torch.int32, device="cuda")
        if static:
            dst.dst_densify_static(idx, val, w.d, w.vocab, dense, out, uniq, cnt, res)
        else:
            ws = torch.empty(dst.dst_workspace_bytes(n, 1, w.d, w.vocab), dtype=torch.uint8, device="cuda")
            dst.dst_densify(idx, val, w.d, w.vocab, dense, out, ws, uniq, cnt, res)
        torch.cuda.synchronize()
        outs.append((out, uniq.cpu().numpy(), cnt.cpu().numpy(), res.cpu().numpy()))
    return outs


def test_static_workspace_entry_point_matches_dst_densify_twice_in_a_row():
    # two calls in a row on different inputs, then the first again: leftovers must not matter
    for w in (make_workload("tiny", seed=0), make_workload("tiny", seed=1, with_dense=False),
              make_workload("tiny", seed=0)):
        assert dst.dst_workspace_bytes(w.n_rows_total, 1, w.d, w.vocab) <= binding.STATIC_WORKSPACE_BYTES
        (o0, u0, c0, r0), (o1, u1, c1, r1) = _both(w)
        got, want = o1.cpu().numpy().astype(np.float64), o0.cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        mag = np.abs(want) + 1.0
        assert np.all(np.abs(got - want) <= 1e-5 * mag + 1e-7)
        assert np.array_equal(raw_bits(o1), raw_bits(o0))      # same chunking, same order: same bits
        assert np.array_equal(u0, u1) and np.array_equal(c0, c1) and np.array_equal(r0, r1)
        assert r1[0] == 0 and r1[1] > 0


def test_static_workspace_entry_point_refuses_shapes_beyond_its_array():
    # grow the input until a caller-owned workspace would have to be larger than the library's array
    vocab, d, n = 5000, 256, 4096
    while dst.dst_workspace_bytes(n, 1, d, vocab) <= binding.STATIC_WORKSPACE_BYTES:
        n *= 2
    rng = np.random.default_rng(0)
    idx = torch.from_numpy(rng.integers(0, vocab, size=n)).cuda()
    val = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)).cuda()
    out = torch.zeros(vocab, d, device="cuda")
    with pytest.raises(dst.DstError) as e:
        dst.dst_densify_static(idx, val, d, vocab, None, out)
    assert e.value.status == 3
    torch.cuda.synchronize()
    assert not out.any()        # nothing was enqueued


def test_static_workspace_entry_point_against_the_oracle_on_both_index_paths_without_allocating():
    """Directly against the CPU oracle, on a shape that takes the one-cluster index path and on one that takes the
    general path (vocabulary above 65536: memset of the library's array, three radix passes, look-back
    descriptors), interleaved so each finds the other's leftovers -- and the device's free memory is the same
    before and after every call: the caller was promised that nothing is allocated."""
    import oracle
    small = make_workload("tiny", seed=3)
    rng = np.random.default_rng(5)
    vocab, d, n = 70000, 64, 2000
    idx = np.where(rng.random(n) < 0.3, 69999, rng.integers(0, vocab, size=n)).astype(np.int64)
    val = rng.standard_normal((n, d)).astype(np.float32)
    dense = rng.standard_normal((vocab, d)).astype(np.float32)
    assert dst.dst_workspace_bytes(n, 1, d, vocab) <= binding.STATIC_WORKSPACE_BYTES
    cases = [(small.indices[0], small.values[0], small.dense_in, small.vocab, small.d), (idx, val, dense, vocab, d)]
    dev = [tuple(torch.from_numpy(a).cuda() for a in c[:3]) for c in cases]
    outs = [torch.full((c[3], c[4]), float("nan"), device="cuda") for c in cases]
    res = torch.zeros(6, dtype=torch.int32, device="cuda")
    dst.dst_densify_static(*dev[0][:2], cases[0][4], cases[0][3], dev[0][2], outs[0], None, None, res)   # first call on the device
    torch.cuda.synchronize()
    for k in (1, 0, 1, 0):
        c = cases[k]
        outs[k].fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        dst.dst_densify_static(dev[k][0], dev[k][1], c[4], c[3], dev[k][2], outs[k], None, None, res)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        orc = oracle.densify([c[0]], [c[1]], c[4], c[3], c[2])
        got = outs[k].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - orc.acc) <= 1e-5 * orc.mag + 1e-7)
        assert int(res[0]) == 0 and int(res[1]) == orc.n_unique
