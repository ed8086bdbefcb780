"""``dst_densify_apply_sgd`` through the C ABI against ``oracle.apply_sgd``: every path the densify call
has (one-cluster index path running beside the copy of the untouched rows, general path, heavy rows with their combine tree,
several slices, no dense partner, rows that are not 16-byte multiples, out-of-range indices)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_04035_b200 as dst
from paper_1905_04035_b200.workloads import make_workload

pytestmark = pytest.mark.gpu


def zipf_indices(rng, n, vocab, s=1.1, dtype=np.int64):
    p = 1.0 / np.arange(1, vocab + 1) ** s
    cdf = np.cumsum(p / p.sum())
    return np.minimum(np.searchsorted(cdf, rng.random(n)), vocab - 1).astype(dtype)


def run(indices, values, d, vocab, dense, weight, lr):
    dev = "cuda"
    slices = [(torch.from_numpy(i).to(dev), torch.from_numpy(v).to(dev)) for i, v in zip(indices, values)]
    n = sum(i.shape[0] for i in indices)
    idt = slices[0][0].dtype if slices else torch.int64
    w = torch.from_numpy(weight.copy()).to(dev)
    dn = torch.from_numpy(dense).to(dev) if dense is not None else None
    ws = torch.empty(max(256, dst.dst_workspace_bytes(n, len(slices), d, vocab, idt)), dtype=torch.uint8, device=dev)
    result = torch.zeros(8, dtype=torch.int32, device=dev)
    dst.dst_densify_apply_sgd(slices, d, vocab, dn, w, lr, ws, result=result, index_dtype=idt)
    torch.cuda.synchronize()
    if dn is not None:
        assert np.array_equal(dn.cpu().numpy(), dense)           # inputs are read-only
    return w.cpu().numpy(), result.cpu().numpy()


def check(indices, values, d, vocab, dense, weight, lr, exact=False):
    got, result = run(indices, values, d, vocab, dense, weight, lr)
    ref = oracle.apply_sgd(indices, values, d, vocab, dense, weight, lr)
    if exact:
        assert np.array_equal(got.astype(np.float64), ref.weight)
    else:
        assert np.all(np.abs(got.astype(np.float64) - ref.weight) <= 1e-5 * ref.mag + 1e-7)
    assert int(result[1]) == ref.grad.n_unique
    return got, ref, result


@pytest.mark.parametrize("name", ["tiny", "base", "big"])
def test_paper_configurations(name):
    w = make_workload(name)                                         # one-cluster index path, output pre-filled
    weight = np.random.default_rng(1).normal(0, 1, size=(w.vocab, w.d)).astype(np.float32)
    check(w.indices, w.values, w.d, w.vocab, w.dense_in, weight, 0.1)


@pytest.mark.parametrize("with_dense", [True, False])
@pytest.mark.parametrize("vocab,d,n,R", [(600, 64, 9000, 3), (70000, 32, 30000, 2), (3000, 1024, 2500, 1), (257, 2056, 40000, 4)])
def test_general_and_small_paths(vocab, d, n, R, with_dense):
    rng = np.random.default_rng(vocab + n)
    sizes = [n // R + (1 if r < n % R else 0) for r in range(R)]
    idx = [zipf_indices(rng, s, vocab) for s in sizes]               # a few very heavy rows: chunks and combine trees
    val = [rng.normal(0, 0.02, size=(s, d)).astype(np.float32) for s in sizes]
    dense = rng.normal(0, 0.02, size=(vocab, d)).astype(np.float32) if with_dense else None
    weight = rng.normal(0, 1, size=(vocab, d)).astype(np.float32)
    got, ref, _ = check(idx, val, d, vocab, dense, weight, 0.05)
    if not with_dense:
        untouched = ref.grad.cnt == 0
        assert np.array_equal(got[untouched], weight[untouched])     # rows nobody names keep their bits


def test_small_integers_are_exact_and_lr_sign():
    rng = np.random.default_rng(4)
    vocab, d, n = 900, 48, 20000
    idx = [zipf_indices(rng, n, vocab, dtype=np.int32)]
    val = [rng.integers(-4, 5, size=(n, d)).astype(np.float32)]
    dense = rng.integers(-4, 5, size=(vocab, d)).astype(np.float32)
    weight = rng.integers(-100, 101, size=(vocab, d)).astype(np.float32)
    for lr in (0.5, -0.25, 0.0):
        check(idx, val, d, vocab, dense, weight, lr, exact=True)


def test_unaligned_rows_and_out_of_range_indices():
    rng = np.random.default_rng(6)
    vocab, d, n = 300, 7, 2000                                      # 28-byte rows: the scalar kernel
    idx = [rng.integers(0, vocab, size=n)]
    idx[0][[3, 500, 1999]] = [-1, vocab, 1 << 40]
    val = [rng.integers(-4, 5, size=(n, d)).astype(np.float32)]
    dense = rng.integers(-4, 5, size=(vocab, d)).astype(np.float32)
    weight = rng.integers(-9, 10, size=(vocab, d)).astype(np.float32)
    _, ref, result = check(idx, val, d, vocab, dense, weight, 0.5, exact=True)
    assert int(result[0]) == 4 and ref.grad.n_out_of_range == 3     # DST_ERR_INDEX_OUT_OF_RANGE, rows skipped
    vocab, d = 300, 64
    val = [rng.integers(-4, 5, size=(n, d)).astype(np.float32)]
    dense = rng.integers(-4, 5, size=(vocab, d)).astype(np.float32)
    weight = rng.integers(-9, 10, size=(vocab, d)).astype(np.float32)
    _, _, result = check(idx, val, d, vocab, dense, weight, 0.5, exact=True)
    assert int(result[0]) == 4


def test_no_gradient_rows_and_refusals():
    vocab, d = 128, 16
    dense = np.ones((vocab, d), np.float32)
    weight = np.full((vocab, d), 3.0, np.float32)
    got, _ = run([], [], d, vocab, dense, weight, 0.5)
    assert np.all(got == 2.5)
    dev = "cuda"
    w = torch.zeros(vocab, d, device=dev)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=dev)
    with pytest.raises(dst.DstError):
        dst.dst_densify_apply_sgd([], d, vocab, w, w, 0.1, ws)        # the weight is not its own gradient
