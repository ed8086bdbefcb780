"""Pins for the oracle of the paper's accumulation strategies (Algorithm 1, Algorithm 2, Listing 1)."""
import numpy as np
import pytest

import oracle
from oracle import accumulate_oracle as ao


def _case(seed=0, vocab=11, d=3, sizes=(5, 7), with_dense=True):
    rng = np.random.default_rng(seed)
    grads = []
    if with_dense:
        grads.append(ao.Grad(rng.integers(-4, 5, size=(vocab, d)).astype(np.float32)))
    for n in sizes:
        grads.append(ao.Grad(rng.integers(-4, 5, size=(n, d)).astype(np.float32),
                             rng.integers(0, vocab, size=n).astype(np.int64)))
    return grads, d, vocab


def test_hand_worked_example():
    # vocab 3, d 1: dense [10, 20, 30]; slices {(2, 1), (0, 5), (2, 7)}
    dense = ao.Grad(np.array([[10.0], [20.0], [30.0]], np.float32))
    sl = ao.Grad(np.array([[1.0], [5.0], [7.0]], np.float32), np.array([2, 0, 2], np.int64))
    out = ao.accumulate([dense, sl], 1, 3, ao.PROPOSED)
    assert out.branch == ao.CONVERT_AND_REDUCE and out.grad.is_dense
    assert out.grad.values.ravel().tolist() == [15.0, 20.0, 38.0]
    st = ao.accumulate([dense, sl], 1, 3, ao.STOCK)
    assert st.branch == ao.GATHER and not st.grad.is_dense
    assert st.grad.indices.tolist() == [0, 1, 2, 2, 0, 2]
    assert st.grad.values.ravel().tolist() == [10.0, 20.0, 30.0, 1.0, 5.0, 7.0]


@pytest.mark.parametrize("strategy", [ao.STOCK, ao.PROPOSED, ao.SPARSE_AS_DENSE])
def test_branches(strategy):
    grads, d, vocab = _case()
    assert ao.accumulate([], d, vocab, strategy).grad is None
    one = ao.accumulate(grads[:1], d, vocab, strategy)
    assert one.branch == ao.PASS_THROUGH and one.grad is grads[0]
    dd = ao.accumulate([grads[0], grads[0]], d, vocab, strategy)
    assert dd.branch == ao.REDUCE and np.array_equal(dd.grad.values, 2.0 * grads[0].values)
    mixed = ao.accumulate(grads, d, vocab, strategy)
    assert mixed.branch == {ao.STOCK: ao.GATHER, ao.PROPOSED: ao.CONVERT_AND_REDUCE, ao.SPARSE_AS_DENSE: ao.REDUCE}[strategy]
    sparse = ao.accumulate(grads[1:], d, vocab, strategy)
    assert sparse.branch == (ao.REDUCE if strategy == ao.SPARSE_AS_DENSE else ao.GATHER)


def test_accumulated_value_does_not_depend_on_the_strategy():
    """Gather and reduce are two encodings of the same gradient: densifying the gathered slices gives the
    reduced tensor (exact here: small integers)."""
    grads, d, vocab = _case(seed=3, vocab=17, d=4, sizes=(9, 30, 1))
    ref = ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values
    direct = np.zeros((vocab, d))
    direct += grads[0].values
    for g in grads[1:]:
        np.add.at(direct, g.indices, g.values.astype(np.float64))     # library scatter-add
    assert np.array_equal(ref, direct)
    st = ao.accumulate(grads, d, vocab, ao.STOCK).grad
    assert np.array_equal(ao.densified(st, d, vocab), ref)
    assert np.array_equal(ao.accumulate(grads, d, vocab, ao.SPARSE_AS_DENSE).grad.values, ref)
    # all-sparse input: the gathered slices densify to what sparse_as_dense reduces to
    sp = ao.accumulate(grads[1:], d, vocab, ao.STOCK).grad
    assert np.array_equal(ao.densified(sp, d, vocab), ao.accumulate(grads[1:], d, vocab, ao.SPARSE_AS_DENSE).grad.values)


def test_gather_row_count_is_the_papers_accounting():
    """Section 4: with the projection gradient turned into vocab slices, one rank gathers vocab + n_enc + n_dec
    rows; 64 such ranks at 5000 tokens each give the 11.4 GB the paper prints, against 139 MB dense."""
    vocab, d, n = 33708, 2, 5000
    rng = np.random.default_rng(0)
    grads = [ao.Grad(np.zeros((vocab, d), np.float32))] + [
        ao.Grad(np.zeros((n, d), np.float32), rng.integers(0, vocab, size=n)) for _ in range(2)]
    st = ao.accumulate(grads, d, vocab, ao.STOCK)
    assert st.grad.indices.shape[0] == vocab + 2 * n == 43708
    rep = oracle.bytes_report([2 * n] * 64, 1024, vocab)
    assert rep["gather_all_value_bytes"] == 64 * 43708 * 1024 * 4       # 11.46 GB
    assert rep["dense_bytes"] == 138067968                               # 139 MB
    assert ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values.shape == (vocab, d)


def test_gather_keeps_input_order_and_index_dtype():
    grads, d, vocab = _case(seed=5, with_dense=False, sizes=(4, 6))
    out = ao.accumulate(grads, d, vocab, ao.STOCK, index_dtype=np.int32).grad
    assert out.indices.dtype == np.int32
    assert np.array_equal(out.indices, np.concatenate([g.indices for g in grads]))
    assert np.array_equal(out.values, np.concatenate([g.values for g in grads]))
