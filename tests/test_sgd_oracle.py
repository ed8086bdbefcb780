"""Pins for the oracle of the fused SGD step (``oracle.apply_sgd``)."""
import numpy as np

import oracle


def test_hand_worked_example():
    # vocab 3, d 2, lr 0.5: w = [[1,1],[2,2],[3,3]], dense = [[2,0],[0,2],[4,4]], slices name row 2 twice and row 0 once
    w = np.array([[1, 1], [2, 2], [3, 3]], np.float32)
    dense = np.array([[2, 0], [0, 2], [4, 4]], np.float32)
    idx = [np.array([2, 0, 2], np.int64)]
    val = [np.array([[2, 2], [4, 6], [6, 6]], np.float32)]
    r = oracle.apply_sgd(idx, val, 2, 3, dense, w, 0.5)
    # gradient: row0 = [6,6], row1 = [0,2], row2 = [12,12]
    assert r.weight.tolist() == [[-2.0, -2.0], [2.0, 1.0], [-3.0, -3.0]]
    assert r.out.dtype == np.float32 and r.out.tolist() == r.weight.tolist()
    assert r.mag.tolist() == [[1 + 3, 1 + 3], [2 + 0, 2 + 1], [3 + 6, 3 + 6]]


def test_equals_densify_then_a_library_step_and_is_linear_in_lr():
    rng = np.random.default_rng(0)
    vocab, d, n = 37, 5, 200
    idx = [rng.integers(0, vocab, size=n)]
    val = [rng.integers(-8, 9, size=(n, d)).astype(np.float32)]
    dense = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    w = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    g = np.zeros((vocab, d))
    np.add.at(g, idx[0], val[0].astype(np.float64))             # library scatter-add
    g += dense
    for lr in (0.0, 0.25, -2.0):
        r = oracle.apply_sgd(idx, val, d, vocab, dense, w, lr)
        assert np.array_equal(r.weight, w - lr * g)              # exact: small integers, dyadic lr
    assert np.array_equal(oracle.apply_sgd(idx, val, d, vocab, None, w, 1.0).weight, w - (g - dense))
    # rows nobody names and no dense partner: the weight stays
    r = oracle.apply_sgd([np.array([3])], [np.ones((1, d), np.float32)], d, vocab, None, w, 0.5)
    keep = np.arange(vocab) != 3
    assert np.array_equal(r.weight[keep], w[keep]) and np.array_equal(r.weight[3], w[3] - 0.5)
