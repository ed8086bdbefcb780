"""Pins for the multi-core fp32 CPU baseline (``oracle/dst_cpu_threads.c``).

It is only a timed baseline, but a baseline that computed something else would make its number
meaningless, so it is held to the fp64 oracle (itself pinned in ``test_oracle_pins.py``) and to
closed forms: small-integer data must agree bit for bit whatever the number of threads.
"""
import numpy as np
import pytest

import oracle
from paper_1905_04035_b200.workloads import make_workload, to_bf16_bits


def _int_case(seed, n, d, vocab, R, index_dtype=np.int64):
    rng = np.random.default_rng(seed)
    sizes = [n // R + (1 if r < n % R else 0) for r in range(R)]
    idx = [rng.integers(0, vocab, size=s).astype(index_dtype) for s in sizes]
    val = [rng.integers(-8, 9, size=(s, d)).astype(np.float32) for s in sizes]
    dense = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    return idx, val, dense


@pytest.mark.parametrize("n_threads", [1, 3, 8, 64])
def test_small_integers_bit_exact_for_any_thread_count(n_threads):
    idx, val, dense = _int_case(1, 3000, 40, 97, 3)
    ref = oracle.densify(idx, val, 40, 97, dense)
    out, bad, used = oracle.densify_threads(idx, val, 40, 97, dense, n_threads=n_threads)
    assert bad == 0 and used == min(n_threads, 40)
    assert np.array_equal(out, ref.out)


def test_no_dense_partner_and_int32_indices():
    idx, val, _ = _int_case(2, 500, 16, 33, 2, np.int32)
    ref = oracle.densify(idx, val, 16, 33, None)
    out, bad, _ = oracle.densify_threads(idx, val, 16, 33, None, n_threads=4)
    assert bad == 0 and np.array_equal(out, ref.out)
    untouched = np.setdiff1d(np.arange(33), np.concatenate(idx))
    assert np.all(out[untouched] == 0.0)


def test_out_of_range_rows_are_skipped_and_counted():
    idx, val, dense = _int_case(3, 400, 8, 21, 1)
    idx[0][5] = -1
    idx[0][17] = 21
    idx[0][399] = 10**12
    ref = oracle.densify(idx, val, 8, 21, dense)
    out, bad, _ = oracle.densify_threads(idx, val, 8, 21, dense, n_threads=5)
    assert bad == 3 == ref.n_out_of_range
    assert np.array_equal(out, ref.out)


def test_all_same_index_closed_form():
    n, d, vocab = 4096, 24, 7
    idx = [np.full((n,), 4, np.int64)]
    val = [np.ones((n, d), np.float32)]
    out, _, _ = oracle.densify_threads(idx, val, d, vocab, None, n_threads=6)
    assert np.all(out[4] == float(n))
    assert np.all(np.delete(out, 4, axis=0) == 0.0)


def test_real_valued_data_within_fp32_tolerance():
    w = make_workload("tiny")
    ref = oracle.densify(w.indices, w.values, w.d, w.vocab, w.dense_in)
    out, bad, _ = oracle.densify_threads(w.indices, w.values, w.d, w.vocab, w.dense_in, n_threads=7)
    assert bad == 0
    # a sequential fp32 sum of n terms: error below n * 2^-24 * sum|terms|
    tol = (ref.max_segment + 1) * 2.0 ** -24 * ref.mag + 1e-30
    assert np.all(np.abs(out.astype(np.float64) - ref.acc) <= tol)


def test_bf16_values_and_bf16_output():
    rng = np.random.default_rng(5)
    n, d, vocab = 800, 32, 50
    idx = [rng.integers(0, vocab, size=n).astype(np.int32)]
    val = [to_bf16_bits(rng.integers(-8, 9, size=(n, d)).astype(np.float32))]
    ref = oracle.densify(idx, val, d, vocab, None, value_dtype="bf16", out_dtype="bf16")
    out, _, _ = oracle.densify_threads(idx, val, d, vocab, None, value_dtype="bf16", out_dtype="bf16", n_threads=4)
    # integer sums below 2^24 are exact in fp32, and one rounding to bf16 follows on both sides
    assert np.array_equal(out, ref.out)


def test_empty_input_returns_the_dense_partner():
    dense = np.arange(12, dtype=np.float32).reshape(3, 4)
    out, bad, _ = oracle.densify_threads([], [], 4, 3, dense, n_threads=2)
    assert bad == 0 and np.array_equal(out, dense)
