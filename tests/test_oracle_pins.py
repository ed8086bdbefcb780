"""Pins for the CPU oracle: checks that do not come from the oracle itself.

Each check targets a mistake the oracle could plausibly contain (a dropped
term, last-write-wins instead of a sum, an off-by-one row, a transposed value
block, a forgotten slice, invalid rows being counted).  The same battery is
run over deliberately broken NumPy implementations at the end of this file to
show that every one of those mistakes is caught.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_1905_04035_b200.workloads import make_workload, to_bf16_bits


# --------------------------------------------------------------------------
# independent formulations
# --------------------------------------------------------------------------
def brute_force(indices, values, d, vocab, dense_in):
    """Gather form, element by element, with exactly rounded sums (math.fsum)."""
    out = np.zeros((vocab, d), np.float64)
    idx = np.concatenate(indices) if len(indices) else np.zeros((0,), np.int64)
    val = np.concatenate(values, axis=0).astype(np.float64) if len(values) else np.zeros((0, d))
    for v in range(vocab):
        rows = [i for i in range(idx.shape[0]) if idx[i] == v]
        for c in range(d):
            terms = [val[i, c] for i in rows]
            if dense_in is not None:
                terms.append(float(dense_in[v, c]))
            out[v, c] = math.fsum(terms)
    return out


def oracle_acc(indices, values, d, vocab, dense_in):
    return oracle.densify(indices, values, d, vocab, dense_in).acc


def _small_case(seed, vocab=13, d=5, ns=(7, 0, 9), with_dense=True, integer=False):
    rng = np.random.default_rng(seed)
    indices = [rng.integers(0, vocab, size=n).astype(np.int64) for n in ns]
    if integer:
        values = [rng.integers(-8, 9, size=(n, d)).astype(np.float32) for n in ns]
        dense = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32) if with_dense else None
    else:
        values = [rng.standard_normal((n, d)).astype(np.float32) for n in ns]
        dense = rng.standard_normal((vocab, d)).astype(np.float32) if with_dense else None
    return indices, values, d, vocab, dense


# --------------------------------------------------------------------------
# the battery: takes any implementation f(indices, values, d, vocab, dense_in) -> [vocab, d] float64
# --------------------------------------------------------------------------
def pin_brute_force(f):
    for seed in range(3):
        case = _small_case(seed, with_dense=(seed != 1))
        got = f(*case)
        want = brute_force(*case)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)


def pin_library_scatter_add(f):
    w = make_workload("tiny")
    got = f(w.indices, w.values, w.d, w.vocab, w.dense_in)
    ref = w.dense_in.astype(np.float64).copy()
    np.add.at(ref, w.indices[0], w.values[0].astype(np.float64))
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    t = torch.from_numpy(w.dense_in).double()
    t.index_add_(0, torch.from_numpy(w.indices[0]), torch.from_numpy(w.values[0]).double())
    np.testing.assert_allclose(got, t.numpy(), rtol=0, atol=1e-12)


def pin_column_sums(f):
    w = make_workload("base", scale=0.05)
    got = f(w.indices, w.values, w.d, w.vocab, w.dense_in)
    want = w.dense_in.astype(np.float64).sum(axis=0)
    for v in w.values:
        want = want + v.astype(np.float64).sum(axis=0)
    scale = np.abs(w.dense_in.astype(np.float64)).sum(axis=0)
    for v in w.values:
        scale = scale + np.abs(v.astype(np.float64)).sum(axis=0)
    assert np.all(np.abs(got.sum(axis=0) - want) <= 1e-12 * scale)


def pin_exact_integers(f):
    # small integers: every partial sum is an integer below 2^24, so any order is exact
    case = _small_case(11, vocab=17, d=6, ns=(40, 25), integer=True)
    indices, values, d, vocab, dense = case
    ref = dense.astype(np.int64).copy()
    for ix, va in zip(indices, values):
        np.add.at(ref, ix, va.astype(np.int64))
    got = f(*case)
    assert np.array_equal(got, ref.astype(np.float64))


def pin_all_same_index(f):
    n, d, vocab, v0 = 4096, 3, 9, 4
    idx = [np.full((n,), v0, np.int64)]
    val = [np.ones((n, d), np.float32)]
    dense = np.full((vocab, d), 0.5, np.float32)
    got = f(idx, val, d, vocab, dense)
    want = np.full((vocab, d), 0.5)
    want[v0, :] = n + 0.5
    assert np.array_equal(got, want)
    got = f(idx, val, d, vocab, None)
    want = np.zeros((vocab, d))
    want[v0, :] = n
    assert np.array_equal(got, want)


def pin_all_unique(f):
    rng = np.random.default_rng(5)
    vocab, d, n = 50, 4, 20
    idx = [rng.permutation(vocab)[:n].astype(np.int64)]
    val = [rng.standard_normal((n, d)).astype(np.float32)]
    dense = rng.standard_normal((vocab, d)).astype(np.float32)
    got = f(idx, val, d, vocab, dense)
    want = dense.astype(np.float64).copy()
    want[idx[0]] = dense[idx[0]].astype(np.float64) + val[0].astype(np.float64)
    assert np.array_equal(got, want)
    # untouched rows are the dense partner exactly
    untouched = np.setdiff1d(np.arange(vocab), idx[0])
    assert np.array_equal(got[untouched], dense[untouched].astype(np.float64))


def pin_linearity(f):
    indices, values, d, vocab, dense = _small_case(21, vocab=11, d=4, ns=(30, 12), integer=True)
    both = f(indices, values, d, vocab, dense)
    first = f(indices[:1], values[:1], d, vocab, dense)
    second = f(indices[1:], values[1:], d, vocab, first.astype(np.float32))
    assert np.array_equal(both, second)
    # slice order and row order are irrelevant for exact data
    p = np.random.default_rng(0).permutation(indices[0].shape[0])
    shuffled = f([indices[1], indices[0][p]], [values[1], values[0][p]], d, vocab, dense)
    assert np.array_equal(both, shuffled)


def pin_empty_inputs(f):
    indices, values, d, vocab, dense = _small_case(3, ns=(6,))
    base = f(indices, values, d, vocab, dense)
    e_i, e_v = np.zeros((0,), np.int64), np.zeros((0, d), np.float32)
    with_empty = f([e_i, indices[0], e_i], [e_v, values[0], e_v], d, vocab, dense)
    assert np.array_equal(base, with_empty)
    assert np.array_equal(f([], [], d, vocab, dense), dense.astype(np.float64))
    assert np.array_equal(f([e_i], [e_v], d, vocab, None), np.zeros((vocab, d)))


def pin_out_of_range_rows_are_skipped(f):
    indices, values, d, vocab, dense = _small_case(8, ns=(10,))
    idx = indices[0].copy()
    idx[[2, 5]] = [-1, vocab]
    got = f([idx], values, d, vocab, dense)
    keep = np.array([i for i in range(10) if i not in (2, 5)])
    want = f([indices[0][keep]], [values[0][keep]], d, vocab, dense)
    assert np.array_equal(got, want)


BATTERY = [pin_brute_force, pin_library_scatter_add, pin_column_sums, pin_exact_integers,
           pin_all_same_index, pin_all_unique, pin_linearity, pin_empty_inputs,
           pin_out_of_range_rows_are_skipped]


@pytest.mark.parametrize("pin", BATTERY, ids=lambda p: p.__name__)
def test_oracle_passes(pin):
    pin(oracle_acc)


# --------------------------------------------------------------------------
# everything else the oracle returns
# --------------------------------------------------------------------------
def test_counts_and_unique_rows():
    for name, scale in (("tiny", 1.0), ("base", 0.25)):
        w = make_workload(name, scale=scale)
        r = oracle.densify(w.indices, w.values, w.d, w.vocab, w.dense_in)
        allidx = np.concatenate(w.indices)
        u, c = np.unique(allidx, return_counts=True)
        assert np.array_equal(r.unique_rows, u) and r.unique_rows.dtype == allidx.dtype
        assert np.array_equal(r.counts, c.astype(np.int32))
        assert r.n_unique == u.shape[0] and r.counts.sum() == allidx.shape[0]
        assert r.max_segment == c.max() and r.n_out_of_range == 0
        assert np.array_equal(r.cnt, np.bincount(allidx, minlength=w.vocab))


def test_counts_skip_out_of_range():
    idx = np.array([3, -7, 3, 10, 9, 2 ** 40], dtype=np.int64)
    val = np.ones((6, 2), np.float32)
    r = oracle.densify([idx], [val], 2, 10)
    assert r.n_out_of_range == 3
    assert np.array_equal(r.unique_rows, [3, 9]) and np.array_equal(r.counts, [2, 1])
    idx32 = np.array([0, -1, 5, 5], dtype=np.int32)
    r = oracle.densify([idx32], [np.ones((4, 1), np.float32)], 1, 5)
    assert r.n_out_of_range == 3 and r.unique_rows.dtype == np.int32 and np.array_equal(r.unique_rows, [0])


def test_mag_is_sum_of_absolute_terms():
    indices, values, d, vocab, dense = _small_case(4)
    r = oracle.densify(indices, values, d, vocab, dense)
    absr = oracle.densify(indices, [np.abs(v) for v in values], d, vocab, np.abs(dense))
    np.testing.assert_allclose(r.mag, absr.acc, rtol=0, atol=1e-13)
    np.testing.assert_allclose(r.mag, brute_force(indices, [np.abs(v) for v in values], d, vocab, np.abs(dense)),
                               rtol=0, atol=1e-13)
    assert np.all(r.mag >= np.abs(r.acc) - 1e-13)


def test_rounded_output_fp32():
    indices, values, d, vocab, dense = _small_case(6)
    r = oracle.densify(indices, values, d, vocab, dense)
    assert r.out.dtype == np.float32
    assert np.array_equal(r.out, r.acc.astype(np.float32))


def test_bf16_widening_is_exact_and_rounding_is_nearest_even():
    # every finite bf16 pattern survives widen -> round
    for bits in range(0, 1 << 16, 1):
        if (bits & 0x7F80) == 0x7F80:
            continue  # inf / nan
        x = oracle.widen_bf16(bits)
        u = np.array([bits << 16], dtype=np.uint32).view(np.float32)[0]
        assert x == float(u)
        if bits % 97 == 0 or bits < 300:
            assert oracle.round_bf16(x) == bits
    one, nxt = 0x3F80, 0x3F81           # 1.0 and 1 + 2^-7
    mid = 1.0 + 2.0 ** -8
    assert oracle.round_bf16(mid) == one                   # tie -> even mantissa
    assert oracle.round_bf16(1.0 + 2.0 ** -7 + 2.0 ** -8) == 0x3F82   # tie -> even (up)
    assert oracle.round_bf16(mid + 2.0 ** -40) == nxt      # would be lost by rounding through fp32 first
    assert oracle.round_bf16(mid - 2.0 ** -40) == one
    assert oracle.round_bf16(-mid - 2.0 ** -40) == (0x8000 | nxt)
    assert oracle.round_bf16(0.0) == 0 and oracle.round_bf16(float("inf")) == 0x7F80
    assert oracle.round_bf16(3.4e38) == 0x7F80             # rounds past the largest finite bf16
    assert oracle.round_bf16(2.0 ** -133) == 0x0001        # smallest subnormal
    assert oracle.round_bf16(2.0 ** -134) == 0x0000        # tie to even (zero)


def test_bf16_values_match_torch_scatter_add():
    rng = np.random.default_rng(9)
    vocab, d, n = 40, 8, 300
    idx = rng.integers(0, vocab, size=n).astype(np.int32)
    bits = to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    r = oracle.densify([idx], [bits], d, vocab, None, value_dtype="bf16", out_dtype="bf16")
    vals = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double()
    ref = torch.zeros(vocab, d, dtype=torch.float64).index_add_(0, torch.from_numpy(idx).long(), vals)
    np.testing.assert_allclose(r.acc, ref.numpy(), rtol=0, atol=1e-12)
    assert r.out.dtype == np.uint16
    # rounded output within half a bf16 ulp of the fp64 sum
    back = torch.from_numpy(r.out.view(np.int16)).view(torch.bfloat16).double().numpy()
    assert np.all(np.abs(back - r.acc) <= 2.0 ** -8 * np.abs(r.acc) + 1e-300)
    # bf16 dense partner is widened exactly
    dn = to_bf16_bits(rng.standard_normal((vocab, d)).astype(np.float32))
    r2 = oracle.densify([idx], [bits], d, vocab, dn, value_dtype="bf16", out_dtype="bf16")
    dn64 = torch.from_numpy(dn.view(np.int16)).view(torch.bfloat16).double().numpy()
    np.testing.assert_allclose(r2.acc, ref.numpy() + dn64, rtol=0, atol=1e-12)


def test_int32_and_int64_indices_agree():
    indices, values, d, vocab, dense = _small_case(12)
    a = oracle.densify(indices, values, d, vocab, dense)
    b = oracle.densify([i.astype(np.int32) for i in indices], values, d, vocab, dense)
    assert np.array_equal(a.acc, b.acc) and np.array_equal(a.counts, b.counts)


def test_concat_equals_physical_concatenation():
    w = make_workload("r64", scale=0.002)
    a = oracle.densify(w.indices, w.values, w.d, w.vocab, w.dense_in)
    ci, cv = w.concatenated()
    b = oracle.densify([ci], [cv], w.d, w.vocab, w.dense_in)
    assert np.array_equal(a.acc, b.acc) and np.array_equal(a.cnt, b.cnt)


# --------------------------------------------------------------------------
# planted mistakes (all on the CPU, in NumPy): the battery must reject each
# --------------------------------------------------------------------------
def _dense_or_zero(dense, vocab, d):
    return dense.astype(np.float64).copy() if dense is not None else np.zeros((vocab, d))


def _valid(ix, vocab):
    return (ix >= 0) & (ix < vocab)


def correct_numpy(indices, values, d, vocab, dense):
    out = _dense_or_zero(dense, vocab, d)
    for ix, va in zip(indices, values):
        m = _valid(ix, vocab)
        np.add.at(out, ix[m], va[m].astype(np.float64))
    return out


def mutant_last_write_wins(indices, values, d, vocab, dense):
    out = _dense_or_zero(dense, vocab, d)
    base = out.copy()
    for ix, va in zip(indices, values):
        m = _valid(ix, vocab)
        out[ix[m]] = base[ix[m]] + va[m].astype(np.float64)
    return out


def mutant_drops_dense(indices, values, d, vocab, dense):
    return correct_numpy(indices, values, d, vocab, None)


def mutant_row_off_by_one(indices, values, d, vocab, dense):
    return correct_numpy([np.where(ix + 1 < vocab, ix + 1, ix) for ix in indices], values, d, vocab, dense)


def mutant_transposed_values(indices, values, d, vocab, dense):
    tv = [np.ascontiguousarray(va.T).reshape(va.shape) for va in values]
    return correct_numpy(indices, tv, d, vocab, dense)


def mutant_forgets_later_slices(indices, values, d, vocab, dense):
    return correct_numpy(indices[:1], values[:1], d, vocab, dense)


def mutant_clamps_bad_rows(indices, values, d, vocab, dense):
    return correct_numpy([np.clip(ix, 0, vocab - 1) for ix in indices], values, d, vocab, dense)


def mutant_dense_added_per_occurrence(indices, values, d, vocab, dense):
    out = np.zeros((vocab, d))
    dn = _dense_or_zero(dense, vocab, d)
    touched = np.zeros(vocab, bool)
    for ix, va in zip(indices, values):
        m = _valid(ix, vocab)
        np.add.at(out, ix[m], va[m].astype(np.float64) + dn[ix[m]])
        touched[ix[m]] = True
    out[~touched] = dn[~touched]
    return out


def mutant_fp32_accumulate_sign_flip_on_negative_zero_row(indices, values, d, vocab, dense):
    # subtracts instead of adding for row 0 only
    out = correct_numpy(indices, values, d, vocab, dense)
    dn = _dense_or_zero(dense, vocab, d)
    out[0] = 2 * dn[0] - out[0]
    return out


MUTANTS = [mutant_last_write_wins, mutant_drops_dense, mutant_row_off_by_one, mutant_transposed_values,
           mutant_forgets_later_slices, mutant_clamps_bad_rows, mutant_dense_added_per_occurrence,
           mutant_fp32_accumulate_sign_flip_on_negative_zero_row]


def test_battery_accepts_a_correct_numpy_version():
    for pin in BATTERY:
        pin(correct_numpy)


@pytest.mark.parametrize("mutant", MUTANTS, ids=lambda m: m.__name__)
def test_battery_rejects_planted_mistakes(mutant):
    failed = []
    for pin in BATTERY:
        try:
            pin(mutant)
        except AssertionError:
            failed.append(pin.__name__)
    assert failed, "no pin notices %s" % mutant.__name__
