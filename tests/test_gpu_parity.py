"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_04035_b200 as dst
from paper_1905_04035_b200.workloads import Workload, make_workload, to_bf16_bits

from gpu_helpers import assert_parity, oracle_of, raw_bits, run_library, to_device, to_numpy_f64

pytestmark = pytest.mark.gpu


def _custom(vocab, d, ns, *, seed=0, index_dtype="i64", value_dtype="f32", out_dtype="f32", with_dense=True,
            integer=False, idx_fn=None, std=1.0):
    rng = np.random.default_rng(seed)
    idt = np.int64 if index_dtype == "i64" else np.int32
    indices, values = [], []
    for n in ns:
        ix = idx_fn(rng, n) if idx_fn else rng.integers(0, max(vocab, 1), size=n)
        indices.append(np.asarray(ix).astype(idt))
        if integer:
            v = rng.integers(-8, 9, size=(n, d)).astype(np.float32)
        else:
            v = (rng.standard_normal((n, d)) * std).astype(np.float32)
        values.append(to_bf16_bits(v) if value_dtype == "bf16" else v)
    dense = None
    if with_dense:
        dn = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32) if integer else \
            (rng.standard_normal((vocab, d)) * std).astype(np.float32)
        dense = to_bf16_bits(dn) if out_dtype == "bf16" else dn
    return Workload("custom", vocab, d, indices, values, dense, index_dtype, value_dtype, out_dtype, seed, "custom")


# ---------------------------------------------------------------------------
# the named configurations at full size, in the launch configuration the benchmark times
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "base", "big"])
def test_transformer_configs(name):
    w = make_workload(name)
    orc = assert_parity(w, run_library(w, mode="concat"))
    single = run_library(w, mode="single")
    assert_parity(w, single, orc)


def test_r64_concatenated_slices_full_size():
    w = make_workload("r64")
    assert_parity(w, run_library(w, mode="concat"))


@pytest.mark.parametrize("dist", ["uniform", "zipf", "same"])
def test_sweep_bf16_full_size(dist):
    w = make_workload("sweep_" + dist)
    assert_parity(w, run_library(w, mode="single"))


def test_sweep_bf16_values_fp32_out():
    w = make_workload("sweep_zipf", scale=0.125, out_dtype="f32")
    assert_parity(w, run_library(w, mode="single"))


def test_hot_rows_not_at_low_ids():
    w = make_workload("big", permute_vocab=True)
    assert_parity(w, run_library(w))
    w = make_workload("r64", scale=0.1, permute_vocab=True)
    assert_parity(w, run_library(w))


# ---------------------------------------------------------------------------
# determinism and the concat == concatenation contract
# ---------------------------------------------------------------------------
def test_runs_are_bit_identical_and_concat_equals_concatenation():
    w = make_workload("r64", scale=0.25)
    a = run_library(w, mode="concat")
    b = run_library(w, mode="concat")
    c = run_library(w, mode="single")
    assert np.array_equal(raw_bits(a.out), raw_bits(b.out))
    assert np.array_equal(raw_bits(a.out), raw_bits(c.out))
    assert np.array_equal(a.unique_rows, c.unique_rows) and np.array_equal(a.counts, c.counts)


def test_exact_integer_data_is_bit_exact():
    # small integers: every summation order is exact, so GPU == oracle bit for bit
    hot = lambda rng, n: np.where(rng.random(n) < 0.5, 3, rng.integers(0, 500, size=n))
    w = _custom(500, 256, [5000, 0, 3000], integer=True, idx_fn=hot)
    run = run_library(w)
    orc = assert_parity(w, run)
    assert np.array_equal(to_numpy_f64(run.out), orc.acc)
    assert orc.max_segment > 2000   # exercises chunked heavy rows and the combine tree


# ---------------------------------------------------------------------------
# degenerate and edge cases
# ---------------------------------------------------------------------------
def test_all_same_index_ones():
    n, d, vocab = 1 << 16, 128, 300
    w = _custom(vocab, d, [n], with_dense=False, idx_fn=lambda rng, k: np.full(k, 77))
    w.values[0][:] = 1.0
    run = run_library(w)
    out = to_numpy_f64(run.out)
    assert np.all(out[77] == n) and not out[np.arange(vocab) != 77].any()
    assert run.result["n_unique"] == 1 and run.counts.tolist() == [n] and run.result["max_segment"] == n


def test_all_unique_rows_single_add_is_exact():
    vocab, d = 4096, 512
    w = _custom(vocab, d, [3000], idx_fn=lambda rng, k: rng.permutation(vocab)[:k])
    run = run_library(w)
    assert_parity(w, run)
    want = w.dense_in.copy()
    want[w.indices[0]] = w.values[0] + w.dense_in[w.indices[0]]      # one IEEE fp32 add per element
    assert np.array_equal(raw_bits(run.out), want.view(np.uint32))
    assert np.all(run.counts == 1)


def test_empty_inputs():
    w = _custom(1000, 64, [0])
    assert_parity(w, run_library(w, mode="single"))
    w = _custom(1000, 64, [])
    assert_parity(w, run_library(w, mode="concat"))
    w = _custom(1000, 64, [], with_dense=False)
    assert_parity(w, run_library(w, mode="concat"))
    w = _custom(777, 64, [0, 300, 0, 0, 41, 0])
    orc = assert_parity(w, run_library(w, mode="concat"))
    w2 = Workload("c", w.vocab, w.d, [w.indices[1], w.indices[4]], [w.values[1], w.values[4]], w.dense_in,
                  "i64", "f32", "f32", 0, "")
    assert np.array_equal(raw_bits(run_library(w2).out), raw_bits(run_library(w).out))


def test_out_of_range_indices_are_skipped_and_counted():
    def idx(rng, n):
        ix = rng.integers(0, 900, size=n)
        ix[::7] = -1 - rng.integers(0, 5, size=ix[::7].shape[0])
        ix[3::11] = 900 + rng.integers(0, 2 ** 33, size=ix[3::11].shape[0])
        return ix
    w = _custom(900, 64, [4000, 100], idx_fn=idx)
    run = run_library(w)
    orc = assert_parity(w, run)
    assert orc.n_out_of_range > 500 and run.result["status"] == 4
    w = _custom(900, 64, [500], index_dtype="i32",
                idx_fn=lambda rng, n: np.where(rng.random(n) < 0.3, -5, rng.integers(0, 900, size=n)))
    assert_parity(w, run_library(w))
    w = _custom(50, 64, [64], idx_fn=lambda rng, n: np.full(n, 50))     # every row invalid
    assert_parity(w, run_library(w))


def test_in_place_accumulate():
    w = make_workload("base", scale=0.5)
    run = run_library(w, in_place=True)
    orc = oracle_of(w)
    got = to_numpy_f64(run.out)
    assert np.all(np.abs(got - orc.acc) <= 1e-5 * orc.mag + 1e-7)
    assert np.array_equal(raw_bits(run.out), raw_bits(run_library(w).out))


@pytest.mark.parametrize("vocab,passes", [(200, 1), (256, 1), (257, 2), (70000, 3), (1 << 17, 3)])
def test_radix_pass_counts(vocab, passes):
    hot = lambda rng, n: np.where(rng.random(n) < 0.3, vocab - 1, rng.integers(0, vocab, size=n))
    w = _custom(vocab, 64, [9000, 5000], idx_fn=hot, index_dtype="i32")
    assert_parity(w, run_library(w))


@pytest.mark.parametrize("d", [8, 64, 136, 520, 1024, 2056, 4096])
def test_row_widths(d):
    w = _custom(300, d, [2500], idx_fn=lambda rng, n: np.minimum(rng.zipf(1.3, size=n) - 1, 299))
    assert_parity(w, run_library(w))


@pytest.mark.parametrize("d", [1, 3, 50, 1001])
def test_unaligned_row_widths_take_the_scalar_kernel(d):
    w = _custom(100, d, [700, 0, 30])
    assert_parity(w, run_library(w))
    w = _custom(100, d, [300], value_dtype="bf16", out_dtype="bf16", index_dtype="i32")
    assert_parity(w, run_library(w))


@pytest.mark.parametrize("vt,ot", [("f32", "bf16"), ("bf16", "f32"), ("bf16", "bf16")])
def test_dtype_pairs(vt, ot):
    hot = lambda rng, n: np.where(rng.random(n) < 0.4, 5, rng.integers(0, 2000, size=n))
    w = _custom(2000, 512, [6000, 2000], value_dtype=vt, out_dtype=ot, idx_fn=hot)
    assert_parity(w, run_library(w))
    w = _custom(2000, 512, [6000], value_dtype=vt, out_dtype=ot, idx_fn=hot, with_dense=False)
    assert_parity(w, run_library(w))


# ---------------------------------------------------------------------------
# the two index paths and the pre-filled output of the small-input path
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n,vocab,R", [
    (65535, 65536, 1),      # largest input of the one-kernel index path
    (65536, 65536, 1),      # one more row: general path
    (3000, 65537, 1),       # one more vocabulary row: general path
    (3000, 65536, 64),      # most slices the one-kernel path takes
    (3000, 65536, 65),      # one more slice: general path
    (3000, 1000, 3),        # small path, more rows than vocabulary: nothing is pre-filled
])
def test_index_path_boundaries(n, vocab, R):
    ns = [n // R + (1 if r < n % R else 0) for r in range(R)]
    hot = lambda rng, k: np.where(rng.random(k) < 0.3, vocab - 1, rng.integers(0, vocab, size=k))
    w = _custom(vocab, 64, ns, idx_fn=hot)
    a = run_library(w, mode="concat")
    assert_parity(w, a)
    assert np.array_equal(raw_bits(a.out), raw_bits(run_library(w, mode="single").out))


@pytest.mark.parametrize("d,with_dense,in_place", [(64, True, False), (2056, True, False), (512, False, False),
                                                   (512, True, True), (4096, True, True)])
def test_prefilled_output_small_inputs(d, with_dense, in_place):
    # few rows against the vocabulary: most of out is written by the index kernel's extra clusters
    vocab = 40000 if d <= 512 else 6000
    hot = lambda rng, k: np.where(rng.random(k) < 0.4, 7, rng.integers(0, vocab, size=k))
    w = _custom(vocab, d, [1500, 0, 700], idx_fn=hot, with_dense=with_dense, std=0.5)
    run = run_library(w, in_place=in_place)
    if in_place:
        orc = oracle_of(w)
        assert np.all(np.abs(to_numpy_f64(run.out) - orc.acc) <= 1e-5 * orc.mag + 1e-7)
        assert np.array_equal(raw_bits(run.out), raw_bits(run_library(w).out))
    else:
        assert_parity(w, run)


def test_prefilled_output_bf16_and_out_of_range():
    vocab = 50000
    def idx(rng, k):
        ix = rng.integers(0, vocab, size=k)
        ix[::9] = vocab + rng.integers(0, 100, size=ix[::9].shape[0])
        return ix
    w = _custom(vocab, 256, [4000], idx_fn=idx, value_dtype="bf16", out_dtype="bf16", index_dtype="i32")
    assert_parity(w, run_library(w))
    w = _custom(vocab, 256, [4000], idx_fn=idx, value_dtype="bf16", out_dtype="f32", with_dense=False)
    assert_parity(w, run_library(w))


@pytest.mark.parametrize("name,scale", [("big", 1.0), ("r64", 0.1)])
def test_cuda_graph_replay_matches_eager_calls(name, scale):
    # the benchmark times CUDA-graph replays of one library call: same bits as the eager call, replay after replay
    w = make_workload(name, scale=scale)
    eager = run_library(w, mode="concat")
    assert_parity(w, eager)
    slices = [(to_device(i, w.index_dtype), to_device(v, w.value_dtype)) for i, v in zip(w.indices, w.values)]
    dense = to_device(w.dense_in, w.out_dtype)
    out = torch.full((w.vocab, w.d), float("nan"), device="cuda")
    eng = dst.Densifier(w.n_rows_total, w.R, w.d, w.vocab)
    eng(slices, dense, out)                        # first call outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        eng(slices, dense, out)
    for _ in range(3):
        out.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(raw_bits(out), raw_bits(eager.out))
        assert eng.read_result()["status"] == 0 and eng.read_result()["n_unique"] == eager.result["n_unique"]


def test_many_slices_use_several_histogram_launches():
    ns = [int(x) for x in np.random.default_rng(1).integers(0, 200, size=150)]
    w = _custom(1500, 128, ns)
    a = run_library(w, mode="concat")
    assert_parity(w, a)
    assert np.array_equal(raw_bits(a.out), raw_bits(run_library(w, mode="single").out))


def test_workspace_is_reusable_across_shapes():
    w1 = make_workload("tiny")
    w2 = _custom(640, 64, [100])
    eng = dst.Densifier(2048, 4, 64, 1000)
    from gpu_helpers import to_device
    for w in (w1, w2, w1):
        out = torch.empty(w.vocab, w.d, device="cuda")
        dst.dst_densify(to_device(w.indices[0], "i64"), to_device(w.values[0], "f32"), w.d, w.vocab,
                        to_device(w.dense_in, "f32"), out, eng.workspace, None, None, eng.result)
        torch.cuda.synchronize()
        orc = oracle_of(w)
        assert np.all(np.abs(to_numpy_f64(out) - orc.acc) <= 1e-5 * orc.mag + 1e-7)


def test_host_entry_point_matches_device_entry_point():
    w = make_workload("base", scale=0.25)
    slices = [(torch.from_numpy(i).pin_memory(), torch.from_numpy(v).pin_memory()) for i, v in zip(w.indices, w.values)]
    dense = torch.from_numpy(w.dense_in).pin_memory()
    out = torch.empty(w.vocab, w.d).pin_memory()
    res = torch.zeros(6, dtype=torch.int32).pin_memory()
    staging = torch.empty(dst.dst_host_staging_bytes(w.n_rows_total, w.d, w.vocab), dtype=torch.uint8, device="cuda")
    ws = torch.empty(dst.dst_workspace_bytes(w.n_rows_total, 1, w.d, w.vocab), dtype=torch.uint8, device="cuda")
    dst.dst_densify_concat_host(slices, w.d, w.vocab, dense, out, staging, ws, res)
    torch.cuda.synchronize()
    ref = run_library(w, mode="single")
    assert np.array_equal(out.numpy().view(np.uint32), raw_bits(ref.out))
    assert res[0].item() == 0 and res[1].item() == ref.result["n_unique"]


def test_bytes_report_matches_oracle():
    for ns, d, vocab, it, vt, ot in (([10000] * 64, 1024, 33708, "i64", "f32", "f32"),
                                     ([1048576], 1024, 65536, "i32", "bf16", "bf16"), ([], 8, 10, "i64", "f32", "f32")):
        from gpu_helpers import TORCH_DT
        got = dst.dst_bytes_report(ns, d, vocab, TORCH_DT[it], TORCH_DT[vt], TORCH_DT[ot])
        want = oracle.bytes_report(ns, d, vocab, index_dtype=it, value_dtype=vt, out_dtype=ot)
        for k, v in want.items():
            assert got[k] == v or abs(got[k] - v) <= 1e-12 * abs(v), k
