"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_04035_b200 as dst
from paper_1905_04035_b200.workloads import Workload, make_workload, to_bf16_bits

from gpu_helpers import TORCH_DT, assert_parity, oracle_of, raw_bits, run_library, to_device, to_numpy_f64, tolerance

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


@pytest.mark.parametrize("vocab,ns", [
    (33707, [9000] * 70),                     # odd vocabulary; more slices than one validation launch describes
    (65536, [20000, 0, 8192, 8193, 40000]),   # largest vocabulary counted in shared memory; slices of several CTAs
    (65537, [70000]),                         # one more row: counts come from the sorted keys instead
    (513, [100000]),                          # every row heavy; two digits, the second nearly empty
])
def test_row_counts_taken_while_validating(vocab, ns):
    """Large inputs over a small vocabulary: the validation kernel counts the rows and the scan rides in the first
    radix pass.  Runs of one row longer than a warp (the one-add-per-warp case), with out-of-range and negative
    indices inside them, and rows at both ends of the vocabulary."""
    def idx(rng, k):
        ix = rng.integers(0, vocab, size=k)
        run = np.arange(k) % 1000 < 200            # 200 consecutive entries of one row in every 1000
        ix[run] = (np.arange(k)[run] // 1000) % 2 * (vocab - 1)
        ix[5::997] = vocab + 3
        ix[6::1499] = -1
        return ix
    w = _custom(vocab, 64, ns, idx_fn=idx, integer=True)
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
# the two index paths; small inputs, where the row kernel copies the unnamed rows beside the index cluster
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n,vocab,R", [
    (65535, 65536, 1),      # largest input of the one-kernel index path
    (65536, 65536, 1),      # one more row: general path
    (3000, 65537, 1),       # one more vocabulary row: general path
    (3000, 65536, 64),      # most slices the one-kernel path takes
    (3000, 65536, 65),      # one more slice: general path
    (3000, 1000, 3),        # small, but more rows than vocabulary: general path
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
def test_small_inputs_unnamed_rows_are_copied(d, with_dense, in_place):
    # few rows against the vocabulary: most rows of out are plain copies of dense_in (or zeros)
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


def test_small_inputs_bf16_and_out_of_range():
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


# ---------------------------------------------------------------------------
# branches and guarantees that the named workloads do not reach
# ---------------------------------------------------------------------------
def test_more_heavy_rows_than_the_shared_memory_table_holds():
    # every one of 3000 rows is heavy (about 67 entries each against chunks of 32): the row-reduction kernel
    # keeps the first chunk ids of at most 1024 heavy rows in shared memory and searches the global table beyond
    vocab, d, n = 3000, 64, 200_000
    w = _custom(vocab, d, [n], std=0.05)
    run = run_library(w)
    orc = assert_parity(w, run)
    assert orc.n_unique == vocab and int(orc.counts.min()) > 32


def test_nan_inf_and_negative_zero_propagate():
    # IEEE propagation: a NaN or an infinity in a value row or in dense_in reaches exactly the output elements it
    # belongs to; zeros compare numerically (the accumulators start at +0, so a sum of negative zeros only is +0
    # where the oracle, which starts from dense_in, has -0), and an unnamed row keeps its dense_in bits, -0 included
    vocab, d = 500, 64
    w = _custom(vocab, d, [3000], idx_fn=lambda rng, n: rng.integers(0, 300, size=n))     # rows 300.. are unnamed
    v, dn, ix = w.values[0], w.dense_in, w.indices[0]
    v[10, 3] = np.nan; v[11, 4] = np.inf; v[12, 5] = -np.inf
    ix[20] = ix[11]; v[20, 4] = -np.inf                              # +inf and -inf meet in one output element: NaN
    dn[7, 9] = np.nan; dn[450, 1] = np.inf; dn[451, 2] = -0.0        # rows 450, 451 are unnamed
    rows0 = np.flatnonzero(ix == 42)
    v[rows0, 17] = -0.0; dn[42, 17] = -0.0                           # only negative zeros meet
    run = run_library(w)
    orc = oracle_of(w)
    got = to_numpy_f64(run.out)
    want = orc.acc
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isposinf(got), np.isposinf(want)) and np.array_equal(np.isneginf(got), np.isneginf(want))
    fin = np.isfinite(want)
    assert np.all(np.abs(got[fin] - want[fin]) <= 1e-5 * orc.mag[fin] + 1e-7)
    assert np.isnan(got[ix[10], 3]) and np.isnan(got[ix[11], 4]) and np.isneginf(got[ix[12], 5]) and np.isnan(got[7, 9])
    assert np.isposinf(got[450, 1])
    bits = raw_bits(run.out)
    assert bits[451, 2] == 0x80000000 and got[42, 17] == 0.0 and want[42, 17] == 0.0
    assert run.result["status"] == 0


@pytest.mark.parametrize("name", ["tiny", "custom_general", "custom_bf16"])
def test_nothing_is_written_beyond_the_buffers(name):
    # guard words behind every buffer the library writes: out, unique_rows, counts, the result block and the workspace
    if name == "tiny":
        w = make_workload("tiny")
    elif name == "custom_general":
        hot = lambda rng, n: np.where(rng.random(n) < 0.5, 3, rng.integers(0, 2000, size=n))
        w = _custom(2000, 136, [70000, 0, 9000], idx_fn=hot)          # general index path, heavy rows
    else:
        w = _custom(70000, 64, [5000], value_dtype="bf16", out_dtype="bf16", index_dtype="i32")   # three radix passes
    from gpu_helpers import TORCH_DT
    idt, vdt, odt = TORCH_DT[w.index_dtype], TORCH_DT[w.value_dtype], TORCH_DT[w.out_dtype]
    guard = 64                                                       # guard elements of each buffer's own type
    def guarded(n, dtype, fill):
        t = torch.full((n + guard,), fill, dtype=dtype, device="cuda")
        return t, t[:n]
    cap = max(1, min(w.n_rows_total, w.vocab))
    out_all, out = guarded(w.vocab * w.d, odt, 7.0)
    uniq_all, uniq = guarded(cap, idt, -3)
    cnt_all, cnt = guarded(cap, torch.int32, -3)
    res_all, res = guarded(6, torch.int32, -3)
    ws_bytes = dst.dst_workspace_bytes(w.n_rows_total, len(w.indices), w.d, w.vocab, idt, vdt, odt)
    ws_all = torch.full((ws_bytes + 4096,), 0xA5, dtype=torch.uint8, device="cuda")
    slices = [(to_device(i, w.index_dtype), to_device(v, w.value_dtype)) for i, v in zip(w.indices, w.values)]
    dense = to_device(w.dense_in, w.out_dtype) if w.dense_in is not None else None
    dst.dst_densify_concat(slices, w.d, w.vocab, dense, out.view(w.vocab, w.d), ws_all[:ws_bytes], uniq, cnt, res)
    torch.cuda.synchronize()
    assert bool((out_all[w.vocab * w.d:] == 7.0).all())
    assert bool((uniq_all[cap:] == -3).all()) and bool((cnt_all[cap:] == -3).all()) and bool((res_all[6:] == -3).all())
    assert bool((ws_all[ws_bytes:] == 0xA5).all())
    orc = oracle_of(w)
    nu = int(res[1])
    assert nu == orc.n_unique and np.array_equal(uniq[:nu].cpu().numpy(), orc.unique_rows)
    assert bool((uniq[nu:] == -3).all()) and bool((cnt[nu:] == -3).all())      # nor beyond the entries that exist
    got = to_numpy_f64(out.view(w.vocab, w.d))
    from gpu_helpers import tolerance
    assert np.all(np.abs(got - orc.acc) <= tolerance(w, orc))


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    # the give-up path of the bounded device-side waits: nothing arrives on the barrier, the limit is 100,000 cycles
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    res = torch.zeros(6, dtype=torch.int32, device="cuda")
    dst.dst_selftest_wait_limit(100_000, ws, res)
    torch.cuda.synchronize()                                          # returns: the wait ended by itself
    assert int(res[0]) == 5 and dst.dst_status_string(5).startswith("a bounded device-side wait gave up")
    assert int(ws[:4].view(torch.int32)[0]) == 5                      # the status word of the workspace header
    with pytest.raises(dst.DstError):
        dst.dst_selftest_wait_limit(0, ws, res)
    w = make_workload("tiny")                                         # and the next call is an ordinary one
    assert_parity(w, run_library(w))


def test_nvtx_ranges_can_be_switched_on_and_change_nothing():
    w = make_workload("tiny")
    plain = run_library(w)
    dst.dst_profile_ranges(True)
    try:
        ranged = run_library(w)
    finally:
        dst.dst_profile_ranges(False)
    assert np.array_equal(raw_bits(plain.out), raw_bits(ranged.out))


# ---------------------------------------------------------------------------
# nothing may depend on what the workspace held before the call
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("name,scale", [("tiny", 1.0), ("base", 1.0), ("r64", 0.05), ("sweep_zipf", 0.02)])
def test_a_dirty_workspace_changes_nothing(name, scale):
    """The workspace is filled with 0xFF, then with 0x01 (every flag and counter of a header 'set'), and is also
    used as an earlier call left it: all four outputs are bit-identical and within tolerance of the oracle."""
    w = make_workload(name, scale=scale)
    idt, vdt, odt = TORCH_DT[w.index_dtype], TORCH_DT[w.value_dtype], TORCH_DT[w.out_dtype]
    slices = [(to_device(i, w.index_dtype), to_device(v, w.value_dtype)) for i, v in zip(w.indices, w.values)]
    dense = to_device(w.dense_in, w.out_dtype) if w.dense_in is not None else None
    eng = dst.Densifier(w.n_rows_total, len(slices), w.d, w.vocab, index_dtype=idt, value_dtype=vdt, out_dtype=odt)
    outs = []
    for fill in (0xFF, None, 0x01, None):
        if fill is not None:
            eng.workspace.fill_(fill)
        out = torch.full((w.vocab, w.d), float("nan"), dtype=odt, device="cuda")
        eng(slices, dense, out)
        torch.cuda.synchronize()
        assert eng.read_result()["status"] == 0
        outs.append(out)
    for o in outs[1:]:
        assert np.array_equal(raw_bits(o), raw_bits(outs[0]))
    orc = oracle_of(w)
    assert np.all(np.abs(to_numpy_f64(outs[0]) - orc.acc) <= tolerance(w, orc))
