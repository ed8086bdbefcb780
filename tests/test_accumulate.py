"""The accumulation dispatcher (Algorithms 1 and 2, Listing 1).

CPU part: the host-only plan against the oracle's branch and output size.
GPU part: ``dst_accumulate`` through the C ABI against ``oracle.accumulate_oracle`` -- gathered
IndexedSlices bit for bit, dense sums within the tolerance of the densify tests.
"""
import numpy as np
import pytest
import torch

import paper_1905_04035_b200 as dst
from oracle import accumulate_oracle as ao
from paper_1905_04035_b200.workloads import to_bf16_bits

STRATEGIES = {dst.DST_ACC_STOCK: ao.STOCK, dst.DST_ACC_PROPOSED: ao.PROPOSED, dst.DST_ACC_SPARSE_AS_DENSE: ao.SPARSE_AS_DENSE}
# composition of the list: 'D' a dense gradient, a number an IndexedSlices gradient of that many rows
LISTS = [[], ["D"], [40], ["D", "D"], ["D", 300, 17], [300, "D", 0, 1200], [64, 2000], ["D", "D", "D", 900],
         ["D"] * 9 + [500], ["D"] * 17]


def make_list(spec, vocab, d, seed, index_dtype=np.int64, integers=False):
    rng = np.random.default_rng(seed)
    grads = []
    for s in spec:
        if s == "D":
            v = rng.integers(-4, 5, size=(vocab, d)) if integers else rng.normal(0, 0.02, size=(vocab, d))
            grads.append(ao.Grad(v.astype(np.float32)))
        else:
            v = rng.integers(-4, 5, size=(s, d)) if integers else rng.normal(0, 0.02, size=(s, d))
            grads.append(ao.Grad(v.astype(np.float32), rng.integers(0, vocab, size=s).astype(index_dtype)))
    return grads


def as_host_tensors(grads):
    return [torch.from_numpy(g.values) if g.is_dense else (torch.from_numpy(g.indices), torch.from_numpy(g.values))
            for g in grads]


@pytest.mark.parametrize("strategy", sorted(STRATEGIES))
@pytest.mark.parametrize("spec", LISTS, ids=lambda s: "-".join(map(str, s)) or "empty")
def test_plan_matches_oracle_branch(spec, strategy):
    vocab, d = 97, 8
    grads = make_list(spec, vocab, d, 1)
    ref = ao.accumulate(grads, d, vocab, STRATEGIES[strategy])
    plan = dst.dst_accumulate_plan(as_host_tensors(grads), d, vocab, strategy, index_dtype=torch.int64,
                                   value_dtype=torch.float32, out_dtype=torch.float32)
    if ref.grad is None:
        assert plan["branch"] == "empty" and plan["out_kind"] is None
        return
    assert plan["branch"] == ref.branch
    assert plan["out_kind"] == ("dense" if ref.grad.is_dense else "slices")
    rows = vocab if ref.grad.is_dense else ref.grad.indices.shape[0]
    assert plan["out_rows"] == rows
    assert plan["out_bytes"] == rows * d * 4 + (0 if ref.grad.is_dense else rows * 8)
    assert plan["converts"] == (ref.grad.is_dense and any(not g.is_dense for g in grads))


def test_plan_rejects_bad_arguments():
    with pytest.raises(dst.DstError):
        dst.dst_accumulate_plan([torch.zeros(4, 2)], 2, 4, strategy=7)


# ------------------------------------------------------------------------------------------------
def run_gpu(grads, d, vocab, strategy, value_kind="f32", index_dtype=torch.int64):
    dev = "cuda"
    def vals(a, kind):
        if kind == "bf16":
            return torch.from_numpy(to_bf16_bits(a).view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)
    vdt = torch.bfloat16 if value_kind == "bf16" else torch.float32
    tg = [vals(g.values, value_kind) if g.is_dense
          else (torch.from_numpy(g.indices).to(dev).to(index_dtype), vals(g.values, value_kind)) for g in grads]
    plan = dst.dst_accumulate_plan(tg, d, vocab, strategy, index_dtype=index_dtype, value_dtype=vdt, out_dtype=vdt)
    out_dense = torch.full((vocab, d), float("nan"), dtype=vdt, device=dev)
    rows = max(plan["out_rows"], 1)
    out_idx = torch.full((rows,), -7, dtype=index_dtype, device=dev)
    out_val = torch.full((rows, d), float("nan"), dtype=vdt, device=dev)
    ws = torch.empty(max(256, dst.dst_workspace_bytes(plan["n_slice_rows"], plan["n_slices"], d, vocab, index_dtype, vdt, vdt)),
                     dtype=torch.uint8, device=dev)
    result = torch.zeros(8, dtype=torch.int32, device=dev)
    before = dst.dst_kernel_launches()
    got = dst.dst_accumulate(tg, d, vocab, strategy, out_dense=out_dense, out_indices=out_idx, out_values=out_val,
                             workspace=ws, result=result, index_dtype=index_dtype, value_dtype=vdt, out_dtype=vdt)
    torch.cuda.synchronize()
    assert got == plan
    return plan, out_dense, out_idx, out_val, result, dst.dst_kernel_launches() - before


def widen(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.gpu
@pytest.mark.parametrize("strategy", sorted(STRATEGIES))
@pytest.mark.parametrize("spec", LISTS, ids=lambda s: "-".join(map(str, s)) or "empty")
def test_accumulate_matches_oracle_fp32(spec, strategy):
    vocab, d = 1500, 64
    grads = make_list(spec, vocab, d, 11)
    ref = ao.accumulate(grads, d, vocab, STRATEGIES[strategy])
    plan, out_dense, out_idx, out_val, result, launches = run_gpu(grads, d, vocab, strategy)
    if ref.grad is None:
        assert plan["branch"] == "empty" and launches == 0
        assert torch.isnan(out_dense).all()
        return
    assert plan["branch"] == ref.branch
    if ref.grad.is_dense:
        mag = np.zeros((vocab, d))
        for g in grads:
            if g.is_dense:
                mag += np.abs(g.values)
            else:
                np.add.at(mag, g.indices, np.abs(g.values.astype(np.float64)))
        err = np.abs(widen(out_dense) - np.asarray(ref.grad.values, np.float64))
        assert np.all(err <= 1e-5 * mag + 1e-7)
        assert (torch.isnan(out_val)).all()                      # the other kind of output is not touched
        if plan["converts"]:
            assert int(result[0]) == 0
    else:
        n = ref.grad.indices.shape[0]
        assert np.array_equal(out_idx[:n].cpu().numpy(), ref.grad.indices)
        assert np.array_equal(out_val[:n].cpu().numpy(), ref.grad.values)      # copies: bit for bit
        assert torch.isnan(out_dense).all()


@pytest.mark.gpu
@pytest.mark.parametrize("strategy", sorted(STRATEGIES))
def test_accumulate_exact_on_small_integers_and_strategy_independent(strategy):
    """Small-integer data sums exactly in any order: every strategy must give the same gradient, bit for
    bit, once the gathered form is densified (on the CPU, by the oracle)."""
    vocab, d = 700, 24                       # rows of 96 bytes: the 16-byte vector path
    grads = make_list(["D", 900, "D", 5000, 33], vocab, d, 5, integers=True)
    want = ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values
    plan, out_dense, out_idx, out_val, _, _ = run_gpu(grads, d, vocab, strategy)
    if plan["out_kind"] == "dense":
        assert np.array_equal(widen(out_dense), want)
    else:
        n = plan["out_rows"]
        assert n == 2 * vocab + 900 + 5000 + 33
        back = ao.densified(ao.Grad(out_val[:n].cpu().numpy(), out_idx[:n].cpu().numpy()), d, vocab)
        assert np.array_equal(back, want)


@pytest.mark.gpu
def test_accumulate_bf16_int32_and_unaligned_rows():
    vocab, d = 300, 7                        # 14-byte rows: scalar paths
    grads = make_list(["D", "D", 400, 50], vocab, d, 9, index_dtype=np.int32, integers=True)
    want = ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values
    for strategy in (dst.DST_ACC_PROPOSED, dst.DST_ACC_SPARSE_AS_DENSE):
        _, out_dense, _, _, _, _ = run_gpu(grads, d, vocab, strategy, value_kind="bf16", index_dtype=torch.int32)
        assert np.array_equal(widen(out_dense), want)          # integers of this size are exact in bf16
    plan, _, out_idx, out_val, _, _ = run_gpu(grads, d, vocab, dst.DST_ACC_STOCK, value_kind="bf16", index_dtype=torch.int32)
    n = plan["out_rows"]
    assert n == 2 * vocab + 450 and out_idx.dtype == torch.int32
    back = ao.densified(ao.Grad(widen(out_val[:n]).astype(np.float32), out_idx[:n].cpu().numpy()), d, vocab)
    assert np.array_equal(back, want)


@pytest.mark.gpu
def test_accumulate_in_place_and_capacity_check():
    vocab, d = 512, 32
    grads = make_list(["D", 1000], vocab, d, 3, integers=True)
    dev = "cuda"
    dense = torch.from_numpy(grads[0].values).to(dev)
    sl = (torch.from_numpy(grads[1].indices).to(dev), torch.from_numpy(grads[1].values).to(dev))
    ws = torch.empty(dst.dst_workspace_bytes(1000, 1, d, vocab), dtype=torch.uint8, device=dev)
    dst.dst_accumulate([dense, sl], d, vocab, dst.DST_ACC_PROPOSED, out_dense=dense, workspace=ws)   # out is the dense gradient
    torch.cuda.synchronize()
    assert np.array_equal(widen(dense), ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values)
    small_i = torch.empty(10, dtype=torch.int64, device=dev)
    small_v = torch.empty(10, d, device=dev)
    with pytest.raises(dst.DstError):
        dst.dst_accumulate([dense, sl], d, vocab, dst.DST_ACC_STOCK, out_indices=small_i, out_values=small_v)


@pytest.mark.gpu
@pytest.mark.parametrize("spec, alias", [(["D"] * 9 + [500], 8), (["D"] * 17, 16), (["D"] * 17, 3),
                                         (["D"] * 12 + [100, 40], 11), (["D"] * 9, 0)])
def test_accumulate_out_is_a_late_dense_gradient(spec, alias):
    """out_dense may be one of the dense gradients, whatever its place in the list: with more than eight
    dense gradients the sum runs in several passes through out_dense, and the aliased gradient must
    have been read before the first pass lands.  Small integers: exact in any order."""
    vocab, d = 600, 32
    grads = make_list(spec, vocab, d, 21, integers=True)
    want = ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values
    dev = "cuda"
    tg = [torch.from_numpy(g.values).to(dev) if g.is_dense
          else (torch.from_numpy(g.indices).to(dev), torch.from_numpy(g.values).to(dev)) for g in grads]
    n_rows = sum(s for s in spec if s != "D")
    n_sl = sum(1 for s in spec if s != "D")
    ws = torch.empty(max(256, dst.dst_workspace_bytes(n_rows, max(n_sl, 1), d, vocab)), dtype=torch.uint8, device=dev)
    dst.dst_accumulate(tg, d, vocab, dst.DST_ACC_PROPOSED, out_dense=tg[alias], workspace=ws)
    torch.cuda.synchronize()
    assert np.array_equal(widen(tg[alias]), want)
    for k, g in enumerate(grads):                  # every other gradient is untouched
        if g.is_dense and k != alias:
            assert np.array_equal(tg[k].cpu().numpy(), g.values)


@pytest.mark.gpu
def test_accumulate_paper_case_at_full_size():
    """One rank's gradients of the tied weight at the size the benchmark times (vocab 33708, d 1024, two lookups of
    12,800 rows): the proposed strategy is one fused densify; the stock strategy gathers vocab + 25,600 rows."""
    from paper_1905_04035_b200.workloads import make_workload
    w = make_workload("big")
    grads = [ao.Grad(w.dense_in)] + [ao.Grad(v, i) for i, v in zip(w.indices, w.values)]
    ref = ao.accumulate(grads, w.d, w.vocab, ao.PROPOSED)
    plan, out_dense, _, _, result, launches = run_gpu(grads, w.d, w.vocab, dst.DST_ACC_PROPOSED)
    assert plan["branch"] == "convert+reduce" and launches == 2          # index cluster + row reduction, no sum kernel
    mag = np.abs(w.dense_in).astype(np.float64)
    for i, v in zip(w.indices, w.values):
        np.add.at(mag, i, np.abs(v.astype(np.float64)))
    assert np.all(np.abs(widen(out_dense) - ref.grad.values) <= 1e-5 * mag + 1e-7)
    plan, _, out_idx, out_val, _, _ = run_gpu(grads, w.d, w.vocab, dst.DST_ACC_STOCK)
    assert plan["branch"] == "gather" and plan["out_rows"] == w.vocab + w.n_rows_total
    assert plan["out_bytes"] == (w.vocab + w.n_rows_total) * (w.d * 4 + 8)
    st = ao.accumulate(grads, w.d, w.vocab, ao.STOCK).grad
    assert np.array_equal(out_idx.cpu().numpy(), st.indices) and np.array_equal(out_val.cpu().numpy(), st.values)
