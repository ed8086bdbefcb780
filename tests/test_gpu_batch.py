"""``dst_densify_batch`` through the C ABI: R ranks x (dense tensor, IndexedSlices) accumulated in one pass,
against ``oracle.accumulate_oracle`` (the proposed rule: convert everything and sum)."""
import numpy as np
import pytest
import torch

import paper_1905_04035_b200 as dst
from oracle import accumulate_oracle as ao

pytestmark = pytest.mark.gpu


def make_ranks(R, vocab, d, rows, seed, integers=False, dense_every=1):
    rng = np.random.default_rng(seed)
    ranks = []
    for r in range(R):
        if integers:
            dense = rng.integers(-4, 5, size=(vocab, d)).astype(np.float32)
        else:
            dense = rng.normal(0, 0.02, size=(vocab, d)).astype(np.float32)
        sl = []
        for n in rows:
            idx = np.minimum(rng.zipf(1.3, size=n) - 1, vocab - 1).astype(np.int64)
            val = (rng.integers(-4, 5, size=(n, d)) if integers else rng.normal(0, 0.02, size=(n, d))).astype(np.float32)
            sl.append((idx, val))
        ranks.append((dense if r % dense_every == 0 else None, sl))
    return ranks


def reference(ranks, d, vocab):
    grads, mag = [], np.zeros((vocab, d))
    for dense, sl in ranks:
        if dense is not None:
            grads.append(ao.Grad(dense)); mag += np.abs(dense)
        for idx, val in sl:
            grads.append(ao.Grad(val, idx)); np.add.at(mag, idx, np.abs(val.astype(np.float64)))
    return ao.accumulate(grads, d, vocab, ao.PROPOSED).grad.values, mag


def run(ranks, d, vocab, alias=None):
    dev = [(None if dn is None else torch.from_numpy(dn).cuda(),
            [(torch.from_numpy(i).cuda(), torch.from_numpy(v).cuda()) for i, v in sl]) for dn, sl in ranks]
    n = sum(i.shape[0] for _, sl in ranks for i, _ in sl)
    n_sl = sum(len(sl) for _, sl in ranks)
    out = dev[alias][0] if alias is not None else torch.full((vocab, d), float("nan"), device="cuda")
    ws = torch.empty(max(256, dst.dst_workspace_bytes(n, max(n_sl, 1), d, vocab)), dtype=torch.uint8, device="cuda")
    res = torch.zeros(6, dtype=torch.int32, device="cuda")
    dst.dst_densify_batch(dev, d, vocab, out, ws, result=res)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64), res.cpu().numpy(), dev


@pytest.mark.parametrize("R", [2, 8, 64])
def test_ranks_in_one_pass_match_the_oracle(R):
    vocab, d = 3000, 64
    ranks = make_ranks(R, vocab, d, [300, 200], R)
    want, mag = reference(ranks, d, vocab)
    got, res, _ = run(ranks, d, vocab)
    assert not np.isnan(got).any() and int(res[0]) == 0
    assert np.all(np.abs(got - want) <= 1e-5 * mag + 1e-7)


@pytest.mark.parametrize("vocab,d,rows,R,alias", [(900, 64, [4000, 3000], 5, None), (70000, 32, [9000], 3, 1),
                                                  (400, 1024, [20000], 4, 0), (2000, 7, [500], 3, None)])
def test_exact_on_small_integers_all_paths_and_in_place(vocab, d, rows, R, alias):
    # small integers: every order exact.  General index path, heavy rows with combine trees (dense rows at the
    # root), rows that are not 16-byte multiples (scalar kernel), and `out` being one of the dense tensors
    ranks = make_ranks(R, vocab, d, rows, vocab + R, integers=True, dense_every=1 if alias is not None else 2)
    want, _ = reference(ranks, d, vocab)
    got, res, dev = run(ranks, d, vocab, alias=alias)
    assert np.array_equal(got, want) and int(res[0]) == 0
    for r, (dn, _) in enumerate(ranks):                 # inputs other than the aliased one are untouched
        if dn is not None and r != alias:
            assert np.array_equal(dev[r][0].cpu().numpy(), dn)


def test_more_dense_tensors_than_one_pass_takes_is_refused():
    vocab, d = 64, 8
    ranks = [(np.zeros((vocab, d), np.float32), []) for _ in range(65)]
    with pytest.raises(dst.DstError) as e:
        run(ranks, d, vocab)
    assert e.value.status == 2
