"""``dst_densify_apply`` through the C ABI against ``oracle.optimizer_oracle``: momentum SGD and Adam fused into
the densify pass, fp32 and bf16 (loss-scaled) gradients, on both index paths, with heavy rows, several slices, no
dense partner, rows that are not 16-byte multiples and out-of-range indices.

Tolerances (fp32 arithmetic on the device, fp64 in the oracle).  With eg = 1.1e-5 * grad_mag the bound on the
gradient's error (the densify bound of the other tests plus the scaling's rounding) and u = 2^-23:
  momentum  |b' - b'*| <= eg + 2u (mu |b| + |g|)                     |w' - w'*| <= |lr| * that + 2u (|w| + |lr b'|)
  Adam      |m' - m'*| <= (1 - beta1) eg + 3u (beta1 |m| + (1 - beta1) |g|)
            |v' - v'*| <= (1 - beta2) (2 |g| eg + eg^2) + 4u v'
            step = mhat / (sqrt(vhat) + eps):  first-order propagation of the two, with |sqrt a - sqrt b| <=
            min(|a - b| / (2 sqrt a), sqrt |a - b|), plus 8u |step|;   |w' - w'*| <= |lr| * that + 2u (|w| + |lr step|)
Each bound is doubled in the checks and gets 1e-7 (weight, momentum buffer) or 1e-12 (second moment) of slack.
"""
import dataclasses

import numpy as np
import pytest
import torch

import paper_1905_04035_b200 as dst
from oracle import optimizer_oracle as oo
from paper_1905_04035_b200.workloads import make_workload, to_bf16_bits

pytestmark = pytest.mark.gpu
U = 2.0 ** -23
KIND = {oo.SGD: dst.DST_OPT_SGD, oo.MOMENTUM: dst.DST_OPT_MOMENTUM, oo.ADAM: dst.DST_OPT_ADAM}


def zipf_indices(rng, n, vocab, s=1.1, dtype=np.int64):
    p = 1.0 / np.arange(1, vocab + 1) ** s
    cdf = np.cumsum(p / p.sum())
    return np.minimum(np.searchsorted(cdf, rng.random(n)), vocab - 1).astype(dtype)


def dev_tensor(a, kind="f32"):
    if kind == "bf16":
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def run(indices, values, d, vocab, dense, weight, hyper, state1, state2, grad="f32"):
    slices = [(torch.from_numpy(i).cuda(), dev_tensor(v, grad)) for i, v in zip(indices, values)]
    n = sum(i.shape[0] for i in indices)
    idt = slices[0][0].dtype if slices else torch.int64
    gdt = torch.bfloat16 if grad == "bf16" else torch.float32
    w = torch.from_numpy(weight.copy()).cuda()
    s1 = torch.from_numpy(state1.copy()).cuda() if state1 is not None else None
    s2 = torch.from_numpy(state2.copy()).cuda() if state2 is not None else None
    dn = dev_tensor(dense, grad) if dense is not None else None
    ws = torch.empty(max(256, dst.dst_workspace_bytes(n, len(slices), d, vocab, idt, gdt, gdt)), dtype=torch.uint8, device="cuda")
    result = torch.zeros(8, dtype=torch.int32, device="cuda")
    dst.dst_densify_apply(slices, d, vocab, dn, w, ws, kind=KIND[hyper.kind], lr=hyper.lr, momentum=hyper.momentum,
                          beta1=hyper.beta1, beta2=hyper.beta2, eps=hyper.eps, step=hyper.step,
                          grad_scale=hyper.grad_scale, state1=s1, state2=s2, result=result, index_dtype=idt, grad_dtype=gdt)
    torch.cuda.synchronize()
    f64 = lambda t: None if t is None else t.cpu().numpy().astype(np.float64)
    return f64(w), f64(s1), f64(s2), result.cpu().numpy()


def check(indices, values, d, vocab, dense, weight, hyper, state1=None, state2=None, grad="f32", exact=False):
    got_w, got_s1, got_s2, result = run(indices, values, d, vocab, dense, weight, hyper, state1, state2, grad)
    ref = oo.apply_step(indices, values, d, vocab, dense, weight, hyper, state1, state2, value_dtype=grad)
    if exact:
        assert np.array_equal(got_w, ref.weight)
        if ref.state1 is not None:
            assert np.array_equal(got_s1, ref.state1)
        if ref.state2 is not None:
            assert np.array_equal(got_s2, ref.state2)
        return ref, result
    lr = abs(hyper.lr)
    w = np.abs(weight.astype(np.float64))
    g = np.abs(ref.grad)
    eg = 1.1e-5 * ref.grad_mag
    if hyper.kind == oo.SGD:
        tol_w = lr * eg + 2 * U * (w + lr * g)
    elif hyper.kind == oo.MOMENTUM:
        tol_b = eg + 2 * U * (abs(hyper.momentum) * np.abs(state1) + g)
        assert np.all(np.abs(got_s1 - ref.state1) <= 2 * tol_b + 1e-7)
        tol_w = lr * tol_b + 2 * U * (w + lr * np.abs(ref.state1))
    else:
        b1, b2, t = hyper.beta1, hyper.beta2, hyper.step
        tol_m = (1 - b1) * eg + 3 * U * (b1 * np.abs(state1) + (1 - b1) * g)
        tol_v = (1 - b2) * (2 * g * eg + eg * eg) + 4 * U * ref.state2
        assert np.all(np.abs(got_s1 - ref.state1) <= 2 * tol_m + 1e-9)
        assert np.all(np.abs(got_s2 - ref.state2) <= 2 * tol_v + 1e-12)
        bc1, bc2 = 1 / (1 - b1 ** t), 1 / (1 - b2 ** t)
        mhat, vhat = np.abs(ref.state1) * bc1, ref.state2 * bc2
        e_vhat = tol_v * bc2
        e_sqrt = np.minimum(e_vhat / np.maximum(2 * np.sqrt(vhat), 1e-300), np.sqrt(e_vhat))
        den = np.sqrt(vhat) + hyper.eps
        step = mhat / den
        tol_step = tol_m * bc1 / den + mhat * e_sqrt / (den * np.maximum(den - e_sqrt, 1e-300)) + 8 * U * step
        tol_w = lr * tol_step + 2 * U * (w + lr * step)
    err = np.abs(got_w - ref.weight)
    bad = err > 2 * tol_w + 1e-7
    assert not bad.any(), "%d weights out of tolerance, worst err/tol %.3g" % (int(bad.sum()), float((err / (2 * tol_w + 1e-7)).max()))
    return ref, result


def make_case(vocab, d, sizes, seed, with_dense=True, std=0.05, integers=False):
    rng = np.random.default_rng(seed)
    idx = [zipf_indices(rng, s, vocab) for s in sizes]
    if integers:
        val = [rng.integers(-4, 5, size=(s, d)).astype(np.float32) for s in sizes]
        dense = rng.integers(-4, 5, size=(vocab, d)).astype(np.float32) if with_dense else None
        weight = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
        s1 = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
        s2 = rng.integers(0, 9, size=(vocab, d)).astype(np.float32)
    else:
        val = [(rng.standard_normal((s, d)) * std).astype(np.float32) for s in sizes]
        dense = (rng.standard_normal((vocab, d)) * std).astype(np.float32) if with_dense else None
        weight = rng.standard_normal((vocab, d)).astype(np.float32)
        s1 = (rng.standard_normal((vocab, d)) * std).astype(np.float32)
        s2 = (rng.random((vocab, d)) * std * std).astype(np.float32)
    return idx, val, dense, weight, s1, s2


HYPERS = [oo.Hyper(kind=oo.MOMENTUM, lr=0.05, momentum=0.9),
          oo.Hyper(kind=oo.ADAM, lr=0.002, beta1=0.9, beta2=0.98, eps=1e-6, step=3),
          oo.Hyper(kind=oo.SGD, lr=0.1, grad_scale=0.5)]


@pytest.mark.parametrize("hyper", HYPERS, ids=lambda h: h.kind)
@pytest.mark.parametrize("name", ["tiny", "base", "big"])
def test_paper_configurations(name, hyper):
    w = make_workload(name)                                         # one-cluster index path: copy items take the unnamed rows
    rng = np.random.default_rng(1)
    weight = rng.normal(0, 1, size=(w.vocab, w.d)).astype(np.float32)
    s1 = rng.normal(0, 0.02, size=(w.vocab, w.d)).astype(np.float32)
    s2 = (rng.random((w.vocab, w.d)) * 4e-4).astype(np.float32)
    check(w.indices, w.values, w.d, w.vocab, w.dense_in, weight, hyper, s1, s2)


@pytest.mark.parametrize("hyper", HYPERS[:2], ids=lambda h: h.kind)
@pytest.mark.parametrize("with_dense", [True, False])
@pytest.mark.parametrize("vocab,d,sizes", [(600, 64, [3000, 3000, 3000]), (70000, 32, [15000, 15000]), (3000, 1024, [2500]),
                                           (257, 2056, [10000] * 4), (5000, 7, [900, 40])])
def test_general_and_small_paths(vocab, d, sizes, with_dense, hyper):
    idx, val, dense, weight, s1, s2 = make_case(vocab, d, sizes, vocab + d, with_dense)
    ref, result = check(idx, val, d, vocab, dense, weight, hyper, s1, s2)
    assert int(result[0]) == 0


@pytest.mark.parametrize("kind", [oo.MOMENTUM, oo.ADAM])
def test_exact_on_small_integers_with_dyadic_hyper_parameters(kind):
    # every intermediate is a small dyadic number: fp32 on the device and fp64 in the oracle agree bit for bit
    # (Adam at step 1 with beta1 = 1/2, beta2 = 3/4 from zero state: mhat = g, vhat = g^2, step = g / (|g| + eps))
    vocab, d = 900, 64
    idx, val, dense, weight, s1, s2 = make_case(vocab, d, [1500, 700], 4, integers=True)
    if kind == oo.MOMENTUM:
        check(idx, val, d, vocab, dense, weight, oo.Hyper(kind=kind, lr=0.25, momentum=0.5), s1, exact=True)
    else:
        z = np.zeros_like(weight)
        got_w, got_m, got_v, _ = run(idx, val, d, vocab, dense, weight, oo.Hyper(kind=kind, lr=0.5, beta1=0.5, beta2=0.75, eps=1.0, step=1), z, z)
        ref = oo.apply_step(idx, val, d, vocab, dense, weight, oo.Hyper(kind=kind, lr=0.5, beta1=0.5, beta2=0.75, eps=1.0, step=1), z, z)
        assert np.array_equal(got_m, ref.state1) and np.array_equal(got_v, ref.state2)      # g / 2 and g^2 / 4: exact
        assert np.all(np.abs(got_w - ref.weight) <= 4 * U * (np.abs(ref.weight) + 1))         # one division, rounded once more


@pytest.mark.parametrize("hyper", HYPERS[:2], ids=lambda h: h.kind)
def test_bf16_gradients_with_a_loss_scale(hyper):
    # reduced-precision gradients, scaled by 1024 upstream: bf16 value rows and dense partner, fp32 weight and state
    vocab, d, scale = 4000, 256, 1024.0
    idx, val, dense, weight, s1, s2 = make_case(vocab, d, [3000, 1200], 8)
    valb = [to_bf16_bits(v * scale) for v in val]
    denseb = to_bf16_bits(dense * scale)
    h = dataclasses.replace(hyper, grad_scale=1.0 / scale)
    check(idx, valb, d, vocab, denseb, weight, h, s1, s2, grad="bf16")
    # general index path, no dense partner
    vocab = 70000
    idx, val, dense, weight, s1, s2 = make_case(vocab, 64, [20000], 9, with_dense=False)
    check(idx, [to_bf16_bits(v * scale) for v in val], 64, vocab, None, weight, h, s1, s2, grad="bf16")


def test_out_of_range_indices_and_argument_checks():
    vocab, d = 500, 64
    idx, val, dense, weight, s1, s2 = make_case(vocab, d, [2000], 11)
    idx[0][::5] = vocab + 3
    ref, result = check(idx, val, d, vocab, dense, weight, HYPERS[1], s1, s2)
    assert int(result[0]) == 4 and int(result[2]) == ref.grad.shape[0] * 0 + int((idx[0] >= vocab).sum())
    w = torch.zeros(vocab, d, device="cuda")
    ws = torch.empty(dst.dst_workspace_bytes(2000, 1, d, vocab), dtype=torch.uint8, device="cuda")
    sl = [(torch.from_numpy(idx[0]).cuda(), torch.from_numpy(val[0]).cuda())]
    with pytest.raises(dst.DstError):                              # Adam without its second moment
        dst.dst_densify_apply(sl, d, vocab, None, w, ws, kind=dst.DST_OPT_ADAM, lr=0.1, state1=torch.zeros_like(w))
    with pytest.raises(dst.DstError):                              # the weight is not its own state
        dst.dst_densify_apply(sl, d, vocab, None, w, ws, kind=dst.DST_OPT_MOMENTUM, lr=0.1, state1=w)
    with pytest.raises(dst.DstError):                              # step numbers start at 1
        dst.dst_densify_apply(sl, d, vocab, None, w, ws, kind=dst.DST_OPT_ADAM, lr=0.1, step=0,
                              state1=torch.zeros_like(w), state2=torch.zeros_like(w))
