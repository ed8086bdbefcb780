"""Pins for the oracle of the optimizer steps fused into the densify pass (``oracle.optimizer_oracle``):
hand-worked two-step examples, exactness on dyadic hyper-parameters, the library optimizers of PyTorch run in
fp64 on a gradient densified by ``numpy.add.at``, and planted mistakes that those checks must reject."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import optimizer_oracle as oo
from paper_1905_04035_b200.workloads import to_bf16_bits

# vocab 2, d 2: dense = [[1,0],[0,0]]; the slices name row 0 twice and row 1 once  ->  g = [[4,2],[4,4]]
IDX = [np.array([0, 0, 1], np.int64)]
VAL = [np.array([[1, 1], [2, 1], [4, 4]], np.float32)]
DENSE = np.array([[1, 0], [0, 0]], np.float32)


def test_gradient_is_the_pinned_scatter_sum_times_the_scale():
    g, mag = oo.gradient(IDX, VAL, 2, 2, DENSE)
    assert g.tolist() == [[4.0, 2.0], [4.0, 4.0]] and mag.tolist() == [[4.0, 2.0], [4.0, 4.0]]
    g, mag = oo.gradient(IDX, VAL, 2, 2, DENSE, grad_scale=-0.25)
    assert g.tolist() == [[-1.0, -0.5], [-1.0, -1.0]] and mag.tolist() == [[1.0, 0.5], [1.0, 1.0]]


def test_momentum_hand_worked_two_steps():
    h = oo.Hyper(kind=oo.MOMENTUM, lr=0.25, momentum=0.5)
    w0 = np.ones((2, 2), np.float32)
    b0 = np.array([[2, 0], [0, -2]], np.float32)
    s1 = oo.apply_step(IDX, VAL, 2, 2, DENSE, w0, h, b0)
    assert s1.state1.tolist() == [[5.0, 2.0], [4.0, 3.0]]                    # 0.5 * b0 + g
    assert s1.weight.tolist() == [[-0.25, 0.5], [0.0, 0.25]]                 # w0 - 0.25 * b1
    s2 = oo.apply_step(IDX, VAL, 2, 2, DENSE, s1.weight.astype(np.float32), h, s1.state1.astype(np.float32))
    assert s2.state1.tolist() == [[6.5, 3.0], [6.0, 5.5]]
    assert s2.weight.tolist() == [[-1.875, -0.25], [-1.5, -1.125]]


def test_adam_hand_worked_two_steps():
    # beta1 = 1/2, beta2 = 3/4, eps = 4, g = [[4,-4],[12,0]]: after bias correction mhat = g and vhat = g^2 at t = 1,
    # and again at t = 2 when g repeats, so each step moves w by lr * g / (|g| + 4) = lr * [[1/2,-1/2],[3/4,0]]
    idx = [np.array([1, 0], np.int64)]
    val = [np.array([[12, 0], [3, -4]], np.float32)]
    dense = np.array([[1, 0], [0, 0]], np.float32)
    h = oo.Hyper(kind=oo.ADAM, lr=0.5, beta1=0.5, beta2=0.75, eps=4.0, step=1)
    z = np.zeros((2, 2), np.float32)
    s1 = oo.apply_step(idx, val, 2, 2, dense, z, h, z, z)
    assert s1.grad.tolist() == [[4.0, -4.0], [12.0, 0.0]]
    assert s1.state1.tolist() == [[2.0, -2.0], [6.0, 0.0]] and s1.state2.tolist() == [[4.0, 4.0], [36.0, 0.0]]
    assert s1.weight.tolist() == [[-0.25, 0.25], [-0.375, 0.0]]
    h2 = dataclasses.replace(h, step=2)
    s2 = oo.apply_step(idx, val, 2, 2, dense, s1.weight.astype(np.float32), h2, s1.state1.astype(np.float32),
                       s1.state2.astype(np.float32))
    assert s2.state1.tolist() == [[3.0, -3.0], [9.0, 0.0]]                   # 3/4 g
    assert s2.state2.tolist() == [[7.0, 7.0], [63.0, 0.0]]                   # 7/16 g^2
    assert s2.weight.tolist() == [[-0.5, 0.5], [-0.75, 0.0]]
    # a gradient that changes sign: m2 = -1, v2 = 7, mhat = -4/3, vhat = 16, step = lr * (-4/3) / (4 + 4)
    s2b = oo.apply_step([np.array([0], np.int64)], [np.array([[-4, 0]], np.float32)], 2, 2, None,
                        np.zeros((2, 2), np.float32), h2, np.array([[2, 0], [0, 0]], np.float32),
                        np.array([[4, 0], [0, 0]], np.float32))
    assert s2b.state1[0, 0] == -1.0 and s2b.state2[0, 0] == 7.0
    assert abs(s2b.weight[0, 0] - 0.5 * (4.0 / 3.0) / 8.0) < 1e-16


def test_rows_nobody_names_still_take_the_step_with_momentum_and_adam():
    w = np.full((3, 1), 8.0, np.float32)
    idx, val = [np.array([1], np.int64)], [np.array([[2.0]], np.float32)]
    s = oo.apply_step(idx, val, 1, 3, None, w, oo.Hyper(kind=oo.MOMENTUM, lr=0.5, momentum=0.5), np.full((3, 1), 4.0, np.float32))
    assert s.state1[:, 0].tolist() == [2.0, 4.0, 2.0] and s.weight[:, 0].tolist() == [7.0, 6.0, 7.0]
    s = oo.apply_step(idx, val, 1, 3, None, w, oo.Hyper(kind=oo.ADAM, lr=1.0, beta1=0.5, beta2=0.75, eps=1.0, step=1),
                      np.full((3, 1), 4.0, np.float32), np.full((3, 1), 4.0, np.float32))
    # row 0: g = 0: m = 2, v = 3, mhat = 4, vhat = 12
    assert s.state1[0, 0] == 2.0 and s.state2[0, 0] == 3.0
    assert abs(s.weight[0, 0] - (8.0 - 4.0 / (np.sqrt(12.0) + 1.0))) < 1e-15
    s = oo.apply_step(idx, val, 1, 3, None, w, oo.Hyper(kind=oo.SGD, lr=0.5))
    assert s.weight[:, 0].tolist() == [8.0, 7.0, 8.0]                         # plain SGD leaves them alone


def test_loss_scale_reciprocal_and_bf16_gradients_are_exact_on_small_integers():
    rng = np.random.default_rng(2)
    vocab, d, n = 23, 4, 150
    idx = [rng.integers(0, vocab, size=n)]
    val = rng.integers(-8, 9, size=(n, d)).astype(np.float32)
    dense = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    w = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    b = rng.integers(-8, 9, size=(vocab, d)).astype(np.float32)
    h = oo.Hyper(kind=oo.MOMENTUM, lr=0.5, momentum=0.25)
    plain = oo.apply_step(idx, [val], d, vocab, dense, w, h, b)
    scaled = oo.apply_step(idx, [val * 128], d, vocab, dense * 128, w, dataclasses.replace(h, grad_scale=1.0 / 128), b)
    assert np.array_equal(plain.weight, scaled.weight) and np.array_equal(plain.state1, scaled.state1)
    half = oo.apply_step(idx, [to_bf16_bits(val * 128)], d, vocab, to_bf16_bits(dense * 128), w,
                         dataclasses.replace(h, grad_scale=1.0 / 128), b, value_dtype="bf16")
    assert np.array_equal(plain.weight, half.weight) and np.array_equal(plain.grad_mag, half.grad_mag)


# ---------------------------------------------------------------------------------------------------------
# the library optimizers in fp64, three steps with a new gradient each step
# ---------------------------------------------------------------------------------------------------------
def _torch_reference(kind, hyper, w0, grads):
    w = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    if kind == oo.SGD:
        opt = torch.optim.SGD([w], lr=hyper.lr)
    elif kind == oo.MOMENTUM:
        opt = torch.optim.SGD([w], lr=hyper.lr, momentum=hyper.momentum)
    else:
        opt = torch.optim.Adam([w], lr=hyper.lr, betas=(hyper.beta1, hyper.beta2), eps=hyper.eps)
    out = []
    for g in grads:
        w.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        out.append(w.detach().numpy().copy())
    return out


def _three_steps(stepper, kind):
    """Runs ``stepper`` (the oracle, or a copy of it with a planted mistake) for three steps against the library."""
    rng = np.random.default_rng(7)
    vocab, d, n = 31, 6, 300
    hyper = oo.Hyper(kind=kind, lr=0.03, momentum=0.8, beta1=0.85, beta2=0.97, eps=1e-6)
    w0 = rng.standard_normal((vocab, d)).astype(np.float32)
    inputs, grads = [], []
    for _ in range(3):
        idx = rng.integers(0, vocab, size=n)
        val = rng.standard_normal((n, d)).astype(np.float32)
        dense = rng.standard_normal((vocab, d)).astype(np.float32)
        g = dense.astype(np.float64)
        np.add.at(g, idx, val.astype(np.float64))                # library scatter-add
        inputs.append((idx, val, dense)); grads.append(g)
    ref = _torch_reference(kind, hyper, w0.astype(np.float64), grads)
    w, s1, s2 = w0.astype(np.float64), np.zeros((vocab, d)), np.zeros((vocab, d))
    worst = 0.0
    for t, (idx, val, dense) in enumerate(inputs, start=1):
        r = stepper([idx], [val], d, vocab, dense, w, dataclasses.replace(hyper, step=t), s1, s2)
        worst = max(worst, float(np.abs(r.weight - ref[t - 1]).max()))
        w, s1, s2 = r.weight, r.state1, r.state2
    return worst


def _oracle_fp64_state(indices, values, d, vocab, dense_in, weight, hyper, state1, state2):
    """The update rules with fp64 state carried between steps, as the library optimizers keep it (the oracle
    itself takes fp32 weight and state, as the CUDA library's tensors are; the test below ties the two)."""
    g, _ = oo.gradient(indices, values, d, vocab, dense_in, hyper.grad_scale)
    return _formula(g, weight, hyper, state1, state2)


def _formula(g, w, h, s1, s2, mistake=None):
    if h.kind == oo.SGD:
        return oo.Stepped(w - h.lr * g, None, None, g, None)
    if h.kind == oo.MOMENTUM:
        b = h.momentum * s1 + (g if mistake != "dampened" else (1 - h.momentum) * g)
        return oo.Stepped(w - h.lr * b if mistake != "sign" else w + h.lr * b, b, None, g, None)
    m = h.beta1 * s1 + (1 - h.beta1) * g
    v = h.beta2 * s2 + (1 - h.beta2) * (g * g if mistake != "no_square" else np.abs(g))
    mhat = m / (1 - h.beta1 ** h.step) if mistake != "no_bias1" else m
    vhat = v / (1 - h.beta2 ** h.step) if mistake != "no_bias2" else v
    den = np.sqrt(vhat) + h.eps if mistake != "eps_inside" else np.sqrt(vhat + h.eps)
    return oo.Stepped(w - h.lr * mhat / den, m, v, g, None)


@pytest.mark.parametrize("kind", [oo.SGD, oo.MOMENTUM, oo.ADAM])
def test_three_steps_equal_the_library_optimizers_in_fp64(kind):
    assert _three_steps(_oracle_fp64_state, kind) < 1e-13
    # and the oracle proper (fp32 state in, as the library's tensors are) equals that formula on fp32-exact state
    rng = np.random.default_rng(3)
    vocab, d, n = 19, 3, 80
    idx, val = [rng.integers(0, vocab, size=n)], [rng.standard_normal((n, d)).astype(np.float32)]
    dense, w = rng.standard_normal((vocab, d)).astype(np.float32), rng.standard_normal((vocab, d)).astype(np.float32)
    s1, s2 = rng.standard_normal((vocab, d)).astype(np.float32), rng.random((vocab, d)).astype(np.float32)
    h = oo.Hyper(kind=kind, lr=0.01, momentum=0.7, beta1=0.8, beta2=0.9, eps=1e-5, step=4, grad_scale=0.5)
    a = oo.apply_step(idx, val, d, vocab, dense, w, h, s1, s2)
    b = _oracle_fp64_state(idx, val, d, vocab, dense, w.astype(np.float64), h, s1.astype(np.float64), s2.astype(np.float64))
    assert np.allclose(a.weight, b.weight, rtol=1e-14, atol=0)
    if kind != oo.SGD:
        assert np.allclose(a.state1, b.state1, rtol=1e-14, atol=0)
    if kind == oo.ADAM:
        assert np.allclose(a.state2, b.state2, rtol=1e-14, atol=0)


@pytest.mark.parametrize("kind,mistake", [(oo.MOMENTUM, "sign"), (oo.MOMENTUM, "dampened"), (oo.ADAM, "no_bias1"),
                                          (oo.ADAM, "no_bias2"), (oo.ADAM, "no_square"), (oo.ADAM, "eps_inside")])
def test_planted_mistakes_are_rejected_by_the_library_comparison(kind, mistake):
    def wrong(indices, values, d, vocab, dense_in, weight, hyper, state1, state2):
        g, _ = oo.gradient(indices, values, d, vocab, dense_in, hyper.grad_scale)
        return _formula(g, weight, hyper, state1, state2, mistake)
    assert _three_steps(wrong, kind) > 1e-6
