"""Oracle for the optimizer steps fused into the densify pass.  TEST INFRASTRUCTURE ONLY.

The paper hands the accumulated gradient of the tied weight to the optimizer that
``DistributedOptimizer(opt, sparse_as_dense=True)`` wraps (Section 4) and mentions training in
reduced precision (Section 1).  What that optimizer computes is not the paper's subject; the
update rules below are the published ones, written out step by step in fp64:

* plain SGD                       w <- w - lr * g
* SGD with momentum (heavy ball)  b <- mu * b + g;  w <- w - lr * b
* Adam (Kingma & Ba, Algorithm 1) m <- beta1 * m + (1 - beta1) * g;  v <- beta2 * v + (1 - beta2) * g^2
                                  mhat = m / (1 - beta1^t);  vhat = v / (1 - beta2^t)
                                  w <- w - lr * mhat / (sqrt(vhat) + eps)

with g the dense gradient of the paper's Section 4: ``grad_scale * (dense_in + scatter-sum of the
value rows)``.  ``grad_scale`` is the reciprocal of the loss scale of reduced-precision training
(1 when gradients are not scaled); it multiplies the fp64 sum (multiplying every term first differs
by fp64 rounding only, and not at all for a power of two).  Gradients may be fp32 or bf16
(``value_dtype``; the dense partner has the same type); weight and optimizer state are fp32.

Every row of the weight and of the state takes the step, named or not: with momentum or Adam a
zero gradient still moves the state and the weight.

Nothing here is imported by the CUDA library or its binding.
Pins: ``tests/test_optimizer_oracle.py`` (hand-worked two-step examples, exactness on dyadic
hyper-parameters, ``torch.optim.SGD`` / ``torch.optim.Adam`` in fp64 on the densified gradient).
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import numpy as np

from . import dst_oracle

SGD, MOMENTUM, ADAM = "sgd", "momentum", "adam"


@dataclasses.dataclass
class Hyper:
    kind: str = SGD
    lr: float = 0.1
    momentum: float = 0.9          # MOMENTUM: mu
    beta1: float = 0.9             # ADAM
    beta2: float = 0.999
    eps: float = 1e-8
    step: int = 1                  # ADAM: t, the number of this step, starting at 1
    grad_scale: float = 1.0        # reciprocal of the loss scale


@dataclasses.dataclass
class Stepped:
    weight: np.ndarray             # fp64 [vocab, d]
    state1: Optional[np.ndarray]   # MOMENTUM: b; ADAM: m
    state2: Optional[np.ndarray]   # ADAM: v
    grad: np.ndarray               # g, fp64
    grad_mag: np.ndarray           # |grad_scale| * sum of |terms| of g (for tolerances)


def gradient(indices: Sequence[np.ndarray], values: Sequence[np.ndarray], d: int, vocab: int,
             dense_in: Optional[np.ndarray], grad_scale: float = 1.0, value_dtype: str = "f32"):
    """g and the sum of |terms| behind it; bf16 tensors come as uint16 bit patterns."""
    r = dst_oracle.densify(indices, values, d, vocab, dense_in, value_dtype=value_dtype, out_dtype=value_dtype)
    return float(grad_scale) * r.acc, abs(float(grad_scale)) * r.mag


def apply_step(indices: Sequence[np.ndarray], values: Sequence[np.ndarray], d: int, vocab: int,
               dense_in: Optional[np.ndarray], weight: np.ndarray, hyper: Hyper,
               state1: Optional[np.ndarray] = None, state2: Optional[np.ndarray] = None,
               value_dtype: str = "f32") -> Stepped:
    g, mag = gradient(indices, values, d, vocab, dense_in, hyper.grad_scale, value_dtype)
    w = np.asarray(weight, np.float32).reshape(vocab, d).astype(np.float64)
    lr = float(hyper.lr)
    if hyper.kind == SGD:
        return Stepped(w - lr * g, None, None, g, mag)
    if hyper.kind == MOMENTUM:
        b = np.asarray(state1, np.float32).reshape(vocab, d).astype(np.float64)
        b = float(hyper.momentum) * b + g
        return Stepped(w - lr * b, b, None, g, mag)
    if hyper.kind == ADAM:
        m = np.asarray(state1, np.float32).reshape(vocab, d).astype(np.float64)
        v = np.asarray(state2, np.float32).reshape(vocab, d).astype(np.float64)
        b1, b2, t = float(hyper.beta1), float(hyper.beta2), int(hyper.step)
        m = b1 * m + (1.0 - b1) * g
        v = b2 * v + (1.0 - b2) * (g * g)
        mhat = m / (1.0 - b1 ** t)
        vhat = v / (1.0 - b2 ** t)
        return Stepped(w - lr * mhat / (np.sqrt(vhat) + float(hyper.eps)), m, v, g, mag)
    raise ValueError(hyper.kind)
