"""Pins for the oracle's quality-head training step (cross-entropy on (score, reward), gradients into the head
only; Sections 4.2 and 4.3 (iii)): torch autograd in float64, finite differences of the oracle's forward, closed
forms."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import headtrain as oh


def _case(N, d, h, seed):
    g = np.random.default_rng(seed)
    x = g.normal(size=(3 * N, d)).astype(np.float32)
    ridx = g.permutation(3 * N)[:N].astype(np.int64)
    y = (g.random(N) < 0.4).astype(np.uint8)
    mask = (g.random(N) < 0.8).astype(np.uint8)
    mask[0] = 1
    mk = lambda *s: g.normal(0, 0.3, size=s).astype(np.float32)
    if h == 0:
        return x, ridx, y, mask, dict(W1=mk(d), b1=mk(1), w2=None, b2=None)
    return x, ridx, y, mask, dict(W1=mk(h, d), b1=mk(h), w2=mk(h), b2=mk(1))


@pytest.mark.parametrize("h", [0, 6])
def test_matches_torch_autograd(h):
    N, d = 11, 9
    x, ridx, y, mask, p = _case(N, d, h, 1 + h)
    loss, grads = oh.head_bce_grad(x, y, p["W1"], p["b1"], p["w2"], p["b2"], row_index=ridx, h=h, mask=mask)
    X = torch.from_numpy(x[ridx]).double()
    tp = {k: torch.from_numpy(v).double().requires_grad_(True) for k, v in p.items() if v is not None}
    if h == 0:
        s = X @ tp["W1"] + tp["b1"]
    else:
        s = torch.nn.functional.gelu(X @ tp["W1"].T + tp["b1"]) @ tp["w2"] + tp["b2"]
    m = torch.from_numpy(mask.astype(bool))
    ref = torch.nn.functional.binary_cross_entropy_with_logits(s[m], torch.from_numpy(y).double()[m])
    ref.backward()
    assert abs(loss - ref.item()) < 1e-13
    for k, gk in grads.items():
        assert np.allclose(gk, tp[k].grad.numpy().reshape(gk.shape), atol=1e-13), k


def test_finite_differences_of_the_forward_oracle():
    N, d, h = 7, 5, 4
    x, ridx, y, mask, p = _case(N, d, h, 5)
    _, grads = oh.head_bce_grad(x, y, p["W1"], p["b1"], p["w2"], p["b2"], row_index=ridx, h=h, mask=mask)

    def L(q):
        s = oracle.head_score(x.astype(np.float64), q["W1"].astype(np.float64), q["b1"].astype(np.float64),
                              q["w2"].astype(np.float64), q["b2"].astype(np.float64), row_index=ridx, h=h)
        m = mask.astype(bool)
        return float(np.mean(np.logaddexp(0.0, s[m]) - y[m] * s[m]))

    eps = 1e-6
    for name, idx in (("W1", (2, 3)), ("b1", (1,)), ("w2", (0,)), ("b2", (0,))):
        plus = {k: v.astype(np.float64).copy() for k, v in p.items()}
        minus = {k: v.astype(np.float64).copy() for k, v in p.items()}
        plus[name][idx] += eps
        minus[name][idx] -= eps
        assert abs((L(plus) - L(minus)) / (2 * eps) - grads[name][idx]) < 1e-8


def test_closed_forms():
    # zero weights: s = 0 for everyone: loss = log 2, ds = (1/2 - y)/n, dw = sum ds x, db = sum ds
    N, d = 6, 4
    g = np.random.default_rng(2)
    x = g.normal(size=(N, d)).astype(np.float32)
    y = np.array([1, 0, 0, 1, 1, 0], np.uint8)
    loss, grads = oh.head_bce_grad(x, y, np.zeros(d, np.float32), np.zeros(1, np.float32))
    assert abs(loss - math.log(2.0)) < 1e-15
    ds = (0.5 - y.astype(np.float64)) / N
    assert np.allclose(grads["W1"], ds @ x.astype(np.float64), atol=1e-15) and abs(grads["b1"][0] - ds.sum()) < 1e-15
    # masked-out rollouts contribute nothing; an empty mask gives zero loss and gradients
    loss2, g2 = oh.head_bce_grad(x, y, np.zeros(d, np.float32), np.zeros(1, np.float32), mask=np.array([1, 1, 1, 0, 0, 0], np.uint8))
    ds2 = (0.5 - y[:3].astype(np.float64)) / 3
    assert np.allclose(g2["W1"], ds2 @ x[:3].astype(np.float64), atol=1e-15)
    loss3, g3 = oh.head_bce_grad(x, y, np.zeros(d, np.float32), np.zeros(1, np.float32), mask=np.zeros(N, np.uint8))
    assert loss3 == 0.0 and np.all(g3["W1"] == 0.0)
    # large logits do not overflow: loss ~ |s| for the wrong label, ~0 for the right one
    w = np.array([800.0, 0, 0, 0], np.float32)
    xs = np.array([[1, 0, 0, 0], [-1, 0, 0, 0]], np.float32)
    loss4, _ = oh.head_bce_grad(xs, np.array([0, 0], np.uint8), w)
    assert abs(loss4 - 400.0) < 1e-9
