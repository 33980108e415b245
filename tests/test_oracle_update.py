"""Pins for the oracle's clipped GRPO / DAPO objective (Section 3) and the lm_head log-prob backward:
closed forms, finite differences of the oracle's own forward functions, and torch autograd in float64."""
import numpy as np
import pytest
import torch

import oracle
from oracle import update as ou


def _batch(seed, S=5, lo=1, hi=9):
    g = np.random.default_rng(seed)
    ell = g.integers(lo, hi + 1, size=S)
    cu = np.concatenate([[0], np.cumsum(ell)]).astype(np.int64)
    T = int(cu[-1])
    logp_old = -g.random(T) * 3
    logp = logp_old + g.normal(0, 0.3, size=T)
    ref = logp_old + g.normal(0, 0.2, size=T)
    adv_s = g.normal(size=S)
    adv = np.repeat(adv_s, ell)
    return cu, logp, logp_old, ref, adv


def test_on_policy_closed_form():
    # logp = logp_old: r = 1 inside the clip range, term = A, d term / d logp = A
    cu, _, logp_old, _, adv = _batch(0)
    S, T = len(cu) - 1, int(cu[-1])
    loss, grad = ou.policy_loss(logp_old, logp_old, adv, cu)
    w = np.repeat(1.0 / (S * np.diff(cu)), np.diff(cu))
    assert abs(loss + np.sum(w * adv)) < 1e-14
    assert np.allclose(grad, -w * adv, atol=1e-15)
    loss1, grad1 = ou.policy_loss(logp_old, logp_old, adv, cu, agg_mode=1)
    assert abs(loss1 + adv.sum() / T) < 1e-14 and np.allclose(grad1, -adv / T, atol=1e-15)


def test_clipping_cases_by_hand():
    cu = np.array([0, 4], dtype=np.int64)
    logp_old = np.zeros(4)
    logp = np.log([1.5, 1.5, 0.5, 0.5])              # ratios outside [0.8, 1.2]
    adv = np.array([1.0, -1.0, 1.0, -1.0])
    loss, grad = ou.policy_loss(logp, logp_old, adv, cu, eps_low=0.2, eps_high=0.2)
    # A>0, r=1.5: min(1.5, 1.2) = 1.2 clipped, no gradient.   A<0, r=1.5: min(-1.5, -1.2) = -1.5, gradient.
    # A>0, r=0.5: min(0.5, 0.8) = 0.5, gradient.              A<0, r=0.5: min(-0.5, -0.8) = -0.8 clipped.
    terms = np.array([1.2, -1.5, 0.5, -0.8])
    assert abs(loss + terms.mean()) < 1e-14
    assert np.allclose(grad, -np.array([0.0, -1.5, 0.5, 0.0]) / 4, atol=1e-15)
    # DAPO's wider upper clip: r = 1.25 with A > 0 is inside [0.8, 1.28] -> unclipped
    loss, grad = ou.policy_loss(np.log([1.25]), np.zeros(1), np.ones(1), np.array([0, 1]), eps_low=0.2, eps_high=0.28)
    assert abs(loss + 1.25) < 1e-14 and abs(grad[0] + 1.25) < 1e-14


@pytest.mark.parametrize("agg_mode,beta", [(0, 0.0), (1, 0.0), (0, 0.04), (1, 0.1)])
def test_policy_loss_matches_torch_autograd(agg_mode, beta):
    cu, logp, logp_old, ref, adv = _batch(3 + agg_mode)
    S, T = len(cu) - 1, int(cu[-1])
    loss, grad = ou.policy_loss(logp, logp_old, adv, cu, logp_ref=ref if beta else None, eps_low=0.2, eps_high=0.28,
                                beta=beta, agg_mode=agg_mode)
    lp = torch.tensor(logp, dtype=torch.float64, requires_grad=True)
    r = torch.exp(lp - torch.tensor(logp_old))
    a = torch.tensor(adv)
    term = torch.minimum(r * a, torch.clamp(r, 0.8, 1.28) * a)
    if beta:
        dlt = torch.tensor(ref) - lp
        term = term - beta * (torch.exp(dlt) - dlt - 1)
    lens = torch.tensor(np.repeat(np.diff(cu), np.diff(cu)), dtype=torch.float64)
    w = 1.0 / (S * lens) if agg_mode == 0 else torch.full((T,), 1.0 / T, dtype=torch.float64)
    ref_loss = -(w * term).sum()
    ref_loss.backward()
    assert abs(loss - ref_loss.item()) < 1e-13
    assert np.allclose(grad, lp.grad.numpy(), atol=1e-13)


def test_lm_head_backward_by_finite_differences_of_the_forward_oracle():
    g = np.random.default_rng(5)
    T, d, V = 6, 5, 11
    H = g.normal(size=(T, d))
    W = g.normal(0, 0.5, size=(V, d))
    y = g.integers(0, V, size=T).astype(np.int32)
    y[2] = -1                                          # ignored position
    c = g.normal(size=T)                               # upstream gradient d L / d logp
    dH, dW = ou.lm_head_backward(H, W, y, c, inv_temp=0.7)

    def L(Hx, Wx):
        lp, _ = oracle.token_logprob(Hx, Wx, y, inv_temp=0.7)
        return float(np.sum(c * lp))                   # ignored rows give logp = 0

    h = 1e-6
    for (t, k) in [(0, 0), (1, 3), (2, 2), (5, 4)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[t, k] += h
        Hm[t, k] -= h
        assert abs((L(Hp, W) - L(Hm, W)) / (2 * h) - dH[t, k]) < 1e-7
    for (v, k) in [(0, 0), (int(y[0]), 1), (10, 4), (int(y[5]), 2)]:
        Wp, Wm = W.copy(), W.copy()
        Wp[v, k] += h
        Wm[v, k] -= h
        assert abs((L(H, Wp) - L(H, Wm)) / (2 * h) - dW[v, k]) < 1e-7
    assert np.all(dH[2] == 0.0)                        # the ignored position has no gradient


def test_lm_head_backward_matches_torch_autograd_and_invariants():
    g = np.random.default_rng(6)
    T, d, V = 9, 16, 40
    Hb = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16)
    Wb = torch.from_numpy(g.normal(0, 0.3, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    y = g.integers(0, V, size=T).astype(np.int32)
    c = g.normal(size=T)
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    dH, dW = ou.lm_head_backward(bits(Hb), bits(Wb), y, c)
    Ht = Hb.double().requires_grad_(True)
    Wt = Wb.double().requires_grad_(True)
    lp = torch.log_softmax(Ht @ Wt.T, -1).gather(1, torch.from_numpy(y).long()[:, None])[:, 0]
    (torch.from_numpy(c) * lp).sum().backward()
    assert np.allclose(dH, Ht.grad.numpy(), atol=1e-12) and np.allclose(dW, Wt.grad.numpy(), atol=1e-12)
    # rows of dz sum to zero: sum_v dW[v, :] = 0
    assert np.abs(dW.sum(0)).max() < 1e-12
