"""Pins for the oracle's deployed stochastic pruning rule and calibrator buffers (Appendix A.4: sliding buffers,
p_i = clip(kappa + delta + lambda (rho - q_i), p_min, p_max), delta by bisection so that E[p] = kappa)."""
from collections import deque
from fractions import Fraction

import numpy as np

import oracle


def test_sliding_buffers_are_fifo_per_label():
    g = np.random.default_rng(0)
    cap = 7
    buf = oracle.ScoreBuffers(cap)
    ref_pos, ref_neg = deque(maxlen=cap), deque(maxlen=cap)
    for _ in range(9):
        n = int(g.integers(0, 6))
        s, y = g.random(n), (g.random(n) < 0.4).astype(np.uint8)
        buf.push(s, y)
        for sk, yk in zip(s, y):
            (ref_pos if yk else ref_neg).append(sk)
        pos, neg = buf.contents()
        assert list(pos) == list(ref_pos) and list(neg) == list(ref_neg)
    cpos, cneg = buf.counts(4)
    assert cpos.sum() == len(ref_pos) and cneg.sum() == len(ref_neg)
    assert list(cpos) == [sum(1 for v in ref_pos if min(3, int(4 * v)) == b) for b in range(4)]


def _expected_keep(cpos, cneg, lut, delta, kappa, lam, rho, pmin, pmax):
    n = int(sum(cpos) + sum(cneg))
    tot = Fraction(0)
    for b in range(len(lut)):
        p = Fraction(kappa) + Fraction(delta) + Fraction(lam) * (Fraction(rho) - Fraction(float(lut[b])))
        p = min(max(p, Fraction(pmin)), Fraction(pmax))
        tot += (int(cpos[b]) + int(cneg[b])) * p
    return tot / n


def test_delta_makes_the_expected_keep_rate_kappa():
    g = np.random.default_rng(1)
    B = 16
    for trial in range(20):
        cpos, cneg = g.integers(0, 40, size=B), g.integers(0, 40, size=B)
        _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
        kappa = [0.5, 0.25, 0.75][trial % 3]
        d = oracle.solve_delta(cpos, cneg, lut, kappa=kappa, lam=0.5, rho=0.5, p_min=0.05, p_max=0.95)
        e = _expected_keep(cpos, cneg, lut, d, kappa, 0.5, 0.5, 0.05, 0.95)     # exact rationals
        assert abs(float(e) - kappa) < 1e-12
    # no clipping active: closed form delta = lambda (E[q] - rho)
    cpos, cneg = np.array([5, 5, 5, 5]), np.array([5, 5, 5, 5])
    lut = np.array([0.3, 0.4, 0.6, 0.7], np.float32)
    d = oracle.solve_delta(cpos, cneg, lut, kappa=0.5, lam=0.5, rho=0.4, p_min=0.0, p_max=1.0)
    eq = float(np.mean(lut.astype(np.float64)))
    assert abs(d - 0.5 * (eq - 0.4)) < 1e-12
    # lambda = 0: p = kappa for everyone, delta = 0; empty buffers: delta = 0
    assert abs(oracle.solve_delta(cpos, cneg, lut, kappa=0.3, lam=0.0)) < 1e-15
    assert oracle.solve_delta(np.zeros(4, np.int64), np.zeros(4, np.int64), lut) == 0.0


def test_survival_probability_shape_and_decisions():
    q = np.linspace(0, 1, 11).astype(np.float32)
    u = np.full(11, 0.5, np.float32)
    keep, p = oracle.select_stochastic(q, u, delta=0.1, kappa=0.5, lam=0.5, rho=0.5, p_min=0.2, p_max=0.8)
    expect = np.clip(0.5 + 0.1 + 0.5 * (0.5 - q.astype(np.float64)), 0.2, 0.8)
    assert np.allclose(p, expect, atol=1e-15)
    assert np.all(np.diff(p) <= 0) and p.min() >= 0.2 and p.max() <= 0.8       # decreasing in q, clipped
    assert np.array_equal(keep, (0.5 < p).astype(np.uint8))                    # survive iff u < p
    # u = p exactly is pruned (strict inequality); ineligible rollouts are always kept with p = 1
    keep, p = oracle.select_stochastic(np.array([0.5, 0.5, 0.9], np.float32), np.array([0.5, 0.25, 0.99], np.float32),
                                       delta=0.0, eligible=np.array([1, 1, 0], np.uint8))
    assert list(keep) == [0, 1, 1] and p[2] == 1.0 and p[0] == 0.5


def test_keep_rate_matches_kappa_in_expectation():
    g = np.random.default_rng(2)
    B, n = 128, 200000
    hist = g.beta(2, 3, size=8192)
    y = (g.random(8192) < hist).astype(np.uint8)
    cpos, cneg = oracle.calib_counts(hist, y, B)
    _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
    d = oracle.solve_delta(cpos, cneg, lut)
    s_new = g.beta(2, 3, size=n)                         # same score distribution as the buffers
    _, bins, q = oracle.prob_map(np.log(s_new / (1 - s_new)), lut)
    keep, p = oracle.select_stochastic(q.astype(np.float32), g.random(n).astype(np.float32), d)
    assert abs(keep.mean() - 0.5) < 0.01
    # as printed, p is affine and decreasing in q: likely-correct rollouts are pruned more often than unlikely ones
    assert p[q > 0.5].mean() < p[q < 0.5].mean()
    assert q[keep == 1].mean() < q[keep == 0].mean()
