"""Pins for the oracle's per-group balancing selection (Section 4.1: Theorem 1's rule
j^ = argmin_j |mu_{-j} - rho|, repeated until K of G remain).

Checked against exact rational brute force of the rule as the paper writes it (with the mean and the
division), worked examples, structural invariants, and the paper's own statements about the rule
(Lemma A.1 and Theorem 1's probabilistic bound).
"""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _brute_force_group(q, K, rho):
    """The rule exactly as printed: at every step evaluate |mean(q over S without j) - rho| for every j in
    exact rationals and remove the minimiser; of several minimisers the highest index goes."""
    S = list(range(len(q)))
    qf = [Fraction(float(v)) for v in q]
    rho = Fraction(rho)
    removed = []
    while len(S) > K:
        devs = {}
        for j in S:
            rest = [qf[i] for i in S if i != j]
            devs[j] = abs(sum(rest) / len(rest) - rho)
        best = min(devs.values())
        j_hat = max(j for j in S if devs[j] == best)
        S.remove(j_hat)
        removed.append(j_hat)
    return S, removed


def test_worked_examples():
    # Dyadic stand-ins (multiples of 1/128) for q = (.9, .8, .3, .1), rho = .5, keep 2, so that every
    # quantity is exact and the example can be followed by hand: mu_{-j} ~ (.40, .43, .60, .67), the closest
    # to .5 is j = 1 (deviation ~.066); then among (.9,.3,.1) removing .3 leaves mean .5.
    q = np.array([115, 102, 38, 13], dtype=np.float32) / 128      # ~ (.9, .8, .3, .1)
    keep, order = oracle.select(q, 1, 4, 2, 0.5, return_order=True)
    S, removed = _brute_force_group(q, 2, Fraction(1, 2))
    assert list(order[0]) == removed == [1, 2]
    assert list(keep) == [1, 0, 0, 1]
    # eight rollouts, keep four; the first step is an exact tie between the two 0.125's -> index 7 goes
    q = np.array([112, 104, 88, 80, 24, 24, 16, 16], dtype=np.float32) / 128
    keep, order = oracle.select(q, 1, 8, 4, 0.5, return_order=True)
    S, removed = _brute_force_group(q, 4, Fraction(1, 2))
    assert list(order[0]) == removed
    assert removed[0] == 7
    assert sorted(np.flatnonzero(keep)) == S
    # by hand: Sigma = 464/128, n = 8, tau = Sigma - 3.5 = 16/128 -> keys |q - tau| minimal (0) at the two 16/128
    assert float(Fraction(464, 128) - Fraction(7, 2)) == 0.125


def test_single_removal_is_the_papers_rule_literally():
    # K = G - 1: one application of j^ = argmin_j |mu_{-j} - rho|  (Theorem 1)
    g = np.random.default_rng(0)
    for G in (2, 3, 5, 8, 16, 32):
        for _ in range(40):
            q = (g.integers(0, 129, size=G) / 128).astype(np.float32)
            rho = Fraction(int(g.integers(0, 9)), 8)
            keep = oracle.select(q, 1, G, G - 1, float(rho))
            mu = {j: abs((sum(Fraction(float(v)) for i, v in enumerate(q) if i != j)) / (G - 1) - rho)
                  for j in range(G)}
            best = min(mu.values())
            j_hat = max(j for j in range(G) if mu[j] == best)
            assert list(np.flatnonzero(keep == 0)) == [j_hat]


@pytest.mark.parametrize("G", [2, 3, 4, 7, 8, 16, 31, 32])
def test_every_greedy_step_is_the_exact_argmin(G):
    g = np.random.default_rng(G)
    for K in sorted({1, max(1, G // 2), G - 1, G}):
        for trial in range(12):
            # coarse dyadic grid -> many exact ties
            q = (g.integers(0, 17, size=G) / 16).astype(np.float32)
            rho = [Fraction(1, 2), Fraction(1, 4), Fraction(3, 8)][trial % 3]
            keep, order = oracle.select(q, 1, G, K, float(rho), return_order=True)
            S, removed = _brute_force_group(q, K, rho)
            assert list(order[0]) == removed
            assert sorted(np.flatnonzero(keep)) == S


def test_exactly_k_survive_for_every_g_and_k():
    g = np.random.default_rng(1)
    for G in range(2, 33):
        P = 3
        q = g.random(P * G).astype(np.float32)
        for K in range(1, G + 1):
            keep = oracle.select(q, P, G, K, 0.5)
            assert keep.dtype == np.uint8 and set(np.unique(keep)) <= {0, 1}
            assert np.array_equal(keep.reshape(P, G).sum(1), np.full(P, K))
        assert np.all(oracle.select(q, P, G, G, 0.5) == 1)       # K = G keeps everyone


def test_groups_are_independent_and_all_equal_q_keeps_the_lowest_indices():
    g = np.random.default_rng(2)
    G, K = 16, 8
    q = g.random(5 * G).astype(np.float32)
    full = oracle.select(q, 5, G, K, 0.5)
    for p in range(5):
        assert np.array_equal(full[p * G:(p + 1) * G], oracle.select(q[p * G:(p + 1) * G], 1, G, K, 0.5))
    for val in (0.0, 0.25, 1.0):
        keep = oracle.select(np.full(G, val, np.float32), 1, G, K, 0.5)
        assert list(keep) == [1] * K + [0] * (G - K)              # every step is a G-way tie: highest index goes


def test_selection_moves_the_kept_mean_toward_rho():
    # Not Lemma 1's strict decrease (a single removal can overshoot), but the purpose of the rule:
    # on spread-out posteriors the kept mean is closer to rho than a random keep of the same size, on average.
    g = np.random.default_rng(3)
    G, K, P = 16, 8, 400
    q = g.beta(0.5, 0.5, size=P * G).astype(np.float32)
    keep = oracle.select(q, P, G, K, 0.5).reshape(P, G).astype(bool)
    qq = q.reshape(P, G)
    dev_sel = np.abs(np.array([qq[p, keep[p]].mean() for p in range(P)]) - 0.5).mean()
    dev_rand = np.abs(qq[:, :K].mean(1) - 0.5).mean()
    assert dev_sel < 0.25 * dev_rand


def test_lemma_a1_error_transfer():
    # |q_i - q*_i| <= eps for all i  =>  |mu_{-j} - mu*_{-j}| <= eps for every j   (Lemma A.1)
    g = np.random.default_rng(4)
    G, eps = 16, 0.05
    for _ in range(50):
        qs = g.random(G)
        q = np.clip(qs + g.uniform(-eps, eps, G), 0, 1)
        for j in range(G):
            mu = (q.sum() - q[j]) / (G - 1)
            mus = (qs.sum() - qs[j]) / (G - 1)
            assert abs(mu - mus) <= eps + 1e-15


def test_theorem_1_bound_holds_with_the_stated_probability():
    # With prob >= 1 - delta:  |p^_{-j^} - rho| <= min_j |mu*_{-j} - rho| + 2 eps + sqrt(log(2/delta) / (2 (G-1)))
    g = np.random.default_rng(5)
    G, eps, delta, rho, trials = 16, 0.05, 0.1, 0.5, 4000
    ok = 0
    for _ in range(trials):
        qs = g.beta(0.7, 0.7, size=G)
        y = (g.random(G) < qs).astype(np.float64)
        q = (qs + g.uniform(-eps, eps, G)).astype(np.float32)
        keep = oracle.select(q, 1, G, G - 1, rho).astype(bool)
        p_hat = y[keep].mean()
        best_true = min(abs((qs.sum() - qs[j]) / (G - 1) - rho) for j in range(G))
        bound = best_true + 2 * (eps + 1e-7) + math.sqrt(math.log(2 / delta) / (2 * (G - 1)))
        ok += abs(p_hat - rho) <= bound
    assert ok / trials >= 1 - delta


def test_argument_checks():
    q = np.zeros(8, np.float32)
    for G, K in ((8, 0), (8, 9), (0, 1)):
        with pytest.raises((ValueError, AssertionError)):
            oracle.select(q[: max(G, 0)], 1, G, K, 0.5)
