"""Pins for the oracle's rank-weighted vote (Section 4.4): hand examples and brute force with Python's sort."""
from collections import OrderedDict
from fractions import Fraction

import numpy as np

from oracle import tts


def _brute(score, answer, G):
    order = sorted(range(G), key=lambda i: (float(score[i]), i))          # stable ascending
    w = [Fraction(0)] * G
    for r, i in enumerate(order):
        w[i] = Fraction(r, G - 1) if G > 1 else Fraction(1)
    totals = OrderedDict()
    for i in range(G):
        if answer[i] >= 0:
            totals[answer[i]] = totals.get(answer[i], Fraction(0)) + w[i]
    if not totals:
        return w, -1, Fraction(0)
    best = max(totals.values())
    win = next(a for a, t in totals.items() if t == best)                  # first to appear among equals
    return w, win, best


def test_hand_example_tie_goes_to_first_appearing_answer():
    score = np.array([0.5, 0.9, 0.1, 0.7], np.float32)
    answer = np.array([42, 7, 42, 42], np.int32)
    wts, win, ww = tts.rank_vote(score, answer, 1, 4)
    assert np.allclose(wts, [1 / 3, 1.0, 0.0, 2 / 3])   # ascending scores: idx 2 < 0 < 3 < 1
    w, bwin, bw = _brute(score, answer, 4)
    assert bwin == 42 and bw == 1
    assert win[0] == bwin and abs(ww[0] - float(bw)) < 1e-15
    # plain majority would also say 42; a confident minority can win: give 7 the two top scores
    score = np.array([0.1, 0.9, 0.2, 0.8, 0.3], np.float32)
    answer = np.array([5, 7, 5, 7, 5], np.int32)
    _, win, ww = tts.rank_vote(score, answer, 1, 5)
    assert win[0] == 7 and abs(ww[0] - (1.0 + 0.75)) < 1e-15     # 7: 1 + 3/4; 5: 0 + 1/4 + 2/4


def test_brute_force_random_groups_with_ties_and_missing_answers():
    g = np.random.default_rng(0)
    for G in (1, 2, 3, 8, 16, 32):
        P = 50
        score = (g.integers(0, 6, size=P * G) / 4).astype(np.float32)     # many equal scores
        answer = g.integers(-1, 4, size=P * G).astype(np.int32)
        answer[:G] = -1                                                  # a group with no answer at all
        w, win, ww = tts.rank_vote(score, answer, P, G)
        for p in range(P):
            bw, bwin, btot = _brute(score[p * G:(p + 1) * G], answer[p * G:(p + 1) * G], G)
            assert np.allclose(w[p * G:(p + 1) * G], [float(x) for x in bw], atol=1e-15)
            assert win[p] == bwin and abs(ww[p] - float(btot)) < 1e-12
        assert win[0] == -1 and ww[0] == 0.0
