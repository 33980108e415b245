"""Pins for the oracle's trace confidence (Section 3 "Trace Confidence"): closed forms, torch in float64, brute force."""
import math

import numpy as np
import torch

from oracle import conf as oc


def test_token_confidence_closed_forms_and_torch():
    g = np.random.default_rng(0)
    T, d, V = 7, 12, 33
    H = g.normal(size=(T, d))
    W = g.normal(0, 0.4, size=(V, d))
    c = oc.token_confidence(H, W)
    ref = -torch.log_softmax(torch.from_numpy(H) @ torch.from_numpy(W).T, -1).sum(-1)
    assert np.allclose(c, ref.numpy(), rtol=0, atol=1e-10)
    # uniform distribution: -sum log(1/V) = V log V, the minimum possible value (Jensen)
    cu = oc.token_confidence(np.zeros((2, d)), W)
    assert np.allclose(cu, V * math.log(V), atol=1e-12)
    assert np.all(c >= V * math.log(V) - 1e-9)
    # two-token vocabulary by hand: logits (0, log 3) -> P = (1/4, 3/4): H = log 4 + log(4/3)
    c2 = oc.token_confidence(np.ones((1, 1)), np.array([[0.0], [math.log(3.0)]]))
    assert abs(c2[0] - (math.log(4) + math.log(4 / 3))) < 1e-14
    # temperature and row subset
    c3 = oc.token_confidence(H, W, rows=np.array([4, 1]), inv_temp=0.5)
    ref3 = -torch.log_softmax(0.5 * (torch.from_numpy(H[[4, 1]]) @ torch.from_numpy(W).T), -1).sum(-1)
    assert np.allclose(c3, ref3.numpy(), atol=1e-10)


def test_trace_confidence_brute_force():
    g = np.random.default_rng(1)
    ell = np.array([1, 5, 0, 17, 64, 9])
    cu = np.concatenate([[0], np.cumsum(ell)])
    Hs = g.random(int(cu[-1])) * 100
    mean = oc.trace_confidence(Hs, cu, mode=0)
    for s, n in enumerate(ell):
        seg = Hs[cu[s]:cu[s + 1]]
        assert abs(mean[s] - (seg.mean() if n else 0.0)) < 1e-10
    for w in (1, 4, 16, 1000):
        mn = oc.trace_confidence(Hs, cu, window=w, mode=1)
        for s, n in enumerate(ell):
            seg = Hs[cu[s]:cu[s + 1]]
            if n == 0:
                assert mn[s] == 0.0
                continue
            ww = min(w, n)
            expect = min(seg[a:a + ww].mean() for a in range(n - ww + 1))
            assert abs(mn[s] - expect) < 1e-10
    # window 1 is the minimum token confidence; a window as long as the trace is the mean
    assert np.allclose(oc.trace_confidence(Hs, cu, window=1, mode=1)[[0, 1, 3]], [Hs[0], Hs[1:6].min(), Hs[6:23].min()])


def test_bottom_tenth_of_the_windows_brute_force():
    """mode 2: mean of the ceil(0.1 n) lowest window means, against a Python sort; hand-worked cases."""
    g = np.random.default_rng(2)
    ell = np.array([1, 9, 10, 11, 0, 25, 137, 64])
    cu = np.concatenate([[0], np.cumsum(ell)])
    Hs = g.random(int(cu[-1])) * 100
    for w in (1, 3, 16, 1000):
        got = oc.trace_confidence(Hs, cu, window=w, mode=2)
        mn = oc.trace_confidence(Hs, cu, window=w, mode=1)
        for s, n in enumerate(ell):
            seg = Hs[cu[s]:cu[s + 1]]
            if n == 0:
                assert got[s] == 0.0
                continue
            ww = min(w, n)
            means = sorted(seg[a:a + ww].mean() for a in range(n - ww + 1))
            k = -(-len(means) // 10)
            assert abs(got[s] - sum(means[:k]) / k) < 1e-10
            assert got[s] >= mn[s] - 1e-12
            if len(means) <= 10:                      # one window in the bottom tenth: the minimum itself
                assert abs(got[s] - mn[s]) < 1e-12
    # by hand: H = 1..20, window 1: 20 windows, bottom 10 % = the two smallest = (1 + 2) / 2
    H = np.arange(1.0, 21.0)[::-1].copy()
    assert oc.trace_confidence(H, np.array([0, 20]), window=1, mode=2)[0] == 1.5
    # window 2 on 1..21 ascending: 20 window means 1.5, 2.5, ...: bottom two average to 2.0
    assert oc.trace_confidence(np.arange(1.0, 22.0), np.array([0, 21]), window=2, mode=2)[0] == 2.0
    # 11 windows -> k = 2 (ceil), not 1 (floor)
    assert oc.trace_confidence(np.arange(1.0, 12.0), np.array([0, 11]), window=1, mode=2)[0] == 1.5
