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
