"""Pins for the oracle's selected-token log-probability (Section 3: log pi_theta(o_t | o_<t) from the lm_head)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import synth


def _rand(T, d, V, seed, scale=1.0, wstd=0.2):
    g = np.random.default_rng(seed)
    H = (g.normal(size=(T, d)) * scale).astype(np.float32)
    W = g.normal(0, wstd, size=(V, d)).astype(np.float32)
    y = g.integers(0, V, size=T).astype(np.int32)
    return H, W, y


def test_tiny_vocabulary_probabilities_sum_to_one():
    T, d, V = 6, 24, 37
    H, W, _ = _rand(T, d, V, 0)
    total = np.zeros(T)
    for v in range(V):
        lp, _ = oracle.token_logprob(H, W, np.full(T, v, np.int32))
        total += np.exp(lp)
    assert np.allclose(total, 1.0, rtol=0, atol=1e-12)


def test_uniform_cases_give_minus_log_v():
    T, d, V = 3, 16, 50
    H, W, y = _rand(T, d, V, 1)
    lp, lse = oracle.token_logprob(np.zeros_like(H), W, y)              # zero hidden state: all logits 0
    assert np.allclose(lp, -math.log(V), atol=1e-14) and np.allclose(lse, math.log(V), atol=1e-14)
    Wsame = np.tile(W[:1], (V, 1))                                       # identical vocabulary rows: equal logits
    lp, _ = oracle.token_logprob(H, Wsame, y)
    assert np.allclose(lp, -math.log(V), atol=1e-12)


def test_shift_and_permutation_invariance():
    T, d, V = 5, 16, 64
    H, W, y = _rand(T, d, V, 2)
    H = np.round(H * 8) / 8                       # few mantissa bits: the shifted products stay exact in fp64
    W = np.round(W * 64) / 64
    c = (np.arange(d) % 5 - 2).astype(np.float32)
    lp0, _ = oracle.token_logprob(H.astype(np.float32), W.astype(np.float32), y)
    lp1, _ = oracle.token_logprob(H.astype(np.float32), (W + c).astype(np.float32), y)   # adds H.c to every logit
    assert np.allclose(lp0, lp1, rtol=0, atol=1e-12)
    perm = np.random.default_rng(3).permutation(V)
    inv = np.empty(V, np.int64)
    inv[perm] = np.arange(V)
    lp2, _ = oracle.token_logprob(H.astype(np.float32), W[perm].astype(np.float32), inv[y].astype(np.int32))
    assert np.allclose(lp0, lp2, rtol=0, atol=1e-12)


@pytest.mark.parametrize("scale", [1.0, 30.0])
def test_matches_torch_log_softmax_in_float64(scale):
    T, d, V = 17, 40, 301
    H, W, y = _rand(T, d, V, 4, scale=scale)
    for inv_temp in (1.0, 0.7):
        lp, lse = oracle.token_logprob(H, W, y, inv_temp=inv_temp)
        z = (torch.from_numpy(H).double() @ torch.from_numpy(W).double().T) * inv_temp
        ref = torch.log_softmax(z, -1).gather(1, torch.from_numpy(y).long()[:, None])[:, 0]
        assert np.allclose(lp, ref.numpy(), rtol=0, atol=1e-11)
        assert np.allclose(lse, torch.logsumexp(z, -1).numpy(), rtol=0, atol=1e-11)


def test_two_pass_equals_online_chunked_evaluation():
    # An independent evaluation order: running (max, sum) over vocabulary chunks of any size.
    T, d, V = 4, 32, 500
    H, W, y = _rand(T, d, V, 5, scale=6.0)
    lp, lse = oracle.token_logprob(H, W, y)
    z = H.astype(np.float64) @ W.astype(np.float64).T
    for chunk in (1, 7, 128, 256, 499, 500, 1000):
        for t in range(T):
            m, l = -np.inf, 0.0
            for v0 in range(0, V, chunk):
                zc = z[t, v0:v0 + chunk]
                m_new = max(m, zc.max())
                l = l * math.exp(m - m_new) + np.exp(zc - m_new).sum()
                m = m_new
            assert abs((m + math.log(l)) - lse[t]) < 1e-12
            assert abs(z[t, y[t]] - (m + math.log(l)) - lp[t]) < 1e-12


def test_hand_example_and_ignored_targets():
    # d = 1, H = 1, W = (0, log 2, log 3): probabilities (1, 2, 3) / 6
    W = np.array([[0.0], [math.log(2)], [math.log(3)]], dtype=np.float64)
    H = np.ones((3, 1), dtype=np.float64)
    lp, lse = oracle.token_logprob(H, W, np.array([0, 1, 2], np.int32))
    assert np.allclose(np.exp(lp), [1 / 6, 2 / 6, 3 / 6], atol=1e-15)
    assert np.allclose(lse, math.log(6), atol=1e-15)
    lp, _ = oracle.token_logprob(H, W, np.array([-1, 2, -100], np.int32))
    assert lp[0] == 0.0 and lp[2] == 0.0 and abs(lp[1] - math.log(0.5)) < 1e-15
    # row subset: outputs follow the order of `rows`
    lp, _ = oracle.token_logprob(H, W, np.array([0, 1, 2], np.int32), rows=np.array([2, 0]))
    assert np.allclose(np.exp(lp), [3 / 6, 1 / 6], atol=1e-15)
    # temperature: z / 2 -> probabilities proportional to sqrt
    lp, _ = oracle.token_logprob(H, W, np.array([0, 1, 2], np.int32), inv_temp=0.5)
    s = 1 + math.sqrt(2) + math.sqrt(3)
    assert np.allclose(np.exp(lp), [1 / s, math.sqrt(2) / s, math.sqrt(3) / s], atol=1e-15)


def test_bf16_workload_rows_match_torch():
    w = synth.WORKLOADS["mini"]
    H = synth.hidden_states(w, 50)
    W = synth.vocab_weights(w)
    y = synth.token_ids(w, 50)
    lp, _ = oracle.token_logprob(synth.as_oracle_array(H), synth.as_oracle_array(W), y)
    ref = torch.log_softmax(H.double() @ W.double().T, -1).gather(1, torch.from_numpy(y).long()[:, None])[:, 0]
    assert np.allclose(lp, ref.numpy(), rtol=0, atol=1e-11)
