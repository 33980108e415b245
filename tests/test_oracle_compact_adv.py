"""Pins for the oracle's filter + re-batch step (Section 4.3 (ii); Algorithm 1 "Filter pruned rollouts,
rebatch") and the group-relative advantage on survivors (Section 3)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import synth


def _case(seed, N=40, G=8, lo=1, hi=30, row_bytes=48):
    g = np.random.default_rng(seed)
    ell = g.integers(lo, hi + 1, size=N).astype(np.int32)
    keep = (g.random(N) < 0.5).astype(np.uint8)
    off = synth.src_offsets(ell)
    T_src = int(off[-1])
    tokens = g.integers(0, 1 << 30, size=T_src).astype(np.int32)
    rows = g.integers(0, 256, size=(T_src, row_bytes)).astype(np.uint8)
    return ell, keep, off, tokens, rows


def test_scan_brute_force_and_order():
    for seed in range(5):
        ell, keep, off, tokens, rows = _case(seed)
        idx, cu, S, T = oracle.survivor_scan(keep, ell)
        expect_idx = [i for i in range(len(keep)) if keep[i]]
        assert list(idx) == expect_idx                      # ascending original order
        assert S == len(expect_idx) and T == int(ell[keep == 1].sum())
        assert cu[0] == 0 and list(np.diff(cu)) == [int(ell[i]) for i in expect_idx]
        assert cu.dtype == np.int64 and idx.dtype == np.int32


def test_gather_brute_force_identity_and_checksum():
    for seed in range(5):
        ell, keep, off, tokens, rows = _case(seed)
        idx, cu, S, T = oracle.survivor_scan(keep, ell)
        dt, dr, seq = oracle.gather(idx, cu, off[:-1], tokens, rows)
        exp_t = np.concatenate([tokens[off[i]:off[i] + ell[i]] for i in idx]) if S else np.zeros(0, np.int32)
        exp_r = np.concatenate([rows[off[i]:off[i] + ell[i]] for i in idx]) if S else np.zeros((0, 48), np.uint8)
        exp_s = np.concatenate([np.full(ell[i], s, np.int32) for s, i in enumerate(idx)])
        assert np.array_equal(dt, exp_t) and np.array_equal(dr, exp_r) and np.array_equal(seq, exp_s)
        # byte-sum over the destination = byte-sum over the survivors' source segments
        assert int(dr.astype(np.int64).sum()) == sum(int(rows[off[i]:off[i] + ell[i]].astype(np.int64).sum()) for i in idx)
    # keep everything from a packed source: the identity
    ell, keep, off, tokens, rows = _case(9)
    keep[:] = 1
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    dt, dr, _ = oracle.gather(idx, cu, off[:-1], tokens, rows)
    assert np.array_equal(cu, off) and np.array_equal(dt, tokens) and np.array_equal(dr, rows)
    # keep nothing
    keep[:] = 0
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    assert S == 0 and T == 0 and list(cu) == [0]


def test_gather_from_a_padded_source():
    # padded source: rollout i starts at i * L_max; only its first ell_i rows are real
    g = np.random.default_rng(3)
    N, L = 12, 20
    ell = g.integers(1, L + 1, size=N).astype(np.int32)
    keep = (np.arange(N) % 3 != 1).astype(np.uint8)
    tokens = g.integers(0, 1000, size=N * L).astype(np.int32)
    off = (np.arange(N) * L).astype(np.int64)
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    dt, _, _ = oracle.gather(idx, cu, off, tokens)
    exp = np.concatenate([tokens[i * L:i * L + ell[i]] for i in range(N) if keep[i]])
    assert np.array_equal(dt, exp)


def test_advantage_closed_form_for_binary_rewards():
    # k ones among n kept, ddof = 0, eps -> 0:  A+ = sqrt((n-k)/k),  A- = -sqrt(k/(n-k))
    for n, k in ((8, 3), (4, 1), (16, 8), (8, 7)):
        r = np.array([1.0] * k + [0.0] * (n - k), np.float32)
        a = oracle.advantages(r, np.ones(n, np.uint8), n, eps=0.0)
        assert np.allclose(a[:k], math.sqrt((n - k) / k), atol=1e-14)
        assert np.allclose(a[k:], -math.sqrt(k / (n - k)), atol=1e-14)
        assert abs(a.sum()) < 1e-12
        a1 = oracle.advantages(r, np.ones(n, np.uint8), n, eps=0.0, ddof=1)
        assert np.allclose(a1, a * math.sqrt((n - 1) / n), atol=1e-14)
    a = oracle.advantages(np.array([1, 0, 0, 0, 1, 1, 0, 0], np.float32), np.ones(8, np.uint8), 8, eps=0.0)
    assert np.allclose(a[[0, 1]], [1.2909944487, -0.7745966692], atol=1e-9)
    a = oracle.advantages(np.array([0, 0, 1, 0], np.float32), np.ones(4, np.uint8), 4, eps=0.0)
    assert np.allclose(a[[2, 0]], [1.7320508076, -0.5773502692], atol=1e-9)


def test_advantage_degenerate_groups_are_exactly_zero():
    G = 8
    r = np.array([0] * G + [1] * G + [1, 0] * (G // 2), np.float32)
    keep = np.ones(3 * G, np.uint8)
    a = oracle.advantages(r, keep, G)
    assert np.all(a[:2 * G] == 0.0)                 # all-0 and all-1 groups: no learning signal
    assert np.all(a[2 * G:] != 0.0)
    # a mixed group whose SURVIVORS are all equal degenerates too: statistics are over the kept rollouts only
    keep2 = np.array([1, 0] * (G // 2), np.uint8)
    a2 = oracle.advantages(np.array([1, 0] * (G // 2), np.float32), keep2, G)
    assert a2.shape == (G // 2,) and np.all(a2 == 0.0)
    # one survivor: defined (0) for ddof = 0 and ddof = 1
    one = np.zeros(G, np.uint8)
    one[5] = 1
    for ddof in (0, 1):
        assert list(oracle.advantages(np.ones(G, np.float32), one, G, ddof=ddof)) == [0.0]


def test_advantage_matches_torch_on_survivors_of_real_valued_rewards():
    g = np.random.default_rng(7)
    P, G = 6, 16
    r = g.normal(size=P * G).astype(np.float32)
    keep = (g.random(P * G) < 0.5).astype(np.uint8)
    keep.reshape(P, G)[:, 0] = 1
    for ddof in (0, 1):
        a = oracle.advantages(r, keep, G, eps=1e-6, ddof=ddof)
        exp = []
        for p in range(P):
            rr = torch.from_numpy(r[p * G:(p + 1) * G][keep[p * G:(p + 1) * G] == 1]).double()
            if rr.numel() - ddof <= 0:
                exp += [0.0] * rr.numel()
                continue
            sd = torch.std(rr, correction=ddof)
            exp += list(((rr - rr.mean()) / (sd + 1e-6)).numpy())
        assert np.allclose(a, exp, rtol=0, atol=1e-12)


def test_pipeline_on_the_tiny_workload_keeps_k_per_group():
    w = synth.WORKLOADS["tiny"]
    ell, rew = synth.lengths(w), synth.rewards(w)
    q = np.random.default_rng(0).random(w.N).astype(np.float32)
    keep = oracle.select(q, w.P, w.G, w.K, w.rho)
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    assert S == w.P * w.K
    a = oracle.advantages(rew, keep, w.G)
    assert a.shape == (S,)
    for p in range(w.P):
        assert abs(a[p * w.K:(p + 1) * w.K].sum()) < 1e-5   # zero-mean per group up to the eps in the denominator
