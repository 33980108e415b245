"""Pins for the oracle's quality head, score normalisation and binned posterior (Section 4.2, Appendix A.4).

The oracle is checked against things other than itself: exact rational arithmetic, closed forms, special
cases with a known answer and torch's float64 library routines.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import synth


def _bf16_bits(x):
    return synth.as_oracle_array(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def _bf16_vals(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).double().numpy()


def test_linear_head_is_the_exact_dot_product():
    g = np.random.default_rng(0)
    N, d = 7, 193
    x = g.normal(size=(N, d)).astype(np.float32)
    w = g.normal(0, 0.02, size=d).astype(np.float32)
    b = g.normal(0, 0.02, size=1).astype(np.float32)
    s = oracle.head_score(x, w, b1=b)
    for i in range(N):
        exact = sum(Fraction(float(w[k])) * Fraction(float(x[i, k])) for k in range(d)) + Fraction(float(b[0]))
        assert abs(s[i] - float(exact)) < 1e-13
    # two more summation orders: reversed, and math.fsum (correctly rounded)
    for i in range(N):
        prods = [float(w[k]) * float(x[i, k]) for k in range(d)] + [float(b[0])]
        assert abs(s[i] - math.fsum(prods)) < 1e-13
        assert abs(s[i] - sum(reversed(prods))) < 1e-13


def test_linear_head_basis_vectors_and_bias():
    d = 16
    w = np.arange(1, d + 1, dtype=np.float32) / 8
    b = np.array([0.25], dtype=np.float32)
    x = np.eye(d, dtype=np.float32)
    s = oracle.head_score(x, w, b1=b)
    assert np.array_equal(s, w.astype(np.float64) + 0.25)       # x = e_k picks w_k, exactly
    assert np.array_equal(oracle.head_score(x, w), w.astype(np.float64))  # NULL bias = 0
    # a transposed or mis-strided operand would fail this: row_index and row_stride are honoured
    big = np.zeros((5, 2 * d), dtype=np.float32)
    big[3, :d] = x[2]
    s2 = oracle.head_score(big.reshape(-1)[: 5 * 2 * d].reshape(5, 2 * d)[:, :d].copy(), w)
    assert s2[3] == w[2]
    s3 = oracle.head_score(big.reshape(10, d), w, row_index=np.array([6], dtype=np.int64))
    assert s3[0] == w[2]


def test_bf16_inputs_are_widened_exactly():
    g = np.random.default_rng(1)
    N, d = 5, 64
    x = g.normal(size=(N, d))
    w = g.normal(0, 0.02, size=d)
    s = oracle.head_score(_bf16_bits(x), _bf16_bits(w))
    ref = torch.from_numpy(_bf16_vals(x)) @ torch.from_numpy(_bf16_vals(w))
    assert np.allclose(s, ref.numpy(), rtol=0, atol=1e-13)


def test_mlp_head_matches_torch_float64_library_ops():
    g = np.random.default_rng(2)
    N, d, h = 9, 80, 12
    x = g.normal(size=(N, d)).astype(np.float32)
    W1 = g.normal(0, 0.3, size=(h, d)).astype(np.float32)
    b1 = g.normal(0, 0.3, size=h).astype(np.float32)
    w2 = g.normal(0, 0.3, size=h).astype(np.float32)
    b2 = g.normal(0, 0.3, size=1).astype(np.float32)
    s = oracle.head_score(x, W1, b1, w2, b2, h=h)
    t = lambda a: torch.from_numpy(a).double()
    u = torch.nn.functional.linear(t(x), t(W1), t(b1))
    ref = torch.nn.functional.gelu(u, approximate="none") @ t(w2) + t(b2)
    assert np.allclose(s, ref.numpy(), rtol=0, atol=1e-12)
    # the tanh approximation is a different function: the oracle must not be it
    ref_tanh = torch.nn.functional.gelu(u, approximate="tanh") @ t(w2) + t(b2)
    assert np.abs(s - ref_tanh.numpy()).max() > 1e-6


def test_mlp_head_reduces_to_linear_for_large_preactivations():
    # W1 rows = unit vectors, b1 = 40: GELU(u) = u to below 1e-300 for u >= 30, so s = w2.(x + 40) + b2.
    d = h = 8
    g = np.random.default_rng(3)
    x = (g.integers(-64, 65, size=(4, d)) / 64).astype(np.float32)   # x + 40 stays exact in binary32
    W1 = np.eye(d, dtype=np.float32)
    b1 = np.full(h, 40.0, dtype=np.float32)
    w2 = g.normal(size=h).astype(np.float32)
    b2 = np.array([0.5], dtype=np.float32)
    s = oracle.head_score(x, W1, b1, w2, b2, h=h)
    lin = oracle.head_score(x + 40.0, w2, b1=b2)
    assert np.allclose(s, lin, rtol=0, atol=1e-12)
    # and GELU(0) = 0, GELU(-40) = 0: zero / very negative pre-activations contribute nothing
    s0 = oracle.head_score(np.zeros((1, d), np.float32), W1, np.full(h, -40.0, np.float32), w2, b2, h=h)
    assert abs(s0[0] - 0.5) < 1e-300 or s0[0] == 0.5


def test_sigmoid_closed_forms_and_bin_edges():
    prob, bins, q = oracle.prob_map(np.array([0.0, 3.0, -3.0, 800.0, -800.0, math.log(3.0)]))
    assert prob[0] == 0.5
    assert abs(prob[1] + prob[2] - 1.0) < 1e-15            # sigmoid(-s) = 1 - sigmoid(s)
    assert prob[3] == 1.0 and prob[4] == 0.0
    assert abs(prob[5] - 0.75) < 1e-15                     # sigmoid(log 3) = 3/4
    assert np.array_equal(q, prob)                         # no table: q = s'
    ref = torch.sigmoid(torch.tensor([0.0, 3.0, -3.0, 800.0, -800.0, math.log(3.0)], dtype=torch.float64))
    assert np.allclose(prob, ref.numpy(), rtol=0, atol=1e-15)
    # b(s') = min(B-1, floor(B s')): s' = 1 lands in the last bin, edges belong to the upper bin
    B = 128
    assert oracle.bin_index(1.0, B) == B - 1
    assert oracle.bin_index(0.0, B) == 0
    assert oracle.bin_index(0.5, B) == 64
    assert oracle.bin_index(np.nextafter(0.5, 0), B) == 63
    assert oracle.bin_index(127 / 128, B) == 127
    lut = np.arange(B, dtype=np.float32) / 256
    prob, bins, q = oracle.prob_map(np.array([0.0, 800.0, -800.0, math.log(3.0)]), lut)
    assert list(bins) == [64, 127, 0, 96]
    assert np.array_equal(q, lut[bins].astype(np.float64))


def _exact_lut(cpos, cneg, alpha):
    B = len(cpos)
    npos, nneg = sum(cpos), sum(cneg)
    pi = Fraction(npos, npos + nneg) if npos + nneg else Fraction(1, 2)
    out = []
    for b in range(B):
        p1 = (Fraction(cpos[b]) + alpha) / (npos + alpha * B)
        p0 = (Fraction(cneg[b]) + alpha) / (nneg + alpha * B)
        out.append(pi * p1 / (pi * p1 + (1 - pi) * p0))
    return out


def test_q_lut_worked_example_in_exact_rationals():
    # B = 4, alpha = 1, c+ = (0,1,2,5), c- = (6,3,2,1): pi = 8/20 and, by hand,
    # q_0 = (2/5 * 1/12) / (2/5 * 1/12 + 3/5 * 7/16) = 8/71, etc.
    cpos, cneg = [0, 1, 2, 5], [6, 3, 2, 1]
    exact = _exact_lut(cpos, cneg, Fraction(1))
    assert exact[0] == Fraction(8, 71)
    q64, q32 = oracle.build_q_lut(cpos, cneg, 1.0)
    assert np.allclose(q64, [float(e) for e in exact], rtol=0, atol=1e-15)
    assert np.allclose(q64, [0.112676, 0.307692, 0.470588, 0.727273], atol=5e-7)
    assert np.array_equal(q32, q64.astype(np.float32))


def test_q_lut_closed_forms():
    g = np.random.default_rng(4)
    c = g.integers(0, 50, size=16)
    q64, _ = oracle.build_q_lut(c, c, 1.0)          # identical histograms: the score says nothing, q = pi = 1/2
    assert np.allclose(q64, 0.5, atol=1e-15)
    c2 = 3 * c                                       # proportional histograms differ only through smoothing
    q64, _ = oracle.build_q_lut(c, c2, 0.0 + 1e-300)
    npos, nneg = c.sum(), c2.sum()
    assert np.allclose(q64[c > 0], npos / (npos + nneg), atol=1e-12)
    q64, _ = oracle.build_q_lut([7], [21], 1.0)      # B = 1: q = pi
    assert abs(q64[0] - 0.25) < 1e-15
    q64, _ = oracle.build_q_lut([0, 0], [0, 0], 1.0)  # empty buffers: pi = 1/2, flat
    assert np.allclose(q64, 0.5)
    # random histograms against exact rationals; alpha = 1/2 as well
    for alpha in (Fraction(1), Fraction(1, 2)):
        cp = [int(v) for v in g.integers(0, 30, size=9)]
        cn = [int(v) for v in g.integers(0, 30, size=9)]
        q64, _ = oracle.build_q_lut(cp, cn, float(alpha))
        assert np.allclose(q64, [float(e) for e in _exact_lut(cp, cn, alpha)], rtol=0, atol=1e-15)
    # a posterior is monotone in the likelihood ratio: more positives in a bin raises q there
    cp, cn = [5, 5, 5, 5], [5, 5, 5, 5]
    base, _ = oracle.build_q_lut(cp, cn, 1.0)
    cp[2] += 10
    up, _ = oracle.build_q_lut(cp, cn, 1.0)
    assert up[2] > base[2]


def test_calib_counts_brute_force():
    w = synth.WORKLOADS["tiny"]
    s, y = synth.calib_history(w, 2000)
    B = 128
    cpos, cneg = oracle.calib_counts(s, y, B)
    assert cpos.sum() == int(y.sum()) and cneg.sum() == int((1 - y).sum())
    bp = np.zeros(B, dtype=np.int64)
    bn = np.zeros(B, dtype=np.int64)
    for sk, yk in zip(s, y):
        b = min(B - 1, int(Fraction(float(sk)) * B))   # exact floor of B * s'
        (bp if yk else bn)[b] += 1
    assert np.array_equal(cpos, bp) and np.array_equal(cneg, bn)
    cpos, cneg = oracle.calib_counts(np.array([1.0, 0.0, 0.999999]), np.array([1, 0, 1], np.uint8), 4)
    assert list(cpos) == [0, 0, 0, 2] and list(cneg) == [1, 0, 0, 0]


@pytest.mark.parametrize("name", ["tiny", "mini"])
def test_head_on_workload_shapes_matches_torch(name):
    w = synth.WORKLOADS[name]
    hw = synth.head_weights(w)
    x = synth.hidden_states(w, w.N)
    arrs = {k: (None if v is None else synth.as_oracle_array(v)) for k, v in hw.items()}
    s = oracle.head_score(synth.as_oracle_array(x), arrs["W1"], arrs["b1"], arrs["w2"], arrs["b2"], h=w.h)
    xd = x.double()
    if w.h == 0:
        ref = xd @ hw["W1"].double() + hw["b1"].double()
    else:
        u = torch.nn.functional.linear(xd, hw["W1"].double(), hw["b1"].double())
        ref = torch.nn.functional.gelu(u) @ hw["w2"].double() + hw["b2"].double()
    assert np.allclose(s, ref.numpy(), rtol=0, atol=1e-12)
