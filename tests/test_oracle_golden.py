"""The stored fixtures: closed-form values from the paper's formulas, and the oracle's frozen outputs on 'tiny'."""
import importlib.util
import math
import os
from fractions import Fraction

import numpy as np

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _closed_forms():
    out = {}
    for line in open(os.path.join(HERE, "golden", "closed_forms.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = v
    return out


def test_closed_form_fixture():
    cf = _closed_forms()
    q64, _ = oracle.build_q_lut([0, 1, 2, 5], [6, 3, 2, 1], 1.0)
    for b in range(4):
        assert abs(q64[b] - float(Fraction(cf["q_lut_b%d" % b]))) < 1e-15
    a = oracle.advantages(np.array([1, 1, 1, 0, 0, 0, 0, 0], np.float32), np.ones(8, np.uint8), 8, eps=0.0)
    assert abs(a[0] - float(cf["adv_pos_n8_k3"])) < 1e-14 and abs(a[7] - float(cf["adv_neg_n8_k3"])) < 1e-14
    a = oracle.advantages(np.array([1, 0, 0, 0], np.float32), np.ones(4, np.uint8), 4, eps=0.0)
    assert abs(a[0] - float(cf["adv_pos_n4_k1"])) < 1e-14 and abs(a[1] - float(cf["adv_neg_n4_k1"])) < 1e-14
    prob, bins, _ = oracle.prob_map(np.array([math.log(3.0)]), np.zeros(128, np.float32))
    assert abs(prob[0] - float(cf["sigmoid_log3"])) < 1e-15 and bins[0] == int(cf["bin_log3_B128"])


def test_tiny_pipeline_fixture_is_what_the_oracle_computes():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = open(os.path.join(HERE, "golden", "tiny_pipeline.txt")).read()
    now = mod.render(mod.compute())
    s_lines, n_lines = stored.splitlines(), now.splitlines()
    assert len(s_lines) == len(n_lines)
    for a, b in zip(s_lines, n_lines):
        ka, kb = a.split(":")[0], b.split(":")[0]
        assert ka == kb
        if ka in ("score", "adv"):
            va = np.array([float(x) for x in a.split(":")[1].split()])
            vb = np.array([float(x) for x in b.split(":")[1].split()])
            assert np.allclose(va, vb, rtol=0, atol=1e-9)
        else:
            assert a == b
