"""Writes tests/golden/tiny_pipeline.txt from the CPU oracle alone (no CUDA code is imported or run).

The file freezes what the oracle computes on the seeded "tiny" workload, so that an accidental change to the
oracle's arithmetic shows up as a diff.  The paper prints no numeric example for this path; the values stored
here are the oracle's, and the oracle itself is pinned to closed forms and exact arithmetic by the other
CPU tests.  Run:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2603_24840_b200 import synth  # noqa: E402


def compute():
    w = synth.WORKLOADS["tiny"]
    ell, rew = synth.lengths(w), synth.rewards(w)
    hw = synth.head_weights(w)
    x = synth.hidden_states(w, w.N)
    s = oracle.head_score(synth.as_oracle_array(x), synth.as_oracle_array(hw["W1"]), synth.as_oracle_array(hw["b1"]))
    hist_s, hist_y = synth.calib_history(w)
    cpos, cneg = oracle.calib_counts(hist_s, hist_y, w.B)
    _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
    prob, bins, q = oracle.prob_map(s, lut)
    keep = oracle.select(q.astype(np.float32), w.P, w.G, w.K, w.rho)
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    adv = oracle.advantages(rew, keep, w.G)
    return {
        "score": ["%.12e" % v for v in s],
        "bin": [int(b) for b in bins],
        "keep": [int(k) for k in keep],
        "survivor_idx": [int(i) for i in idx],
        "cu_seqlens": [int(c) for c in cu],
        "S_T": [S, T],
        "adv": ["%.12e" % v for v in adv],
    }


def render(vals):
    lines = ["# Oracle outputs on the seeded 'tiny' workload (4 prompts x 8 rollouts, keep 4; Section 4.1-4.3 path).",
             "# Written by tests/golden/make_golden.py, which calls only oracle/."]
    for k, v in vals.items():
        lines.append(k + ": " + " ".join(str(x) for x in v))
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_pipeline.txt")
    with open(out, "w") as f:
        f.write(render(compute()))
    print("wrote", out)
