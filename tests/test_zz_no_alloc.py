"""arrol_score_partial_static: the MLP-head scoring entry point for callers that cannot allocate device memory
(frozen memory plans, host applications that own the device heap, latency-critical loops).  It keeps its scratch
in a fixed array inside the library, takes no context and allocates nothing.

Checked here through the C ABI against the regular entry point arrol_score_partial and against the CPU oracle on
the same inputs, three calls in a row with different shapes, so that whatever one call leaves in the shared scratch
cannot leak into the next.  The two entry points run different kernels for a bf16 head (the regular one contracts
on the tensor cores, this one in fp32 on the ordinary ALUs), so scores agree within the scoring tolerance, a bin may
differ by one only next to a bin edge, and q is always the table entry of the call's own bin.
This file sorts last on purpose: a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth

pytestmark = pytest.mark.gpu

PROB_TOL = 1e-3     # the tolerance the other scoring tests use


def _inputs(N, d, h, dtype, seed):
    g = np.random.default_rng(seed)
    mk = lambda std, *s: torch.from_numpy(g.normal(0, std, size=s).astype(np.float32)).to(dtype).cuda()
    x = mk(1.0, 3 * N, d)
    head = {"W1": mk(0.05, h, d), "b1": mk(0.05, h), "w2": mk(0.2, h), "b2": mk(0.05, 1), "h": h}
    ridx = torch.from_numpy(g.permutation(3 * N)[:N].astype(np.int64)).cuda()
    lut = torch.from_numpy(np.sort(g.random(128)).astype(np.float32)).cuda()
    return x, head, ridx, lut


def _outputs(N):
    f = lambda: torch.full((N,), 7.0, device="cuda")
    return f(), f(), f(), torch.full((N,), -5, dtype=torch.int32, device="cuda")


def test_static_entry_matches_the_regular_entry_on_two_calls_in_a_row():
    ctx = B.Context(0)
    try:
        # the second call is smaller in N and wider in h than the first, then a float32 case
        for N, d, h, dtype, seed in ((1500, 512, 256, torch.bfloat16, 1), (333, 264, 512, torch.bfloat16, 2),
                                     (70, 136, 68, torch.float32, 3)):
            x, head, ridx, lut = _inputs(N, d, h, dtype, seed)
            s0, p0, q0, b0 = _outputs(N)
            B.arrol_score_partial(ctx, x, head, N, s0, p0, q0, bin=b0, row_index=ridx, q_lut=lut)
            s1, p1, q1, b1 = _outputs(N)
            B.arrol_score_partial_static(x, head, N, s1, p1, q1, bin=b1, row_index=ridx, q_lut=lut)
            torch.cuda.synchronize()
            assert (s0 - s1).abs().max().item() <= PROB_TOL
            assert (p0 - p1).abs().max().item() <= PROB_TOL
            assert not torch.any(p1 == 7.0)
            # against the fp64 oracle: scores and probabilities within the scoring tolerance
            oa = synth.as_oracle_array
            s_ref = oracle.head_score(oa(x), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]),
                                      row_index=ridx.cpu().numpy(), h=h)
            lut_h = lut.cpu().numpy()
            p_ref, b_ref, _ = oracle.prob_map(s_ref, lut_h)
            assert np.abs(s1.cpu().numpy() - s_ref).max() <= PROB_TOL
            assert np.abs(p1.cpu().numpy() - p_ref).max() <= PROB_TOL
            # bins: the oracle's bin, or its neighbour where 128 s' lies within the tolerance of a bin edge;
            # q is bit-equal to the table entry of the bin this call chose
            bins = b1.cpu().numpy()
            near_edge = np.abs(128 * p_ref - np.rint(128 * p_ref)) <= 128 * PROB_TOL
            assert np.all((bins == b_ref) | (near_edge & (np.abs(bins - b_ref) <= 1)))
            assert np.array_equal(q1.cpu().numpy(), lut_h[bins])
            assert np.array_equal(bins, np.array([oracle.bin_index(float(v), 128) for v in p1.cpu().numpy()]))
            same = b0 == b1
            assert torch.equal(q0[same], q1[same])
            assert np.all(near_edge[(~same).cpu().numpy()])          # the two entry points differ only next to an edge
    finally:
        ctx.close()


def test_static_entry_rejects_sizes_beyond_its_fixed_scratch():
    x, head, ridx, lut = _inputs(64, 64, 64, torch.bfloat16, 4)
    s, p, q, b = _outputs(5000)
    with pytest.raises(B.ArrolError) as e:
        B.arrol_score_partial_static(x, head, 4097, s, p, q)                 # N > 4096
    assert e.value.code == -2
    big = dict(head, h=516)
    with pytest.raises(B.ArrolError) as e:
        B.arrol_score_partial_static(x, big, 64, s, p, q)                    # h > 512
    assert e.value.code == -2
    with pytest.raises(B.ArrolError) as e:
        B.arrol_score_partial_static(x, dict(head, h=0), 64, s, p, q)        # linear head: not this entry point
    assert e.value.code == -1
    B.arrol_score_partial_static(x, head, 0, s, p, q)                        # N = 0: no-op
