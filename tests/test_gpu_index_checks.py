"""Index checks on request (arrol_set_source_rows): an out-of-range row number or source offset is reported through
the status word and the access is skipped, never followed.  The indices used here point far outside the buffers, so
the test passes only if the kernels really do not dereference them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth

pytestmark = pytest.mark.gpu

BAD_INDEX = 16


@pytest.mark.parametrize("h,dtype", [(0, torch.bfloat16), (0, torch.float32), (64, torch.bfloat16), (32, torch.float32)])
def test_scoring_skips_rows_outside_the_source(h, dtype):
    ctx = B.Context(0)
    g = np.random.default_rng(h + 1)
    N, d, R = 200, 128, 300
    x = torch.from_numpy(g.normal(size=(R, d)).astype(np.float32)).to(dtype)
    mk = lambda *s: torch.from_numpy(g.normal(0, 0.05, size=s).astype(np.float32)).to(dtype)
    head = {"W1": mk(d) if h == 0 else mk(h, d), "b1": mk(1) if h == 0 else mk(h), "w2": None if h == 0 else mk(h),
            "b2": None if h == 0 else mk(1)}
    ridx = g.integers(0, R, size=N).astype(np.int64)
    bad = np.array([3, 77, 199])
    ridx_bad = ridx.copy()
    ridx_bad[bad] = [R, -1, 1 << 40]
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    s_ref = oracle.head_score(oa(x), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]), row_index=ridx, h=h)
    zero_ref = oracle.head_score(oa(torch.zeros(1, d, dtype=dtype)), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]),
                                 oa(head["b2"]), h=h)[0]
    dhead = {k: (None if v is None else v.cuda()) for k, v in head.items()}
    dhead["h"] = h
    out = [torch.full((N,), 7.0, device="cuda") for _ in range(3)]
    B.arrol_set_source_rows(ctx, R)
    B.arrol_score_partial(ctx, x.cuda(), dhead, N, out[0], out[1], out[2], row_index=torch.from_numpy(ridx).cuda())
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0                 # all in range: nothing recorded
    assert np.abs(out[0].cpu().numpy() - s_ref).max() <= 1e-3
    B.arrol_score_partial(ctx, x.cuda(), dhead, N, out[0], out[1], out[2], row_index=torch.from_numpy(ridx_bad).cuda())
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == BAD_INDEX
    s = out[0].cpu().numpy()
    good = np.setdiff1d(np.arange(N), bad)
    assert np.abs(s[good] - s_ref[good]).max() <= 1e-3
    assert np.abs(s[bad] - zero_ref).max() <= 1e-3                            # scored as a zero row
    ctx.close()


def test_compaction_gathers_nothing_when_a_kept_rollout_leaves_the_source():
    ctx = B.Context(0)
    g = np.random.default_rng(9)
    P, G = 6, 4
    N = P * G
    ell = g.integers(1, 40, size=N).astype(np.int32)
    off = synth.src_offsets(ell)
    R = int(off[-1])
    keep = (g.random(N) < 0.5).astype(np.uint8)
    keep[5] = 1
    tokens = g.integers(0, 1000, size=R).astype(np.int32)
    rows = torch.from_numpy(g.integers(0, 255, size=(R, 32)).astype(np.uint8))
    rew = g.integers(0, 2, size=N).astype(np.float32)
    cap = int(ell.sum())
    dv = lambda a: torch.from_numpy(a).cuda()

    def run(offsets, with_rows):
        outs = dict(cu=torch.zeros(N + 1, dtype=torch.int64, device="cuda"), idx=torch.zeros(N, dtype=torch.int32, device="cuda"),
                    adv=torch.zeros(N, device="cuda"), num=torch.zeros(2, dtype=torch.int64, device="cuda"),
                    dt=torch.full((cap,), -9, dtype=torch.int32, device="cuda"),
                    dr=torch.full((cap, 32), 201, dtype=torch.uint8, device="cuda"))
        B.arrol_compact(ctx, dv(keep), dv(ell), dv(offsets), N, G, dv(rew), cap, outs["cu"], outs["idx"], outs["adv"],
                        outs["num"], src_tokens=dv(tokens), dst_tokens=outs["dt"],
                        src_rows=rows.cuda() if with_rows else None, dst_rows=outs["dr"] if with_rows else None,
                        row_bytes=32 if with_rows else 0)
        torch.cuda.synchronize()
        return outs

    idx_ref, cu_ref, S, T = oracle.survivor_scan(keep, ell)
    B.arrol_set_source_rows(ctx, R)
    for with_rows in (False, True):
        o = run(off[:-1].copy(), with_rows)
        assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
        dt_ref, _, _ = oracle.gather(idx_ref, cu_ref, off[:-1], tokens)
        assert np.array_equal(o["dt"].cpu().numpy()[:T], dt_ref)
        bad_off = off[:-1].copy()
        bad_off[5] = R - int(ell[5]) + 1                                       # one row past the end of the source
        o = run(bad_off, with_rows)
        assert B.arrol_poll_status(ctx, raise_on_error=False) == BAD_INDEX
        assert o["num"].tolist() == [S, T]                                     # the scan outputs are still written
        assert np.array_equal(o["idx"].cpu().numpy()[:S], idx_ref)
        assert torch.all(o["dt"] == -9) and torch.all(o["dr"] == 201)          # nothing was gathered
        far = off[:-1].copy()
        far[5] = 1 << 45                                                       # far outside: must not be dereferenced
        o = run(far, with_rows)
        assert B.arrol_poll_status(ctx, raise_on_error=False) == BAD_INDEX
        assert torch.all(o["dt"] == -9) and torch.all(o["dr"] == 201)
        o = run(off[:-1].copy(), with_rows)                                    # the gate word clears on the next good call
        assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
        assert np.array_equal(o["dt"].cpu().numpy()[:T], dt_ref)
    # a pruned rollout may point anywhere: it is never read
    pr_off = off[:-1].copy()
    pruned = int(np.flatnonzero(keep == 0)[0])
    pr_off[pruned] = 1 << 45
    o = run(pr_off, False)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    ctx.close()
