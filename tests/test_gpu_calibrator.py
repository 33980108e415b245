"""GPU parity of the online calibrator and the stochastic pruning rule (Appendix A.4) against the oracle: ring
contents, counts, posterior table and delta bit for bit; keep decisions bit for bit; p within 1e-6."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import calibrator as CAL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("n_bins,cap,sizes", [
    (128, 8192, [2048, 4096, 1000, 4096, 4096, 37]),       # fills, then wraps
    (128, 64, [10, 0, 100, 500, 3, 64, 65]),                # pushes larger than the ring
    (16, 5, [1, 1, 1, 1, 1, 1, 7, 2000]),
    (4, 1000, [3000]),
])
def test_calibrator_update_matches_oracle(ctx, n_bins, cap, sizes):
    g = np.random.default_rng(n_bins + cap)
    cal = CAL.Calibrator(ctx, n_bins, cap, alpha=1.0)
    buf = oracle.ScoreBuffers(cap)
    sp = CAL.survival(0.5, 0.5, 0.5, 0.05, 0.95)
    snap = cal.snapshot()
    assert snap["delta"] == 0.0 and np.all(snap["q_lut"] == 0.5) and len(snap["pos"]) == 0
    for step, n in enumerate(sizes):
        prob = g.beta(2, 2, size=n).astype(np.float32)                 # fp32 s' as the scoring kernel emits it
        rew = (g.random(n) < prob).astype(np.float32)
        mask = (g.random(n) < 0.7).astype(np.uint8) if step % 2 else None
        bins = np.array([oracle.bin_index(float(v), n_bins) for v in prob], dtype=np.int32)
        cal.update(torch.from_numpy(bins).cuda(), torch.from_numpy(rew).cuda(), sp,
                   mask=None if mask is None else torch.from_numpy(mask).cuda())
        sel = np.ones(n, bool) if mask is None else mask.astype(bool)
        buf.push(prob[sel].astype(np.float64), rew[sel] > 0.5)
        torch.cuda.synchronize()
        snap = cal.snapshot()
        pos, neg = buf.contents()
        bin_of = lambda arr: np.array([oracle.bin_index(float(v), n_bins) for v in arr], dtype=np.int64)
        assert np.array_equal(snap["pos"], bin_of(pos)) and np.array_equal(snap["neg"], bin_of(neg))   # FIFO order
        cpos, cneg = buf.counts(n_bins)
        assert np.array_equal(snap["cpos"], cpos) and np.array_equal(snap["cneg"], cneg)
        _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
        assert np.array_equal(snap["q_lut"], lut)                                                      # bit-equal
        delta = oracle.solve_delta(cpos, cneg, lut, 0.5, 0.5, 0.5, 0.05, 0.95, iters=64)
        assert snap["delta"] == delta                                                                  # bit-equal
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0


def test_delta_is_bit_equal_over_many_states_and_parameters(ctx):
    """delta decides by comparisons that turn on the last bits near convergence: many random buffer states, skewed
    score distributions and survival parameters, every one bit for bit."""
    g = np.random.default_rng(77)
    params = [(0.5, 0.5, 0.5, 0.05, 0.95), (0.25, 1.0, 0.3, 0.0, 1.0), (0.75, 0.2, 0.6, 0.1, 0.9), (0.5, 0.0, 0.5, 0.0, 1.0),
              (0.9, 2.0, 0.5, 0.05, 0.95), (0.1, 0.5, 0.9, 0.0, 0.5)]
    for case in range(36):
        kappa, lam, rho, pmin, pmax = params[case % len(params)]
        n_bins = [128, 128, 16, 64, 5, 128][case % 6]
        cap = [8192, 300, 64, 1000, 50, 2048][(case // 2) % 6]
        cal = CAL.Calibrator(ctx, n_bins, cap, alpha=1.0)
        buf = oracle.ScoreBuffers(cap)
        sp = CAL.survival(kappa, lam, rho, pmin, pmax)
        a, b = [(2, 2), (0.5, 0.5), (8, 1), (1, 8), (5, 5), (0.3, 3)][case % 6]
        for n in (int(g.integers(1, 3000)), int(g.integers(1, 500))):
            prob = g.beta(a, b, size=n).astype(np.float32)
            rew = (g.random(n) < prob ** [1.0, 0.3, 3.0][case % 3]).astype(np.float32)
            bins = np.array([oracle.bin_index(float(v), n_bins) for v in prob], dtype=np.int32)
            cal.update(torch.from_numpy(bins).cuda(), torch.from_numpy(rew).cuda(), sp)
            buf.push(prob.astype(np.float64), rew > 0.5)
            torch.cuda.synchronize()
            cpos, cneg = buf.counts(n_bins)
            _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
            delta = oracle.solve_delta(cpos, cneg, lut, kappa, lam, rho, pmin, pmax, iters=64)
            assert cal.snapshot()["delta"] == delta, (case, n)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0


def test_stochastic_selection_matches_oracle(ctx):
    g = np.random.default_rng(5)
    N = 100003
    q = g.beta(0.6, 0.6, size=N).astype(np.float32)
    u = g.random(N).astype(np.float32)
    elig = (g.random(N) < 0.9).astype(np.uint8)
    for delta, (kappa, lam, rho, pmin, pmax) in ((0.0371, (0.5, 0.5, 0.5, 0.05, 0.95)), (-0.2, (0.25, 1.0, 0.3, 0.0, 1.0))):
        keep_ref, p_ref = oracle.select_stochastic(q, u, delta, elig, kappa, lam, rho, pmin, pmax)
        sp = CAL.survival(kappa, lam, rho, pmin, pmax)
        keep = torch.full((N,), 9, dtype=torch.uint8, device="cuda")
        p = torch.empty(N, device="cuda")
        d_delta = torch.tensor([delta], dtype=torch.float64, device="cuda")
        CAL.arrol_select_stochastic(ctx, torch.from_numpy(q).cuda(), torch.from_numpy(u).cuda(), keep, sp,
                                    d_delta=d_delta, eligible=torch.from_numpy(elig).cuda(), p_out=p)
        torch.cuda.synchronize()
        assert np.array_equal(keep.cpu().numpy(), keep_ref)
        assert np.abs(p.cpu().numpy() - p_ref).max() <= 1e-6
        keep2 = torch.empty_like(keep)
        CAL.arrol_select_stochastic(ctx, torch.from_numpy(q).cuda(), torch.from_numpy(u).cuda(), keep2, sp, delta=delta,
                                    eligible=torch.from_numpy(elig).cuda())
        assert torch.equal(keep, keep2)                                  # host-supplied delta: same decisions


def test_calibrated_loop_feeds_scoring_and_compaction(ctx):
    """Table and delta stay on the device: calibrator -> arrol_score_partial (q_lut view) -> stochastic selection
    (delta view) -> arrol_compact with a variable number of survivors per group."""
    g = np.random.default_rng(6)
    P, G, d, nb = 40, 16, 256, 128
    N = P * G
    cal = CAL.Calibrator(ctx, nb, 4096)
    sp = CAL.survival()
    hist_p = g.beta(2, 2, size=3000).astype(np.float32)
    hist_b = np.array([oracle.bin_index(float(v), nb) for v in hist_p], np.int32)
    hist_y = (g.random(3000) < hist_p).astype(np.float32)
    cal.update(torch.from_numpy(hist_b).cuda(), torch.from_numpy(hist_y).cuda(), sp)
    x = torch.from_numpy(g.normal(size=(N, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    head = {"W1": torch.from_numpy(g.normal(0, 0.06, size=d).astype(np.float32)).to(torch.bfloat16).cuda(),
            "b1": None, "w2": None, "b2": None, "h": 0}
    score, prob, q = (torch.empty(N, device="cuda") for _ in range(3))
    bins = torch.empty(N, dtype=torch.int32, device="cuda")
    B.arrol_score_partial(ctx, x, head, N, score, prob, q, bin=bins, q_lut=cal.q_lut)
    u = torch.from_numpy(g.random(N).astype(np.float32)).cuda()
    keep = torch.empty(N, dtype=torch.uint8, device="cuda")
    CAL.arrol_select_stochastic(ctx, q, u, keep, sp, d_delta=cal.delta)
    torch.cuda.synchronize()
    snap = cal.snapshot()
    assert np.array_equal(q.cpu().numpy(), snap["q_lut"][bins.cpu().numpy()])
    keep_ref, _ = oracle.select_stochastic(q.cpu().numpy(), u.cpu().numpy(), snap["delta"])
    assert np.array_equal(keep.cpu().numpy(), keep_ref)
    ell = g.integers(1, 50, size=N).astype(np.int32)
    rew = (g.random(N) < 0.4).astype(np.float32)
    off = np.concatenate([[0], np.cumsum(ell)[:-1]]).astype(np.int64)
    tokens = g.integers(0, 1000, size=int(ell.sum())).astype(np.int32)
    idx, cu, S, T = oracle.survivor_scan(keep_ref, ell)
    outs = dict(cu=torch.empty(N + 1, dtype=torch.int64, device="cuda"), idx=torch.empty(N, dtype=torch.int32, device="cuda"),
                adv=torch.empty(N, device="cuda"), num=torch.empty(2, dtype=torch.int64, device="cuda"))
    dst = torch.empty(max(T, 1), dtype=torch.int32, device="cuda")
    dv = lambda a: torch.from_numpy(a).cuda()
    B.arrol_compact(ctx, keep, dv(ell), dv(off), N, G, dv(rew), T, outs["cu"], outs["idx"], outs["adv"], outs["num"],
                    src_tokens=dv(tokens), dst_tokens=dst)
    torch.cuda.synchronize()
    assert outs["num"].cpu().tolist() == [S, T]
    dt_ref, _, _ = oracle.gather(idx, cu, off, tokens)
    assert np.array_equal(dst.cpu().numpy()[:T], dt_ref)
    adv_ref = oracle.advantages(rew, keep_ref, G)
    assert np.abs(outs["adv"].cpu().numpy()[:S] - adv_ref).max() <= 1e-5
    counts = keep_ref.reshape(P, G).sum(1)
    assert counts.min() < counts.max()                                   # ragged groups were exercised


def test_update_with_another_shape_leaves_the_state_untouched(ctx):
    """The state was initialised with (B, cap); an update that names another pair, or a state that was never
    initialised, is reported through the status word and changes nothing."""
    cal = CAL.Calibrator(ctx, 128, 256)
    sp = CAL.survival()
    bins = torch.arange(50, dtype=torch.int32, device="cuda")
    rew = (torch.arange(50, device="cuda") % 2).float()
    cal.update(bins, rew, sp)
    torch.cuda.synchronize()
    good = cal.state.clone()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    for n_bins, cap in ((64, 256), (128, 512)):
        B._check(CAL._lib().arrol_calib_update(ctx.handle, B._ptr(cal.state), n_bins, cap, B._ptr(bins), B._ptr(rew),
                                               None, 50, CAL.C.byref(sp), B._stream()), "arrol_calib_update")
        torch.cuda.synchronize()
        assert B.arrol_poll_status(ctx, raise_on_error=False) == 8          # ARROL_DEV_BAD_STATE
        assert torch.equal(cal.state, good)
    raw = torch.zeros(CAL.arrol_calib_state_bytes(128, 256), dtype=torch.uint8, device="cuda")   # never initialised
    B._check(CAL._lib().arrol_calib_update(ctx.handle, B._ptr(raw), 128, 256, B._ptr(bins), B._ptr(rew), None, 50,
                                           CAL.C.byref(sp), B._stream()), "arrol_calib_update")
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 8
    assert not raw.any()
    cal.update(bins, rew, sp)                                                # the right pair still works
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
