"""GPU parity of the trace-confidence outputs (Section 3 "Trace Confidence") against the oracle.  H_t = V lse - sum z is
of order V log V: tolerance 2e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from oracle import conf as oc
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import confidence as CF
from paper_2603_24840_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d,V", [(130, 64, 300), (300, 192, 1000), (2000, 128, 4096), (140, 256, 20000), (19200, 64, 512),
                                   (200, 128, 151936)])
def test_token_confidence_and_logprob_from_one_launch(T, d, V):
    ctx = B.Context(0)
    g = np.random.default_rng(T + V)
    H = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    y = g.integers(0, V, size=T).astype(np.int32)
    rows = np.unique(np.concatenate([[0, T - 1], g.integers(0, T, size=60)])).astype(np.int64)
    conf_ref = oc.token_confidence(synth.as_oracle_array(H), synth.as_oracle_array(W), rows=rows, inv_temp=0.8)
    lp_ref, _ = oracle.token_logprob(synth.as_oracle_array(H), synth.as_oracle_array(W), y, rows=rows, inv_temp=0.8)
    logp = torch.empty(T, device="cuda")
    conf = torch.empty(T, device="cuda")
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    CF.arrol_token_logprob_conf(ctx, H.cuda(), W.cuda(), torch.from_numpy(y).cuda(), T, d, V, logp, conf, ws,
                                inv_temperature=0.8)
    torch.cuda.synchronize()
    assert np.abs(conf.cpu().numpy()[rows] - conf_ref).max() <= 2e-5 * np.abs(conf_ref).max()
    assert np.abs(logp.cpu().numpy()[rows] - lp_ref).max() <= 2e-3
    # the plain entry point gives the same log-probs
    logp2 = torch.empty(T, device="cuda")
    B.arrol_token_logprob(ctx, H.cuda(), W.cuda(), torch.from_numpy(y).cuda(), T, d, V, logp2, ws, inv_temperature=0.8)
    torch.cuda.synchronize()
    assert torch.equal(logp, logp2)
    ctx.close()


def test_trace_confidence_matches_oracle():
    ctx = B.Context(0)
    g = np.random.default_rng(3)
    ell = np.concatenate([[1, 0, 5, 17, 300, 2048, 2049, 5000], g.integers(1, 400, size=40)])
    cu = np.concatenate([[0], np.cumsum(ell)]).astype(np.int64)
    S, T = len(ell), int(cu[-1])
    Hs = (g.random(T) * 1e5 + 1e6).astype(np.float32)
    d_num = torch.tensor([S, T], dtype=torch.int64, device="cuda")
    for mode, window in ((0, 1), (1, 1), (1, 16), (1, 2048), (1, 100000), (2, 1), (2, 16), (2, 2048), (2, 100000)):
        ref = oc.trace_confidence(Hs.astype(np.float64), cu, window=window, mode=mode)
        out = torch.full((S,), -1.0, device="cuda")
        CF.arrol_trace_confidence(ctx, torch.from_numpy(Hs).cuda(), torch.from_numpy(cu).cuda(), d_num, S, out,
                                  window=window, mode=mode)
        torch.cuda.synchronize()
        assert np.abs(out.cpu().numpy() - ref).max() <= 1e-6 * np.abs(ref).max()
    with pytest.raises(B.ArrolError) as e:
        CF.arrol_trace_confidence(ctx, out, out, d_num, S, out, mode=3)
    assert e.value.code == -2
    ctx.close()


def test_bottom_tenth_on_long_and_tied_traces():
    """mode 2 beyond the shared-memory prefix (len > 8192) and on values with many exact ties."""
    ctx = B.Context(0)
    g = np.random.default_rng(5)
    ell = np.array([8192, 8193, 20000, 3000, 77])
    cu = np.concatenate([[0], np.cumsum(ell)]).astype(np.int64)
    S, T = len(ell), int(cu[-1])
    Hs = g.integers(0, 4, size=T).astype(np.float32) * 1000.0          # four distinct values: ties everywhere
    Hs[cu[3]:cu[4]] = -g.random(3000).astype(np.float32)                # a negative trace: the key map handles the sign
    d_num = torch.tensor([S, T], dtype=torch.int64, device="cuda")
    for window in (1, 7, 4096):
        ref = oc.trace_confidence(Hs.astype(np.float64), cu, window=window, mode=2)
        out = torch.full((S,), -1.0, device="cuda")
        CF.arrol_trace_confidence(ctx, torch.from_numpy(Hs).cuda(), torch.from_numpy(cu).cuda(), d_num, S, out,
                                  window=window, mode=2)
        torch.cuda.synchronize()
        assert np.abs(out.cpu().numpy() - ref).max() <= 1e-6 * max(np.abs(ref).max(), 1.0)
    ctx.close()


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_trace_count_beyond_the_arrays_is_clamped(mode):
    """d_num[0] larger than S_max: only S_max traces are reduced and nothing past trace_conf[S_max] is written."""
    ctx = B.Context(0)
    g = np.random.default_rng(6)
    ell = g.integers(1, 300, size=12)
    cu = np.concatenate([[0], np.cumsum(ell)]).astype(np.int64)
    S_max, T = len(ell), int(cu[-1])
    Hs = g.random(T).astype(np.float32) * 50
    d_num = torch.tensor([S_max + 1000, T], dtype=torch.int64, device="cuda")     # a stale / oversized count
    out = torch.full((S_max + 64,), -7.0, device="cuda")                          # canaries after the S_max results
    CF.arrol_trace_confidence(ctx, torch.from_numpy(Hs).cuda(), torch.from_numpy(cu).cuda(), d_num, S_max, out,
                              window=16, mode=mode)
    torch.cuda.synchronize()
    ref = oc.trace_confidence(Hs.astype(np.float64), cu, window=16, mode=mode)
    got = out.cpu().numpy()
    assert np.abs(got[:S_max] - ref).max() <= 1e-6 * np.abs(ref).max()
    assert np.all(got[S_max:] == -7.0)
    ctx.close()
