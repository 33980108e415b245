"""arrol_token_logprob_gathered: the survivors' log-probs with the hidden rows read in place from the pre-prune buffer
(Section 4.3 (ii); Algorithm 1 "log-probs on R'").  Checked against the fp64 oracle (gather, then log-softmax) within
2e-3, and bit for bit against arrol_compact + arrol_token_logprob on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200.pipeline import PruneRebatch, host_inputs

pytestmark = pytest.mark.gpu
LOGP_TOL = 2e-3


def _case(ctx, ell, keep, d, V, seed, pad=0, inv_temp=1.0):
    """Rollout lengths `ell`, keep mask, source rows padded by `pad` unused rows between rollouts."""
    g = np.random.default_rng(seed)
    N = len(ell)
    ell = np.asarray(ell, dtype=np.int32)
    keep = np.asarray(keep, dtype=np.uint8)
    off = np.zeros(N, dtype=np.int64)
    off[1:] = np.cumsum(ell[:-1].astype(np.int64) + pad)
    R = int(off[-1] + ell[-1] + pad)
    X = torch.from_numpy(g.normal(size=(R, d)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    tokens = g.integers(0, V, size=R).astype(np.int32)
    rew = g.integers(0, 2, size=N).astype(np.float32)
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    cap = max(int(ell.sum()), 1)
    dv = lambda a: torch.from_numpy(a).cuda()
    Xd, Wd = X.cuda(), W.cuda()
    o = dict(cu=torch.zeros(N + 1, dtype=torch.int64, device="cuda"), idx=torch.zeros(N, dtype=torch.int32, device="cuda"),
             adv=torch.zeros(N, device="cuda"), num=torch.zeros(2, dtype=torch.int64, device="cuda"),
             dt=torch.zeros(cap, dtype=torch.int32, device="cuda"), dr=torch.zeros((cap, d), dtype=torch.bfloat16, device="cuda"))
    d_off = dv(off)
    B.arrol_compact(ctx, dv(keep), dv(ell), d_off, N, 1, dv(rew), cap, o["cu"], o["idx"], o["adv"], o["num"],
                    src_tokens=dv(tokens), dst_tokens=o["dt"], src_rows=Xd, dst_rows=o["dr"], row_bytes=2 * d)
    ws = torch.empty(B.arrol_token_logprob_gathered_workspace(ctx, N, cap, d, V), dtype=torch.uint8, device="cuda")
    assert ws.numel() == B.arrol_token_logprob_workspace(ctx, cap, d, V) + N * 128 * d * 2
    lp_packed = torch.full((cap,), 7.0, device="cuda")
    lse_packed = torch.full((cap,), 7.0, device="cuda")
    B.arrol_token_logprob(ctx, o["dr"], Wd, o["dt"], cap, d, V, lp_packed, ws, lse=lse_packed, d_T=o["num"][1:],
                          inv_temperature=inv_temp)
    lp = torch.full((cap,), 7.0, device="cuda")
    lse = torch.full((cap,), 7.0, device="cuda")
    B.arrol_token_logprob_gathered(ctx, Xd, Wd, o["dt"], o["cu"], o["idx"], d_off, o["num"], N, cap, d, V, lp, ws, lse=lse,
                                   inv_temperature=inv_temp)
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    assert o["num"].tolist() == [S, T]
    assert torch.equal(lp[:T], lp_packed[:T]) and torch.equal(lse[:T], lse_packed[:T])     # same operands, same order
    assert torch.all(lp[T:] == 7.0)                                                        # rows past T are not written
    if T:
        dt_ref, dr_ref, _ = oracle.gather(idx, cu, off, tokens, synth.as_oracle_array(X))
        rows = np.unique(np.concatenate([[0, T - 1], cu[:-1][cu[:-1] < T], np.maximum(cu[1:] - 1, 0),
                                         g.integers(0, T, size=40)])).astype(np.int64)
        rows = rows[rows < T]
        if len(rows) > 160:
            rows = np.unique(np.concatenate([rows[:60], rows[-60:], g.choice(rows, 40)]))
        lp_ref, lse_ref = oracle.token_logprob(dr_ref.view(np.uint16).reshape(T, d), synth.as_oracle_array(W), dt_ref,
                                               rows=rows, inv_temp=inv_temp)
        assert np.abs(lp.cpu().numpy()[rows] - lp_ref).max() <= LOGP_TOL
        assert np.abs(lse.cpu().numpy()[rows] - lse_ref).max() <= LOGP_TOL


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    assert B.arrol_poll_status(c, raise_on_error=False) == 0
    c.close()


def test_survivor_boundaries_at_every_kind_of_tile_row(ctx):
    """Boundaries at rows 1, 7, 8, 9, 127 of a tile and at the tile edge; runs of 1 ... 300 rows; padded sources."""
    # kept lengths chosen so that the packed boundaries fall at 1, 8, 15, 24, 151(=128+23), 255(=127 of tile 1), 256, ...
    ell = [1, 7, 7, 9, 127, 104, 1, 300, 33, 64, 2, 3, 5, 128, 129, 70]
    keep = [1] * len(ell)
    _case(ctx, ell, keep, d=192, V=700, seed=1)
    _case(ctx, ell, keep, d=64, V=300, seed=2, pad=3)
    # pruned rollouts in between (their rows are skipped), ragged tail
    keep2 = [1, 0, 1, 1, 0, 1, 1, 1, 0, 1, 1, 0, 1, 1, 0, 1]
    _case(ctx, ell, keep2, d=128, V=1000, seed=3, pad=1, inv_temp=0.7)


def test_zero_length_survivors_and_nobody_kept(ctx):
    ell = [0, 40, 0, 0, 130, 0, 17, 0]
    _case(ctx, ell, [1] * 8, d=64, V=513, seed=4)
    _case(ctx, ell, [1, 0, 1, 1, 1, 1, 0, 1], d=64, V=513, seed=5)
    _case(ctx, [10, 20, 30], [0, 0, 0], d=64, V=300, seed=6)            # T = 0: nothing is written
    _case(ctx, [5], [1], d=64, V=300, seed=7)                            # one short survivor: a single partial tile


def test_many_single_token_survivors_in_one_tile(ctx):
    """Runs of one row each: every tile crosses many survivor boundaries."""
    g = np.random.default_rng(8)
    ell = np.concatenate([np.ones(150, dtype=np.int32), g.integers(1, 4, size=100).astype(np.int32)])
    keep = (g.random(len(ell)) < 0.8).astype(np.uint8)
    _case(ctx, ell, keep, d=64, V=300, seed=8, pad=1)


def test_several_tiles_per_block_and_vocabulary_splits(ctx):
    """More token tiles than SMs (persistent blocks walk several items) and the split + combine path."""
    g = np.random.default_rng(9)
    ell = g.integers(100, 700, size=64).astype(np.int32)                 # ~25k tokens = ~200 tiles
    keep = (g.random(64) < 0.75).astype(np.uint8)
    _case(ctx, ell, keep, d=64, V=520, seed=9)
    ell = g.integers(30, 90, size=8).astype(np.int32)                    # few tiles: the vocabulary is split
    _case(ctx, ell, [1] * 8, d=128, V=6000, seed=10)


@pytest.mark.parametrize("name", ["mini", "profile-small"])
def test_pipeline_without_the_hidden_row_plane(name):
    """score -> select -> compact (token ids only) -> gathered log-probs equals the pipeline that packs the rows."""
    w = synth.WORKLOADS[name]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    pr.step()
    torch.cuda.synchronize()
    S, T = pr.counts()
    ref = pr.logp.clone()
    pr.logp.fill_(7.0)
    pr.dst_rows.fill_(0)                                                  # the packed rows are not used below
    pr.prune_step(with_rows=False)
    pr.token_logprob_gathered()
    torch.cuda.synchronize()
    assert pr.counts() == (S, T)
    assert torch.equal(pr.logp[:T], ref[:T])
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()
