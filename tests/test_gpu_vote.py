"""GPU parity of the rank-weighted vote (Section 4.4): winners bit-exact, weights within 1e-6."""
import numpy as np
import pytest
import torch

from oracle import tts
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import voting

pytestmark = pytest.mark.gpu


def test_rank_vote_matches_oracle():
    ctx = B.Context(0)
    g = np.random.default_rng(0)
    for G in (1, 2, 5, 8, 16, 31, 32):
        for P in (1, 37, 1000):
            score = (g.integers(0, 40, size=P * G) / 8 - 2).astype(np.float32)      # logit-like, many ties
            answer = g.integers(-1, 6, size=P * G).astype(np.int32)
            if P > 1:
                answer[:G] = -1
            w_ref, win_ref, ww_ref = tts.rank_vote(score, answer, P, G)
            w = torch.empty(P * G, device="cuda")
            win = torch.full((P,), -9, dtype=torch.int32, device="cuda")
            ww = torch.empty(P, device="cuda")
            voting.arrol_rank_vote(ctx, torch.from_numpy(score).cuda(), torch.from_numpy(answer).cuda(), P, G, w, win, ww)
            torch.cuda.synchronize()
            assert np.array_equal(win.cpu().numpy(), win_ref)
            assert np.abs(w.cpu().numpy() - w_ref).max() <= 1e-6
            assert np.abs(ww.cpu().numpy() - ww_ref).max() <= 1e-5
    with pytest.raises(B.ArrolError) as e:
        voting.arrol_rank_vote(ctx, w, win, 1, 33, w, win, ww)
    assert e.value.code == -2
    ctx.close()
