"""arrol_prune_rebatch_host (the whole step from host buffers, uploads overlapped with the log-prob kernel) against
the oracle and against the device-resident path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200.pipeline import PruneRebatch, host_inputs

pytestmark = pytest.mark.gpu


def _host_step(pr, w):
    N, cap = w.N, pr.cap
    pin = lambda t: t.cpu().pin_memory()
    h = {"h_hidden": pin(pr.src_rows), "h_src_tokens": pin(pr.src_tokens), "h_lengths": pin(pr.lengths),
         "h_src_tok_off": pin(pr.src_tok_off), "h_rewards": pin(pr.rewards),
         "h_logp": torch.full((cap,), 7.0).pin_memory(), "h_adv": torch.empty(N).pin_memory(),
         "h_cu_seqlens": torch.empty(N + 1, dtype=torch.int64).pin_memory(),
         "h_survivor_idx": torch.empty(N, dtype=torch.int32).pin_memory(),
         "h_num": torch.empty(2, dtype=torch.int64).pin_memory()}
    z = lambda t: torch.zeros_like(t)
    dv = {"W_vocab": pr.W_vocab, "d_hidden": torch.zeros((N, w.d), dtype=torch.bfloat16, device="cuda"),
          "d_lengths": z(pr.lengths), "d_src_tok_off": z(pr.src_tok_off), "d_rewards": z(pr.rewards),
          "d_score": z(pr.score), "d_prob": z(pr.prob), "d_q": z(pr.q), "d_keep": z(pr.keep),
          "d_survivor_idx": z(pr.survivor_idx), "d_cu_seqlens": z(pr.cu_seqlens), "d_adv": z(pr.adv),
          "d_num": z(pr.d_num), "d_dst_tokens": z(pr.dst_tokens), "d_dst_rows": z(pr.dst_rows), "d_logp": z(pr.logp),
          "d_workspace": torch.empty_like(pr.workspace)}
    scal = dict(P=w.P, G=w.G, K=w.K, cutoff=w.cutoff, d=w.d, V=w.V, ddof=0, rho=w.rho, eps=1e-6, inv_temperature=1.0,
                T_src=pr.T_src, dst_capacity_tokens=cap)
    head = {k: (v.to(torch.bfloat16) if torch.is_tensor(v) else v) for k, v in pr.head.items()}
    tensors = dict(h)
    tensors.update(dv)
    step = B.make_host_step(scal, head, pr.q_lut, tensors)
    B.arrol_prune_rebatch_host(pr.ctx, step)
    return h, dv, (head, tensors)


@pytest.mark.parametrize("name", ["mini", "profile-small"])
def test_host_step_matches_device_path_and_oracle(name):
    w = synth.WORKLOADS[name]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    pr.step()
    torch.cuda.synchronize()
    S, T = pr.counts()
    h, dv, _keepalive = _host_step(pr, w)
    assert h["h_num"].tolist() == [S, T]
    assert torch.equal(dv["d_keep"], pr.keep)
    assert torch.equal(h["h_survivor_idx"][:S], pr.survivor_idx.cpu()[:S])
    assert torch.equal(h["h_cu_seqlens"][:S + 1], pr.cu_seqlens.cpu()[:S + 1])
    assert torch.equal(h["h_adv"][:S], pr.adv.cpu()[:S])
    assert torch.equal(dv["d_dst_tokens"][:T], pr.dst_tokens[:T])
    assert torch.equal(dv["d_dst_rows"][:T], pr.dst_rows[:T])                 # rows packed by the uploads
    # log-probs: the chunked launches see the same rows as the single launch (split counts may differ: tolerance)
    assert (h["h_logp"][:T] - pr.logp.cpu()[:T]).abs().max().item() <= 1e-4
    assert torch.all(h["h_logp"][T:] == 7.0)
    # and against the oracle on sampled rows
    g = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, T - 1], g.integers(0, T, size=24)])).astype(np.int64)
    H = dv["d_dst_rows"][torch.from_numpy(rows).cuda()].cpu()
    lp_ref, _ = oracle.token_logprob(synth.as_oracle_array(H), synth.as_oracle_array(pr.W_vocab.cpu()),
                                     pr.dst_tokens.cpu().numpy()[rows])
    assert np.abs(h["h_logp"].numpy()[rows] - lp_ref).max() <= 2e-3
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()


def test_host_step_validates_before_it_copies():
    """A head of another width, a hidden width that is no multiple of 8 and a short workspace are refused up front."""
    w = synth.WORKLOADS["mini"]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    h, dv, (head, tensors) = _host_step(pr, w)
    scal = dict(P=w.P, G=w.G, K=w.K, cutoff=w.cutoff, d=w.d, V=w.V, ddof=0, rho=w.rho, eps=1e-6, inv_temperature=1.0,
                T_src=pr.T_src, dst_capacity_tokens=pr.cap)
    dv["d_lengths"].fill_(-3)
    step = B.make_host_step(scal, head, pr.q_lut, tensors)
    step.head.d = w.d - 8
    with pytest.raises(B.ArrolError) as e:
        B.arrol_prune_rebatch_host(pr.ctx, step)
    assert e.value.code == -1
    step = B.make_host_step(scal, head, pr.q_lut, tensors)
    step.workspace_bytes = 16
    with pytest.raises(B.ArrolError) as e:
        B.arrol_prune_rebatch_host(pr.ctx, step)
    assert e.value.code == -3
    torch.cuda.synchronize()
    assert torch.all(dv["d_lengths"] == -3)            # nothing was uploaded by the refused calls
    pr.ctx.close()
