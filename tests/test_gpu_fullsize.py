"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (PruneRebatch.step()):
outputs the oracle can compute cheaply are compared in full (scores, selection, scan, advantages, token ids);
the hidden-row payload and the token log-probs are compared on sampled rows, plus properties that hold at any
size (every packed row equals its source row; lse >= the target logit; exp(logp) in (0, 1])."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200.pipeline import PruneRebatch, host_inputs

pytestmark = pytest.mark.gpu


def _fullsize(name, n_logp_rows):
    w = synth.WORKLOADS[name]
    inp = host_inputs(w)                       # big tensors are generated on the device
    pr = PruneRebatch(w, inputs=inp)
    pr.step()
    torch.cuda.synchronize()
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    T = _check_state(pr, w, inp, n_logp_rows)
    # the same step with the survivors' rows read in place (no packed copy): identical log-probs
    ref = pr.logp[:T].clone()
    pr.logp.fill_(7.0)
    pr.prune_step(with_rows=False)
    pr.token_logprob_gathered()
    torch.cuda.synchronize()
    assert pr.counts()[1] == T and torch.equal(pr.logp[:T], ref)
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()


def _check_state(pr, w, inp, n_logp_rows):
    """Every output of a finished step of `pr` (a whole workload or one chunk view of it) against the oracle."""
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    head = inp["head"]
    off = inp["src_tok_off"]
    ridx = off[:-1] + (w.cutoff - 1)

    # a1/a2: the N rows the head reads, copied back for the oracle
    x_cut = pr.hidden_score[torch.from_numpy(ridx).to(pr.dev)].cpu()
    s_ref = oracle.head_score(oa(x_cut), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]), h=w.h)
    p_ref, b_ref, _ = oracle.prob_map(s_ref, inp["q_lut"])
    prob = pr.prob.cpu().numpy()
    assert np.abs(pr.score.cpu().numpy() - s_ref).max() <= 1e-3
    assert np.abs(prob - p_ref).max() <= 1e-3
    bins = pr.bin.cpu().numpy()
    assert np.array_equal(bins, np.array([oracle.bin_index(float(v), w.B) for v in prob]))
    q_gpu = pr.q.cpu().numpy()
    assert np.array_equal(q_gpu, inp["q_lut"][bins])

    # a3: selection, bit-exact, on the oracle's q and on the q the pipeline consumed
    _, _, q_ref = oracle.prob_map(s_ref, inp["q_lut"])
    keep_on_oracle_q = torch.empty(w.N, dtype=torch.uint8, device=pr.dev)
    B.arrol_select(pr.ctx, torch.from_numpy(q_ref.astype(np.float32)).to(pr.dev), w.P, w.G, w.K, w.rho,
                   keep_on_oracle_q)
    assert np.array_equal(keep_on_oracle_q.cpu().numpy(), oracle.select(q_ref.astype(np.float32), w.P, w.G, w.K, w.rho))
    keep_ref = oracle.select(q_gpu, w.P, w.G, w.K, w.rho)
    assert np.array_equal(pr.keep.cpu().numpy(), keep_ref)

    # a4/a6: scan and advantages in full
    idx, cu, S, T = oracle.survivor_scan(keep_ref, inp["lengths"])
    assert pr.counts() == (S, T) and S == w.S and T <= pr.cap
    assert np.array_equal(pr.survivor_idx.cpu().numpy()[:S], idx)
    assert np.array_equal(pr.cu_seqlens.cpu().numpy()[:S + 1], cu)
    adv_ref = oracle.advantages(inp["rewards"], keep_ref, w.G)
    adv = pr.adv.cpu().numpy()[:S]
    assert np.abs(adv - adv_ref).max() <= 1e-5
    rew_kept = inp["rewards"][keep_ref == 1].reshape(w.P, w.K)
    flat = (rew_kept.min(1) == rew_kept.max(1))
    assert np.all(adv.reshape(w.P, w.K)[flat] == 0.0)          # all-0 / all-1 survivor sets: exactly zero

    # a5: token ids in full; per-token bookkeeping; hidden rows: every packed row equals its source row
    dt_ref, _, seq_ref = oracle.gather(idx, cu, off[:-1], inp["src_tokens"])
    assert np.array_equal(pr.dst_tokens.cpu().numpy()[:T], dt_ref)
    assert np.array_equal(pr.tok_seq.cpu().numpy()[:T], seq_ref)
    assert np.array_equal(pr.tok_adv.cpu().numpy()[:T], adv[seq_ref])
    src_row = torch.from_numpy(off[:-1][idx][seq_ref] + (np.arange(T) - cu[:-1][seq_ref])).to(pr.dev)
    step = 1 << 16
    for t0 in range(0, T, step):
        t1 = min(T, t0 + step)
        assert torch.equal(pr.dst_rows[t0:t1], pr.src_rows[src_row[t0:t1]])

    # a7: sampled rows against the fp64 oracle; first/last row of every 16th survivor, the forced edge ids, the
    # last (partial) token tile, the rest uniform at random
    g = np.random.default_rng(w.seed)
    rows = np.unique(np.concatenate([[0, T - 1], cu[:-1][::16], cu[1:][::16] - 1, np.arange(T - T % 128, T)[:4],
                                     np.flatnonzero(dt_ref[:4096] >= (w.V // 256) * 256)[:4],
                                     g.integers(0, T, size=n_logp_rows)])).astype(np.int64)
    rows = rows[(rows >= 0) & (rows < T)]
    H = pr.dst_rows[torch.from_numpy(rows).to(pr.dev)].cpu()
    lp_ref, lse_ref = oracle.token_logprob(oa(H), oa(pr.W_vocab.cpu()), dt_ref[rows])
    logp = pr.logp.cpu().numpy()[:T]
    lse = pr.lse.cpu().numpy()[:T]
    assert np.abs(logp[rows] - lp_ref).max() <= 2e-3
    assert np.abs(lse[rows] - lse_ref).max() <= 2e-3
    assert np.all(np.isfinite(logp)) and np.all(logp <= 1e-6) and np.all(logp > -60.0)
    return T


def test_llama_3_2_1b_shaped():
    _fullsize("llama-3.2-1b", 40)


def test_qwen3_1_7b_shaped():
    _fullsize("qwen3-1.7b", 24)


def test_qwen3_4b_shaped():
    _fullsize("qwen3-4b", 16)


def test_qwen3_8b_dapo_shaped_all_prompt_chunks_and_in_place():
    """The largest workload as the benchmark runs it: all 256 prompts' source rows resident, four chunks of 64
    different prompts through one set of packed buffers, every chunk checked; then all prompts in one pass with the
    rows read in place, which must reproduce the chunks' log-probs bit for bit."""
    w = synth.WORKLOADS["qwen3-8b-dapo"]
    parent = PruneRebatch(w, inputs=host_inputs(w), with_rows=False)
    views = PruneRebatch.chunk_views(parent, 4)
    pieces, T_total = [], 0
    for c, v in enumerate(views):
        v.step()
        torch.cuda.synchronize()
        assert B.arrol_poll_status(parent.ctx, raise_on_error=False) == 0
        T = _check_state(v, v.w, v.host, 12 if c in (0, 3) else 4)
        pieces.append(v.logp[:T].clone())
        T_total += T
    parent.prune_step(with_rows=False)
    parent.token_logprob_gathered()
    torch.cuda.synchronize()
    assert B.arrol_poll_status(parent.ctx, raise_on_error=False) == 0
    assert parent.counts() == (w.S, T_total)
    assert torch.equal(parent.logp[:T_total], torch.cat(pieces))
    parent.ctx.close()


def test_llama_3_2_1b_shaped_update_leg():
    """lm_head backward at the benchmark's size and launch configuration (all 35 token chunks of the step's survivors).
    The gradient w.r.t. the log-probs is non-zero on a sample of tokens only (first and last rows, both sides of
    chunk and tile edges, the last partial chunk, random ones), so the oracle can produce the exact dH rows of the
    sample and the whole of dW = sum over the sample; every other dH row must be exactly zero."""
    from oracle import update as ou
    from paper_2603_24840_b200 import update as U
    w = synth.WORKLOADS["llama-3.2-1b"]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    pr.step()
    torch.cuda.synchronize()
    S, T = pr.counts()
    g = np.random.default_rng(11)
    chunk = 9472
    edges = [0, 1, 127, 128, chunk - 1, chunk, chunk + 1, 5 * chunk - 1, 5 * chunk, (T // chunk) * chunk, T - 129, T - 2, T - 1]
    sample = np.unique(np.concatenate([np.array(edges), g.integers(0, T, size=35)])).astype(np.int64)
    grad_s = g.normal(size=sample.size).astype(np.float32)
    grad = torch.zeros(pr.cap, device=pr.dev)
    grad[torch.from_numpy(sample).to(pr.dev)] = torch.from_numpy(grad_s).to(pr.dev)
    dH = torch.full((pr.cap, w.d), 9.0, device=pr.dev)
    dW = torch.full((w.V, w.d), 9.0, device=pr.dev)
    ws = torch.empty(U.arrol_lm_head_backward_workspace(pr.ctx, pr.cap, w.d, w.V), dtype=torch.uint8, device=pr.dev)
    U.arrol_lm_head_backward(pr.ctx, pr.dst_rows, pr.W_vocab, pr.dst_tokens, grad, pr.lse, pr.cap, w.d, w.V, dH, dW, ws,
                             d_T=pr.d_num[1:])
    torch.cuda.synchronize()
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0

    idx = torch.from_numpy(sample).to(pr.dev)
    H_s = pr.dst_rows[idx].cpu()
    y_s = pr.dst_tokens[idx].cpu().numpy()
    dH_ref, dW_ref = ou.lm_head_backward(synth.as_oracle_array(H_s), synth.as_oracle_array(pr.W_vocab.cpu()), y_s,
                                         grad_s.astype(np.float64))
    dH_s = dH[idx].cpu().numpy().astype(np.float64)
    for got, ref in ((dH_s, dH_ref), (dW.cpu().numpy().astype(np.float64), dW_ref)):
        assert np.abs(got - ref).max() <= 1e-2 * np.abs(ref).max()
        assert np.linalg.norm(got - ref) <= 5e-3 * np.linalg.norm(ref)
    rest = torch.ones(T, dtype=torch.bool, device=pr.dev)
    rest[idx] = False
    assert float(dH[:T][rest].abs().max()) == 0.0             # rows without a gradient are exactly zero
    pr.ctx.close()
