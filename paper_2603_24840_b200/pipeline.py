"""Buffers and call sequence of one prune-and-rebatch step on one GPU.

This is orchestration only: it allocates device memory with torch, uploads a workload's inputs and issues the
four library calls on the current stream (score -> select -> compact -> token log-prob) with no host
synchronisation in between; the survivor token count stays on the device.  All arithmetic is in the CUDA library.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as B
from . import synth


def token_capacity(w: synth.Workload, ell: np.ndarray) -> int:
    """Upper bound on the survivor token count: the K longest rollouts of every group."""
    per_group = np.sort(ell.reshape(w.P, w.G).astype(np.int64), axis=1)[:, -w.K:]
    return int(per_group.sum())


class PruneRebatch:
    """Device-resident state of one workload.  `inputs` are host arrays / CPU tensors (see `host_inputs`)."""

    def __init__(self, w: synth.Workload, device: int = 0, with_rows: bool = True, inputs: Optional[Dict] = None,
                 ctx: Optional[B.Context] = None):
        self.w = w
        self.dev = torch.device("cuda", device)
        self.ctx = ctx or B.Context(device)
        self.with_rows = with_rows
        inp = inputs or host_inputs(w)
        self.host = inp
        ell = inp["lengths"]
        self.T_src = int(inp["src_tok_off"][-1])
        self.cap = token_capacity(w, ell)
        dev = self.dev
        i32, i64, f32 = torch.int32, torch.int64, torch.float32

        def up(a, dtype=None):
            t = torch.from_numpy(np.ascontiguousarray(a)) if isinstance(a, np.ndarray) else a
            return t.to(dev) if dtype is None else t.to(dev, dtype)

        self.lengths = up(ell)
        self.rewards = up(inp["rewards"])
        self.src_tok_off = up(inp["src_tok_off"][:-1])
        self.row_index = up(inp["src_tok_off"][:-1] + (w.cutoff - 1))
        self.src_tokens = up(inp["src_tokens"])
        self.head = {k: (None if v is None else v.to(dev)) for k, v in inp["head"].items()}
        self.head["h"] = w.h
        self.q_lut = up(inp["q_lut"])
        # activations and vocabulary weights: generated on the device (seeded) unless supplied
        if "hidden" in inp:
            self.hidden_score = inp["hidden"].to(dev)
        else:
            self.hidden_score = synth.hidden_states(w, self.T_src, device=dev)
        self.src_rows = self.hidden_score if self.hidden_score.dtype == torch.bfloat16 \
            else self.hidden_score.to(torch.bfloat16)
        if "W_vocab" in inp:
            self.W_vocab = inp["W_vocab"].to(dev, torch.bfloat16)
        else:
            self.W_vocab = synth.vocab_weights(w, device=dev, dtype=torch.bfloat16)
        N, cap = w.N, self.cap
        self.score = torch.empty(N, dtype=f32, device=dev)
        self.prob = torch.empty(N, dtype=f32, device=dev)
        self.q = torch.empty(N, dtype=f32, device=dev)
        self.bin = torch.empty(N, dtype=i32, device=dev)
        self.keep = torch.empty(N, dtype=torch.uint8, device=dev)
        self.survivor_idx = torch.empty(N, dtype=i32, device=dev)
        self.cu_seqlens = torch.empty(N + 1, dtype=i64, device=dev)
        self.adv = torch.empty(N, dtype=f32, device=dev)
        self.d_num = torch.zeros(2, dtype=i64, device=dev)
        self.dst_tokens = torch.empty(cap, dtype=i32, device=dev)
        self.tok_adv = torch.empty(cap, dtype=f32, device=dev)
        self.tok_seq = torch.empty(cap, dtype=i32, device=dev)
        self.dst_rows = torch.empty((cap, w.d), dtype=torch.bfloat16, device=dev) if with_rows else None
        self.logp = torch.empty(cap, dtype=f32, device=dev)
        self.lse = torch.empty(cap, dtype=f32, device=dev)
        ws = max(B.arrol_token_logprob_workspace(self.ctx, cap, w.d, w.V),
                 B.arrol_token_logprob_gathered_workspace(self.ctx, N, cap, w.d, w.V))
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)

    @classmethod
    def chunk_views(cls, parent: "PruneRebatch", n_chunks: int) -> List["PruneRebatch"]:
        """Splits a resident workload into `n_chunks` groups of consecutive prompts that are processed one after the
        other through ONE set of work buffers (packed rows, per-token arrays, workspace sized for the largest chunk).
        Every view reads its own prompts' rows in the parent's source buffers (explicit offsets), so all of the
        parent's prompts are covered and nothing is copied."""
        w = parent.w
        if w.P % n_chunks != 0:
            raise ValueError("n_chunks must divide P")
        Pc = w.P // n_chunks
        Nc = Pc * w.G
        wc = dataclasses.replace(w, P=Pc)
        ell = parent.host["lengths"]
        caps = [token_capacity(wc, ell[c * Nc:(c + 1) * Nc]) for c in range(n_chunks)]
        cap = max(caps)
        dev = parent.dev
        i32, i64, f32 = torch.int32, torch.int64, torch.float32
        ws = max(B.arrol_token_logprob_workspace(parent.ctx, cap, w.d, w.V),
                 B.arrol_token_logprob_gathered_workspace(parent.ctx, Nc, cap, w.d, w.V))
        bufs = dict(
            score=torch.empty(Nc, dtype=f32, device=dev), prob=torch.empty(Nc, dtype=f32, device=dev),
            q=torch.empty(Nc, dtype=f32, device=dev), bin=torch.empty(Nc, dtype=i32, device=dev),
            keep=torch.empty(Nc, dtype=torch.uint8, device=dev), survivor_idx=torch.empty(Nc, dtype=i32, device=dev),
            cu_seqlens=torch.empty(Nc + 1, dtype=i64, device=dev), adv=torch.empty(Nc, dtype=f32, device=dev),
            dst_tokens=torch.empty(cap, dtype=i32, device=dev), tok_adv=torch.empty(cap, dtype=f32, device=dev),
            tok_seq=torch.empty(cap, dtype=i32, device=dev),
            dst_rows=torch.empty((cap, w.d), dtype=torch.bfloat16, device=dev),
            logp=torch.empty(cap, dtype=f32, device=dev), lse=torch.empty(cap, dtype=f32, device=dev),
            workspace=torch.empty(ws, dtype=torch.uint8, device=dev))
        views = []
        for c in range(n_chunks):
            v = cls.__new__(cls)
            sl = slice(c * Nc, (c + 1) * Nc)
            v.w, v.dev, v.ctx, v.with_rows = wc, dev, parent.ctx, True
            v.T_src, v.cap = parent.T_src, caps[c]
            v.host = dict(parent.host, lengths=ell[sl], rewards=parent.host["rewards"][sl],
                          src_tok_off=parent.host["src_tok_off"][c * Nc:(c + 1) * Nc + 1])
            for name in ("lengths", "rewards", "src_tok_off", "row_index"):
                setattr(v, name, getattr(parent, name)[sl])
            for name in ("src_tokens", "head", "q_lut", "hidden_score", "src_rows", "W_vocab"):
                setattr(v, name, getattr(parent, name))
            for name, t in bufs.items():
                setattr(v, name, t)
            v.d_num = torch.zeros(2, dtype=i64, device=dev)      # every view keeps its own {S, T}
            views.append(v)
        return views

    # ---- the four calls -------------------------------------------------------------------------------
    def score_partial(self):
        B.arrol_score_partial(self.ctx, self.hidden_score, self.head, self.w.N, self.score, self.prob, self.q,
                              bin=self.bin, row_index=self.row_index, q_lut=self.q_lut)

    def select(self, q: Optional[torch.Tensor] = None):
        B.arrol_select(self.ctx, self.q if q is None else q, self.w.P, self.w.G, self.w.K, self.w.rho, self.keep)

    def compact(self, with_rows: Optional[bool] = None):
        rows = self.with_rows if with_rows is None else with_rows
        B.arrol_compact(self.ctx, self.keep, self.lengths, self.src_tok_off, self.w.N, self.w.G, self.rewards,
                        self.cap, self.cu_seqlens, self.survivor_idx, self.adv, self.d_num,
                        src_tokens=self.src_tokens, dst_tokens=self.dst_tokens,
                        src_rows=self.src_rows if rows else None, dst_rows=self.dst_rows if rows else None,
                        row_bytes=self.w.d * 2 if rows else 0, tok_adv=self.tok_adv, tok_seq=self.tok_seq)

    def token_logprob(self, hidden: Optional[torch.Tensor] = None):
        h = self.dst_rows if hidden is None else hidden
        B.arrol_token_logprob(self.ctx, h, self.W_vocab, self.dst_tokens, self.cap, self.w.d, self.w.V, self.logp,
                              self.workspace, lse=self.lse, d_T=self.d_num[1:])

    def token_logprob_gathered(self):
        """Log-probs with the survivors' rows read in place from the source buffer (no packed copy needed)."""
        B.arrol_token_logprob_gathered(self.ctx, self.src_rows, self.W_vocab, self.dst_tokens, self.cu_seqlens,
                                       self.survivor_idx, self.src_tok_off, self.d_num, self.w.N, self.cap, self.w.d,
                                       self.w.V, self.logp, self.workspace, lse=self.lse)

    def prune_step(self, with_rows: Optional[bool] = None):
        self.score_partial()
        self.select()
        self.compact(with_rows)

    def prune_step_args(self, with_rows: Optional[bool] = None):
        """Argument block of the one-call prune step (arrol_prune_step) over this state's buffers."""
        rows = self.with_rows if with_rows is None else with_rows
        scal = dict(P=self.w.P, G=self.w.G, K=self.w.K, rho=self.w.rho, eps=1e-6, ddof=0,
                    dst_capacity_tokens=self.cap, row_bytes=self.w.d * 2 if rows else 0)
        tensors = dict(row_index=self.row_index, score=self.score, prob=self.prob, q=self.q, bin=self.bin,
                       keep=self.keep, lengths=self.lengths, src_tok_off=self.src_tok_off,
                       src_tokens=self.src_tokens, src_rows=self.src_rows if rows else None, rewards=self.rewards,
                       dst_tokens=self.dst_tokens, dst_rows=self.dst_rows if rows else None,
                       cu_seqlens=self.cu_seqlens, survivor_idx=self.survivor_idx, adv=self.adv,
                       tok_adv=self.tok_adv, tok_seq=self.tok_seq, d_num=self.d_num)
        return B.make_prune_step(self.hidden_score, self.head, self.q_lut, scal, tensors)

    def step(self):
        """One pass of the whole path: score -> select -> compact (tokens + hidden rows) -> token log-prob."""
        self.prune_step()
        self.token_logprob()

    def counts(self):
        n = self.d_num.cpu()
        return int(n[0]), int(n[1])


def host_inputs(w: synth.Workload, with_hidden: bool = False) -> Dict:
    """Host-side inputs of a workload.  The calibration table is built with the library's own host helpers."""
    ell = synth.lengths(w)
    off = synth.src_offsets(ell)
    hist_s, hist_y = synth.calib_history(w)
    cpos, cneg = B.arrol_calib_counts(hist_s, hist_y, w.B)
    out = {
        "lengths": ell,
        "rewards": synth.rewards(w),
        "src_tok_off": off,
        "src_tokens": synth.token_ids(w, int(off[-1])),
        "head": synth.head_weights(w),
        "q_lut": B.arrol_build_q_lut(cpos, cneg, 1.0),
        "calib_history": (hist_s, hist_y),
    }
    if with_hidden:
        out["hidden"] = synth.hidden_states(w, int(off[-1]))
        out["W_vocab"] = synth.vocab_weights(w, dtype=torch.bfloat16)
    return out
