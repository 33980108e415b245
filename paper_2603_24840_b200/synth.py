"""Seeded synthetic inputs for the prune-and-rebatch path.

This module only draws random inputs and lays them out; it contains none of
the method's arithmetic (no head, no sigmoid, no binning, no selection, no
softmax).  Both the CPU oracle's tests and the CUDA path's tests / bench read
their inputs from here so that the two sides see the same arrays.

Shapes follow the paper's training setup (Section 5.1: group size 16, keep
ratio 0.5, detection length 512, maximum sequence length 8192) scaled to the
five workload shapes below.  Small arrays come from numpy's PCG64; the large
activations and vocabulary weights come from a seeded torch generator on the
device that will hold them.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    P: int            # prompts per step
    G: int            # rollouts per prompt (group size)
    K: int            # survivors kept per group
    cutoff: int       # L_detect, tokens generated when the head is evaluated
    L_max: int        # maximum response length
    len_dist: tuple   # ("uniform", lo, hi) or ("lognormal", median, sigma)
    d: int            # hidden width
    V: int            # vocabulary size
    dtype: str        # "f32" or "bf16": storage type of hidden / weights
    h: int            # quality-head hidden width, 0 = linear head
    reward: str       # "bernoulli_half" | "beta_bernoulli"
    seed: int
    degenerate_frac: float = 0.0   # fraction of groups forced all-0 / all-1
    B: int = 128      # calibration bins (Appendix A.4)
    rho: float = 0.5  # target positive ratio

    @property
    def N(self) -> int:
        return self.P * self.G

    @property
    def S(self) -> int:
        return self.P * self.K


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("tiny", 4, 8, 4, 64, 256, ("uniform", 96, 256), 256, 4096, "f32", 0,
                 "bernoulli_half", 0),
        Workload("llama-3.2-1b", 64, 8, 4, 256, 2048, ("uniform", 512, 2048), 2048, 128256, "bf16", 0,
                 "beta_bernoulli", 1),
        Workload("qwen3-1.7b", 128, 16, 8, 512, 4096, ("lognormal", 1500.0, 0.35), 2048, 151936, "bf16", 256,
                 "beta_bernoulli", 2),
        Workload("qwen3-4b", 128, 16, 8, 512, 8192, ("lognormal", 2500.0, 0.35), 2560, 151936, "bf16", 0,
                 "beta_bernoulli", 3, degenerate_frac=0.30),
        Workload("qwen3-8b-dapo", 256, 16, 8, 1024, 8192, ("lognormal", 3000.0, 0.35), 4096, 151936, "bf16", 512,
                 "beta_bernoulli", 4),
        # Small case for profiler captures: the Llama-shaped d and V on ~75k survivor tokens, so that inputs are
        # larger than L2 while the device holds about 1.5 GB and a log-prob launch lasts ~25 ms.
        Workload("profile-small", 48, 8, 4, 256, 512, ("uniform", 256, 512), 2048, 128256, "bf16", 0,
                 "beta_bernoulli", 9),
        # Small case for profiler captures of the MLP head: the Qwen-3-1.7B-shaped N, d, h on short rollouts.
        Workload("profile-mlp", 128, 16, 8, 64, 128, ("uniform", 64, 128), 2048, 8192, "bf16", 256,
                 "beta_bernoulli", 10),
        # Small case for profiler captures at the DAPO-shaped d, V and head: ~75k survivor tokens, about 3 GB on the device.
        Workload("profile-wide", 48, 8, 4, 256, 512, ("uniform", 256, 512), 4096, 151936, "bf16", 512,
                 "beta_bernoulli", 11),
        # Mid-size case for CPU-only tests: several tiles and ragged tails, seconds on the host.
        Workload("mini", 6, 8, 4, 16, 96, ("uniform", 16, 96), 192, 1000, "bf16", 24,
                 "beta_bernoulli", 7, degenerate_frac=0.34),
    ]
}
WORKLOAD_ORDER = ["tiny", "llama-3.2-1b", "qwen3-1.7b", "qwen3-4b", "qwen3-8b-dapo"]


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.float32 if w.dtype == "f32" else torch.bfloat16


def _rng(w: Workload, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([w.seed, stream]))


def lengths(w: Workload) -> np.ndarray:
    """Response length of every rollout, int32 [N], clipped to [cutoff, L_max]."""
    g = _rng(w, 1)
    kind = w.len_dist[0]
    if kind == "uniform":
        ell = g.integers(int(w.len_dist[1]), int(w.len_dist[2]) + 1, size=w.N)
    else:
        ell = np.rint(g.lognormal(np.log(w.len_dist[1]), w.len_dist[2], size=w.N)).astype(np.int64)
    return np.clip(ell, w.cutoff, w.L_max).astype(np.int32)


def rewards(w: Workload) -> np.ndarray:
    """Binary verifiable rewards, float32 [N] (Section 3, R in {0,1})."""
    g = _rng(w, 2)
    if w.reward == "bernoulli_half":
        p = np.full(w.P, 0.5)
    else:
        p = g.beta(0.5, 0.5, size=w.P)
    r = (g.random((w.P, w.G)) < p[:, None]).astype(np.float32)
    if w.degenerate_frac > 0:
        n_forced = int(round(w.degenerate_frac * w.P))
        which = g.permutation(w.P)[:n_forced]
        for j, p_idx in enumerate(which):
            r[p_idx, :] = float(j % 2)  # alternate all-0 / all-1
    return r.reshape(-1)


def _round_to(x: np.ndarray, w: Workload) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch_dtype(w))


def head_weights(w: Workload) -> Dict[str, Optional[torch.Tensor]]:
    """Quality-head parameters N(0, 0.02^2), stored in the workload's dtype (CPU tensors)."""
    g = _rng(w, 3)
    if w.h == 0:
        return {"W1": _round_to(g.normal(0, 0.02, size=w.d), w),
                "b1": _round_to(g.normal(0, 0.02, size=1), w), "w2": None, "b2": None}
    return {"W1": _round_to(g.normal(0, 0.02, size=(w.h, w.d)), w),
            "b1": _round_to(g.normal(0, 0.02, size=w.h), w),
            "w2": _round_to(g.normal(0, 0.02, size=w.h), w),
            "b2": _round_to(g.normal(0, 0.02, size=1), w)}


def calib_history(w: Workload, n: int = 8192):
    """Historical (normalised score, label) pairs that feed the binned estimator's buffers:
    y ~ Bernoulli(0.35), s' ~ Beta(4,2) for positives and Beta(2,4) for negatives."""
    g = _rng(w, 4)
    y = (g.random(n) < 0.35).astype(np.uint8)
    s = np.where(y == 1, g.beta(4, 2, size=n), g.beta(2, 4, size=n))
    return s.astype(np.float64), y


def src_offsets(ell: np.ndarray) -> np.ndarray:
    """First source row of every rollout in the packed pre-prune buffer, int64 [N+1]."""
    off = np.zeros(ell.shape[0] + 1, dtype=np.int64)
    np.cumsum(ell.astype(np.int64), out=off[1:])
    return off


def token_ids(w: Workload, n_tokens: int) -> np.ndarray:
    """Response token ids, int32 [n_tokens], uniform on [0, V) with the first rows forced to
    vocabulary ids that sit on tile edges (0, 127, 128, 255, 256, V-1 and ids in the last chunk)."""
    g = _rng(w, 5)
    t = g.integers(0, w.V, size=n_tokens, dtype=np.int64).astype(np.int32)
    edge = [0, 127, 128, 255, 256, w.V - 1, w.V - 2, (w.V // 256) * 256 % w.V]
    for j, v in enumerate(edge):
        if j < n_tokens:
            t[j] = min(max(v, 0), w.V - 1)
    return t


def normal_tensor(shape, std: float, dtype: torch.dtype, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std^2) drawn in fp32 from a seeded generator on `device`, rounded once to `dtype`."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    rows = shape[0]
    out = torch.empty(shape, dtype=dtype, device=device)
    # Draw in row slabs so the fp32 staging buffer stays small next to the result.
    per_row = 1
    for s in shape[1:]:
        per_row *= s
    slab = max(1, (1 << 27) // max(per_row, 1))
    for r0 in range(0, rows, slab):
        r1 = min(rows, r0 + slab)
        x = torch.randn((r1 - r0,) + tuple(shape[1:]), generator=gen, device=device, dtype=torch.float32)
        out[r0:r1] = (x * std).to(dtype)
    return out


def hidden_states(w: Workload, rows: int, device="cpu", stream: int = 11, scale: float = 1.0) -> torch.Tensor:
    """Policy hidden states N(0,1), [rows, d] in the workload's dtype."""
    return normal_tensor((rows, w.d), scale, torch_dtype(w), w.seed * 1000 + stream, device)


def vocab_weights(w: Workload, device="cpu", dtype: Optional[torch.dtype] = None) -> torch.Tensor:
    """lm_head weight N(0, 0.02^2), stored [V, d] row-major."""
    return normal_tensor((w.V, w.d), 0.02, dtype or torch_dtype(w), w.seed * 1000 + 12, device)


def as_oracle_array(t: torch.Tensor) -> np.ndarray:
    """CPU view of a tensor in the form the oracle reads: float32 / float64 arrays as they are,
    bf16 as its uint16 bit pattern (the oracle widens the bits itself)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
