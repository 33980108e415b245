"""Multi-GPU plumbing of the benchmark: the path shards by prompt group with no exchange step, so ranks only meet
at a barrier and when the timings are reduced (max over ranks) and the processed tokens are summed."""
from __future__ import annotations

import dataclasses

import torch
import torch.distributed as dist

from . import synth


def shard_workload(w: synth.Workload, rank: int, world: int, prompt_chunks: int = 1) -> synth.Workload:
    """Weak scaling: every rank prunes and re-batches its own P / prompt_chunks prompts; rank r draws its inputs
    from seed + 1000 r, so rank 0 of any world size sees the single-GPU workload."""
    if rank < 0 or rank >= world:
        raise ValueError("rank outside the world")
    if w.P % prompt_chunks != 0:
        raise ValueError("prompt_chunks must divide P")
    return dataclasses.replace(w, P=w.P // prompt_chunks, seed=w.seed + 1000 * rank)


def reduce_timings(step_ms: float, e2e_ms: float, tokens: float, device) -> tuple:
    """Returns (max step ms, max e2e ms, total tokens) over all ranks; identity without a process group."""
    t = torch.tensor([step_ms, e2e_ms], dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(n[0])
