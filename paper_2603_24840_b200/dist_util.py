"""Multi-GPU plumbing of the benchmark: the path shards by prompt group with no exchange step, so ranks only meet
at a barrier and when the timings are reduced (max over ranks) and the processed tokens are summed."""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import numpy as np
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


def balanced_partition(group_tokens: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Contiguous ranges [begin, end) of prompt groups for `world` ranks, balanced by token count: `group_tokens[g]`
    is the work of group g (the sum of its rollouts' lengths before pruning, its survivor tokens after).  Greedy on
    the prefix sums: rank r ends at the group whose prefix sum is nearest to (r + 1) / world of the total, with at
    least one group per rank while groups remain.  Groups stay whole and in order, so no exchange is needed."""
    t = np.asarray(group_tokens, dtype=np.int64)
    n = int(t.shape[0])
    if world < 1:
        raise ValueError("world must be positive")
    prefix = np.concatenate([[0], np.cumsum(t)])
    total = int(prefix[-1])
    bounds = [0]
    for r in range(world - 1):
        target = total * (r + 1) / world
        lo = min(bounds[-1] + 1, n)                            # at least one group, if any is left
        hi = max(lo, n - (world - 1 - r))                      # leave one group for every later rank where possible
        cut = int(np.searchsorted(prefix, target, side="left"))
        if cut > 0 and abs(prefix[cut - 1] - target) <= abs(prefix[min(cut, n)] - target):
            cut -= 1
        bounds.append(int(min(max(cut, lo), max(hi, lo))) if lo <= n else n)
    bounds.append(n)
    return [(bounds[r], bounds[r + 1]) for r in range(world)]
