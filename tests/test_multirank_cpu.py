"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks shard the workload by prompt (different seeds, no
exchange on the data path) and reduce their timings as max over ranks and their tokens as a sum."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

from paper_2603_24840_b200 import dist_util, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    from paper_2603_24840_b200 import dist_util, synth
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    w = dist_util.shard_workload(synth.WORKLOADS["mini"], rank, world)
    ell = synth.lengths(w)
    step_ms, e2e_ms, tokens = 10.0 + 5.0 * rank, 30.0 - 7.0 * rank, float(ell.sum())
    dist.barrier()
    out = dist_util.reduce_timings(step_ms, e2e_ms, tokens, "cpu")
    print(json.dumps({"rank": rank, "seed": w.seed, "tokens": tokens, "reduced": out}), flush=True)
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_shard_and_reduce():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=120)
        assert p.returncode == 0, se[-2000:]
        outs.append(__import__("json").loads(so.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["seed"] != outs[1]["seed"] and outs[0]["tokens"] != outs[1]["tokens"]
    total = outs[0]["tokens"] + outs[1]["tokens"]
    for o in outs:
        assert o["reduced"] == [15.0, 30.0, total]          # max, max, sum: the same on every rank


def test_shard_workload_properties():
    w = synth.WORKLOADS["llama-3.2-1b"]
    assert dist_util.shard_workload(w, 0, 8) == w           # rank 0 is the single-GPU workload
    w3 = dist_util.shard_workload(w, 3, 8)
    assert (w3.P, w3.G, w3.K, w3.d, w3.V) == (w.P, w.G, w.K, w.d, w.V) and w3.seed != w.seed   # weak scaling
    assert not np.array_equal(synth.lengths(w), synth.lengths(w3))
    w5 = synth.WORKLOADS["qwen3-8b-dapo"]
    assert dist_util.shard_workload(w5, 0, 1, prompt_chunks=4).P == w5.P // 4
    assert dist_util.reduce_timings(1.0, 2.0, 3.0, "cpu") == (1.0, 2.0, 3.0)   # no process group: identity


def test_token_balanced_partition_of_the_prompt_groups():
    """Contiguous, complete, ordered ranges; imbalance (max / mean tokens per rank) small on the five workloads, both
    before pruning (sum of lengths per group) and after (the K longest rollouts of a group as a stand-in for its
    survivors)."""
    import numpy as np
    from paper_2603_24840_b200 import dist_util, synth
    for name in synth.WORKLOAD_ORDER:
        w = synth.WORKLOADS[name]
        ell = synth.lengths(w).astype(np.int64).reshape(w.P, w.G)
        for tokens in (ell.sum(1), np.sort(ell, axis=1)[:, -w.K:].sum(1)):
            for world in (1, 2, 3, 4, 8):
                if world > w.P:
                    continue
                parts = dist_util.balanced_partition(tokens, world)
                assert parts[0][0] == 0 and parts[-1][1] == w.P
                assert all(parts[r][1] == parts[r + 1][0] for r in range(world - 1))
                assert all(b < e for b, e in parts)
                per_rank = np.array([tokens[b:e].sum() for b, e in parts])
                # never worse than one (largest) group above the even share
                assert per_rank.max() <= tokens.sum() / world + tokens.max()
                if w.P >= 16 * world:
                    assert per_rank.max() / per_rank.mean() <= 1.10
    # degenerate inputs
    assert dist_util.balanced_partition([5, 5], 1) == [(0, 2)]
    assert dist_util.balanced_partition([], 2) == [(0, 0), (0, 0)]
    assert dist_util.balanced_partition([7], 3) == [(0, 1), (1, 1), (1, 1)]
    assert dist_util.balanced_partition([1, 1, 100, 1, 1], 2) in ([(0, 2), (2, 5)], [(0, 3), (3, 5)])
