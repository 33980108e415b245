"""arrol_prune_step (score -> select -> compact in one call) gives exactly what the three calls give."""
import pytest
import torch

from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200.pipeline import PruneRebatch, host_inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,rows", [("tiny", True), ("mini", True), ("mini", False), ("profile-mlp", True)])
def test_one_call_prune_step_equals_three_calls(name, rows):
    w = synth.WORKLOADS[name]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    pr.prune_step(with_rows=rows)
    torch.cuda.synchronize()
    want = {k: getattr(pr, k).clone() for k in ("score", "prob", "q", "bin", "keep", "survivor_idx", "cu_seqlens", "adv",
                                                  "d_num", "dst_tokens", "tok_adv", "tok_seq", "dst_rows")}
    S, T = pr.counts()
    for k in want:
        getattr(pr, k).fill_(0)
    B.arrol_prune_step(pr.ctx, pr.prune_step_args(with_rows=rows))
    torch.cuda.synchronize()
    assert pr.counts() == (S, T)
    for k in ("score", "prob", "q", "bin", "keep", "d_num"):
        assert torch.equal(getattr(pr, k), want[k]), k
    for k in ("survivor_idx", "adv"):
        assert torch.equal(getattr(pr, k)[:S], want[k][:S]), k
    assert torch.equal(pr.cu_seqlens[:S + 1], want["cu_seqlens"][:S + 1])
    for k in ("dst_tokens", "tok_adv", "tok_seq"):
        assert torch.equal(getattr(pr, k)[:T], want[k][:T]), k
    if rows:
        assert torch.equal(pr.dst_rows[:T], want["dst_rows"][:T])
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()


@pytest.mark.parametrize("name,rows", [("mini", True), ("profile-mlp", False)])
def test_prune_step_replayed_from_a_cuda_graph(name, rows):
    """The step allocates nothing and never synchronises, so it can be captured once and replayed; the kernels'
    programmatic launch dependencies survive the capture.  Replays give what the eager call gives."""
    w = synth.WORKLOADS[name]
    pr = PruneRebatch(w, inputs=host_inputs(w))
    args = pr.prune_step_args(with_rows=rows)
    B.arrol_prune_step(pr.ctx, args)
    torch.cuda.synchronize()
    keys = ["score", "q", "keep", "survivor_idx", "cu_seqlens", "adv", "d_num", "dst_tokens", "tok_adv", "tok_seq"]
    if rows:
        keys.append("dst_rows")
    want = {k: getattr(pr, k).clone() for k in keys}
    S, T = pr.counts()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        B.arrol_prune_step(pr.ctx, args)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        B.arrol_prune_step(pr.ctx, args)
    for _ in range(2):
        for k in keys:
            getattr(pr, k).fill_(0)
        graph.replay()
        torch.cuda.synchronize()
        assert pr.counts() == (S, T)
        for k in ("score", "q", "keep", "d_num"):
            assert torch.equal(getattr(pr, k), want[k]), k
        for k in ("survivor_idx", "adv"):
            assert torch.equal(getattr(pr, k)[:S], want[k][:S]), k
        assert torch.equal(pr.cu_seqlens[:S + 1], want["cu_seqlens"][:S + 1])
        for k in ("dst_tokens", "tok_adv", "tok_seq"):
            assert torch.equal(getattr(pr, k)[:T], want[k][:T]), k
        if rows:
            assert torch.equal(pr.dst_rows[:T], want["dst_rows"][:T])
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    del graph
    pr.ctx.close()
