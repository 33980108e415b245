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


def test_back_to_back_steps_never_read_the_previous_steps_results():
    """The kernels of a step start while their predecessor is still running (programmatic dependent launch) and must
    wait before they read its results.  Two steps with different heads are issued back to back without a host
    synchronisation; the buffers must hold exactly what the second step alone produces, in either order."""
    w = synth.WORKLOADS["profile-mlp"]
    pr = PruneRebatch(w, inputs=host_inputs(w), with_rows=False)
    heads = [pr.head, dict(pr.head)]
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    heads[1]["w2"] = (pr.head["w2"].float() * (torch.rand(w.h, generator=gen, device="cuda") * 4 - 2)).to(pr.head["w2"].dtype)
    keys = ("score", "q", "keep", "survivor_idx", "cu_seqlens", "adv", "d_num", "dst_tokens", "tok_seq")
    refs = []
    for hd in heads:
        pr.head = hd
        B.arrol_prune_step(pr.ctx, pr.prune_step_args(with_rows=False))
        torch.cuda.synchronize()
        refs.append(({k: getattr(pr, k).clone() for k in keys}, pr.counts()))
    assert not torch.equal(refs[0][0]["keep"], refs[1][0]["keep"])          # the two steps really differ
    args = []
    for hd in heads:
        pr.head = hd
        args.append(pr.prune_step_args(with_rows=False))
    for first, second in ((0, 1), (1, 0), (0, 1)):
        for _ in range(3):
            B.arrol_prune_step(pr.ctx, args[first])
            B.arrol_prune_step(pr.ctx, args[second])
        torch.cuda.synchronize()
        want, (S, T) = refs[second]
        assert pr.counts() == (S, T)
        for k in ("score", "q", "keep", "d_num"):
            assert torch.equal(getattr(pr, k), want[k]), k
        for k in ("survivor_idx", "adv"):
            assert torch.equal(getattr(pr, k)[:S], want[k][:S]), k
        assert torch.equal(pr.cu_seqlens[:S + 1], want["cu_seqlens"][:S + 1])
        for k in ("dst_tokens", "tok_seq"):
            assert torch.equal(getattr(pr, k)[:T], want[k][:T]), k
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()


@pytest.mark.parametrize("P,G,K", [(1, 1, 1), (7, 1, 1), (5, 3, 2), (9, 5, 1), (3, 32, 7), (40, 32, 16), (200, 4, 4), (333, 2, 1),
                                   (150, 16, 8), (1000, 2, 1)])
def test_fused_prune_step_over_group_shapes(P, G, K):
    """Group sizes that are no power of two, one group per block and many, more blocks than one wave of the chained
    scan would hold (the call then takes the three separate launches): always what the three calls give."""
    import dataclasses
    w = dataclasses.replace(synth.WORKLOADS["mini"], P=P, G=G, K=K, h=0, seed=100 + P + G)
    pr = PruneRebatch(w, inputs=host_inputs(w), with_rows=False)
    pr.prune_step(with_rows=False)
    torch.cuda.synchronize()
    keys = ("score", "prob", "q", "bin", "keep", "survivor_idx", "cu_seqlens", "adv", "d_num", "dst_tokens", "tok_adv", "tok_seq")
    want = {k: getattr(pr, k).clone() for k in keys}
    S, T = pr.counts()
    assert S == P * K
    for _ in range(2):                                  # twice: the chained scan's published totals are cleared in between
        for k in keys:
            getattr(pr, k).fill_(0)
        B.arrol_prune_step(pr.ctx, pr.prune_step_args(with_rows=False))
        torch.cuda.synchronize()
        assert pr.counts() == (S, T)
        for k in ("score", "prob", "q", "bin", "keep", "d_num"):
            assert torch.equal(getattr(pr, k), want[k]), k
        for k in ("survivor_idx", "adv"):
            assert torch.equal(getattr(pr, k)[:S], want[k][:S]), k
        assert torch.equal(pr.cu_seqlens[:S + 1], want["cu_seqlens"][:S + 1])
        for k in ("dst_tokens", "tok_adv", "tok_seq"):
            assert torch.equal(getattr(pr, k)[:T], want[k][:T]), k
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    pr.ctx.close()
