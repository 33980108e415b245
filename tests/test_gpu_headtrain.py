"""GPU parity of the quality-head training step against the oracle (fp32 accumulation over N rollouts and d
columns: 2e-4 of the largest gradient entry; loss 1e-5)."""
import numpy as np
import pytest
import torch

from oracle import headtrain as oh
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import headtrain as HT
from paper_2603_24840_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,d,h,dtype,use_mask", [
    (32, 256, 0, torch.float32, False), (513, 2048, 0, torch.bfloat16, True), (77, 2560, 0, torch.bfloat16, False),
    (48, 192, 24, torch.bfloat16, True), (300, 512, 256, torch.bfloat16, False), (70, 264, 132, torch.float32, True),
    (129, 1024, 512, torch.bfloat16, True),
])
def test_head_grad_matches_oracle(N, d, h, dtype, use_mask):
    ctx = B.Context(0)
    g = np.random.default_rng(N + d + h)
    x = torch.from_numpy(g.normal(size=(2 * N, d)).astype(np.float32)).to(dtype)
    ridx = g.permutation(2 * N)[:N].astype(np.int64)
    mk = lambda *s: torch.from_numpy(g.normal(0, 0.05, size=s).astype(np.float32)).to(dtype)
    head = {"W1": mk(d), "b1": mk(1), "w2": None, "b2": None} if h == 0 else \
           {"W1": mk(h, d), "b1": mk(h), "w2": mk(h) * 4, "b2": mk(1)}
    rew = (g.random(N) < 0.4).astype(np.float32)
    mask = (g.random(N) < 0.6).astype(np.uint8) if use_mask else None
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    loss_ref, gref = oh.head_bce_grad(oa(x), rew > 0.5, oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]),
                                      row_index=ridx, h=h, mask=mask)
    dhead = {k: (None if v is None else v.cuda()) for k, v in head.items()}
    dhead["h"] = h
    hh = max(h, 1)
    grads = {"W1": torch.full((hh, d), 5.0, device="cuda"), "b1": torch.full((hh,), 5.0, device="cuda")}
    if h:
        grads["w2"] = torch.full((h,), 5.0, device="cuda")
        grads["b2"] = torch.full((1,), 5.0, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(HT.arrol_head_grad_workspace(ctx, N, d, h), dtype=torch.uint8, device="cuda")
    HT.arrol_head_grad(ctx, x.cuda(), dhead, N, torch.from_numpy(rew).cuda(), grads, loss, ws,
                       row_index=torch.from_numpy(ridx).cuda(), mask=None if mask is None else torch.from_numpy(mask).cuda())
    torch.cuda.synchronize()
    assert abs(loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))
    for k, ref in gref.items():
        got = grads[k].cpu().numpy().reshape(ref.shape).astype(np.float64)
        assert np.abs(got - ref).max() <= 2e-4 * max(np.abs(ref).max(), 1e-6), k
    ctx.close()


def test_head_grad_empty_inputs():
    ctx = B.Context(0)
    d = 64
    head = {"W1": torch.zeros(d, device="cuda"), "b1": None, "w2": None, "b2": None, "h": 0}
    grads = {"W1": torch.full((d,), 5.0, device="cuda"), "b1": torch.full((1,), 5.0, device="cuda")}
    loss = torch.ones(1, dtype=torch.float64, device="cuda")
    x = torch.zeros(4, d, device="cuda")
    HT.arrol_head_grad(ctx, x, head, 0, torch.zeros(4, device="cuda"), grads, loss, None)
    torch.cuda.synchronize()
    assert loss.item() == 0.0 and torch.all(grads["W1"] == 0) and grads["b1"].item() == 0.0
    ws = torch.empty(HT.arrol_head_grad_workspace(ctx, 4, d, 0), dtype=torch.uint8, device="cuda")
    HT.arrol_head_grad(ctx, x, head, 4, torch.zeros(4, device="cuda"), grads, loss, ws,
                       mask=torch.zeros(4, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert loss.item() == 0.0 and torch.all(grads["W1"] == 0)
    ctx.close()


def test_head_grad_rows_in_place_on_the_tensor_core_path():
    """bf16 MLP head without a row index: the contractions read the rows where they are (no packing)."""
    ctx = B.Context(0)
    g = np.random.default_rng(21)
    N, d, h = 200, 512, 128
    x = torch.from_numpy(g.normal(size=(N, d)).astype(np.float32)).to(torch.bfloat16)
    mk = lambda *s: torch.from_numpy(g.normal(0, 0.05, size=s).astype(np.float32)).to(torch.bfloat16)
    head = {"W1": mk(h, d), "b1": mk(h), "w2": mk(h) * 4, "b2": mk(1)}
    rew = (g.random(N) < 0.4).astype(np.float32)
    oa = synth.as_oracle_array
    loss_ref, gref = oh.head_bce_grad(oa(x), rew > 0.5, oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]), h=h)
    dhead = {k: v.cuda() for k, v in head.items()}
    dhead["h"] = h
    grads = {"W1": torch.full((h, d), 5.0, device="cuda"), "b1": torch.full((h,), 5.0, device="cuda"),
             "w2": torch.full((h,), 5.0, device="cuda"), "b2": torch.full((1,), 5.0, device="cuda")}
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(HT.arrol_head_grad_workspace(ctx, N, d, h), dtype=torch.uint8, device="cuda")
    HT.arrol_head_grad(ctx, x.cuda(), dhead, N, torch.from_numpy(rew).cuda(), grads, loss, ws)
    torch.cuda.synchronize()
    assert abs(loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))
    for k, ref in gref.items():
        got = grads[k].cpu().numpy().reshape(ref.shape).astype(np.float64)
        assert np.abs(got - ref).max() <= 2e-4 * max(np.abs(ref).max(), 1e-6), k
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    ctx.close()
