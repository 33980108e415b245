"""GPU parity of the policy-update calls against the oracle: clipped GRPO / DAPO loss and its gradient (fp32 per
token: 1e-6 relative to the weight scale), and the lm_head log-prob backward (dz is rounded to bf16 before the two
contractions: 1e-2 of the tensor's largest entry, 5e-3 in relative Frobenius norm)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import update as ou
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200 import update as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    assert B.arrol_poll_status(c, raise_on_error=False) == 0
    c.close()


def dv(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("S,lo,hi,agg_mode,beta", [(16, 1, 40, 0, 0.0), (300, 5, 900, 1, 0.0), (64, 1, 300, 0, 0.04),
                                                   (7, 0, 3, 1, 0.1)])
def test_policy_loss_matches_oracle(ctx, S, lo, hi, agg_mode, beta):
    g = np.random.default_rng(S)
    ell = g.integers(lo, hi + 1, size=S)
    ell[0] = max(ell[0], 1)
    cu = np.concatenate([[0], np.cumsum(ell)]).astype(np.int64)
    T = int(cu[-1])
    logp_old = (-g.random(T) * 4).astype(np.float32)
    logp = (logp_old + g.normal(0, 0.25, size=T)).astype(np.float32)
    ref = (logp_old + g.normal(0, 0.2, size=T)).astype(np.float32)
    adv = np.repeat(g.normal(size=S), ell).astype(np.float32)
    seq = np.repeat(np.arange(S), ell).astype(np.int32)
    loss_ref, grad_ref = ou.policy_loss(logp, logp_old, adv, cu, logp_ref=ref if beta else None, eps_low=0.2,
                                        eps_high=0.28, beta=beta, agg_mode=agg_mode)
    cap = T + 5
    pad = lambda a, fill: np.concatenate([a, np.full(cap - T, fill, a.dtype)])
    grad = torch.full((cap,), 77.0, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    U.arrol_policy_loss(ctx, dv(pad(logp, 0)), dv(pad(logp_old, 0)), dv(pad(adv, 0)), dv(pad(seq, 0)), dv(cu),
                        dv(np.array([S, T], np.int64)), cap, grad, loss, logp_ref=dv(pad(ref, 0)) if beta else None,
                        eps_low=0.2, eps_high=0.28, beta=beta, agg_mode=agg_mode)
    torch.cuda.synchronize()
    w_max = 1.0 / T if agg_mode else 1.0 / (S * max(1, ell[ell > 0].min()))
    assert np.abs(grad.cpu().numpy()[:T] - grad_ref).max() <= 2e-5 * w_max * max(1.0, np.abs(adv).max())
    assert np.all(grad.cpu().numpy()[T:] == 77.0)
    assert abs(loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))


def _backward_case(ctx, T, d, V, seed, T_live=None, inv_temp=1.0):
    g = np.random.default_rng(seed)
    H = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(g.normal(0, 0.08, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    y = g.integers(0, V, size=T).astype(np.int32)
    y[:4] = [0, V - 1, -1, min(255, V - 1)][:min(4, T)] if T >= 4 else y[:4]
    gl = g.normal(size=T).astype(np.float32)
    n = T if T_live is None else T_live
    dH_ref, dW_ref = ou.lm_head_backward(synth.as_oracle_array(H[:n]), synth.as_oracle_array(W), y[:n],
                                         gl[:n].astype(np.float64), inv_temp=inv_temp)
    Hd, Wd, yd = H.cuda(), W.cuda(), dv(y)
    if T_live is not None:
        Hd[T_live:] = float("nan")               # rows past the live tokens may hold anything
    logp = torch.empty(T, device="cuda")
    lse = torch.empty(T, device="cuda")
    d_T = None if T_live is None else torch.tensor([T_live], dtype=torch.int64, device="cuda")
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    B.arrol_token_logprob(ctx, Hd, Wd, yd, T, d, V, logp, ws, lse=lse, d_T=d_T, inv_temperature=inv_temp)
    dH = torch.full((T, d), 9.0, device="cuda")
    dW = torch.full((V, d), 9.0, device="cuda")
    ws2 = torch.empty(U.arrol_lm_head_backward_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    U.arrol_lm_head_backward(ctx, Hd, Wd, yd, dv(gl), lse, T, d, V, dH, dW, ws2, d_T=d_T, inv_temperature=inv_temp)
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    dH, dW = dH.cpu().numpy().astype(np.float64), dW.cpu().numpy().astype(np.float64)
    for got, ref in ((dH[:n], dH_ref), (dW, dW_ref)):
        scale = np.abs(ref).max()
        assert np.abs(got - ref).max() <= 1e-2 * scale
        assert np.linalg.norm(got - ref) <= 5e-3 * np.linalg.norm(ref)
    assert np.all(dH[:n][y[:n] < 0] == 0.0)                    # ignored positions carry no gradient
    return dH, n


@pytest.mark.parametrize("T,d,V", [(1, 64, 256), (130, 64, 300), (300, 192, 1000), (700, 256, 3001), (257, 200, 37)])
def test_lm_head_backward_matches_oracle(ctx, T, d, V):
    _backward_case(ctx, T, d, V, seed=T + V)


def test_lm_head_backward_many_chunks_temperature_and_device_T(ctx):
    _backward_case(ctx, 10000, 64, 512, seed=1)               # two token chunks: dW accumulates across them
    _backward_case(ctx, 400, 128, 1024, seed=2, inv_temp=0.6)
    dH, n = _backward_case(ctx, 600, 128, 1024, seed=3, T_live=333)
    assert np.all(dH[n:] == 0.0)                               # rows past T inside a processed chunk are zero
    _backward_case(ctx, 600, 128, 1024, seed=4, T_live=320)    # live rows end exactly on a 64-row block
    _backward_case(ctx, 9700, 64, 512, seed=5, T_live=9500)    # the partly live block is in the second chunk


def test_update_argument_errors(ctx):
    z = torch.zeros(8, device="cuda")
    with pytest.raises(B.ArrolError) as e:
        U.arrol_lm_head_backward(ctx, z, z, z, z, z, 8, 60, 64, z, z, None)
    assert e.value.code == -2
    with pytest.raises(B.ArrolError) as e:
        U.arrol_lm_head_backward(ctx, z, z, z, z, z, 8, 64, 64, z, torch.zeros(64 * 64, device="cuda"), None)
    assert e.value.code == -3
    with pytest.raises(B.ArrolError) as e:
        U.arrol_policy_loss(ctx, z, z, z, None, z, z, 8, z, torch.zeros(1, dtype=torch.float64, device="cuda"),
                            agg_mode=2)
    assert e.value.code == -2
