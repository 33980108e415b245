"""The tensor-core kernels' pipeline waits are bounded.  A test hook silences the log-prob kernel's producer so that
the other roles' waits run out: the kernel must return (no hang, no fault), report it in the status word, and leave
the context usable."""
import pytest
import torch

from paper_2603_24840_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d,V", [(300, 256, 1000), (40000, 512, 4096)])     # one block with work / every SM busy
def test_expired_waits_are_reported_and_the_context_stays_usable(T, d, V):
    ctx = B.Context(0)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(T)
    hidden = torch.randn((T, d), generator=gen, device="cuda").to(torch.bfloat16)
    W = (torch.randn((V, d), generator=gen, device="cuda") * 0.05).to(torch.bfloat16)
    targets = torch.randint(0, V, (T,), generator=gen, device="cuda", dtype=torch.int32)
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")

    def run():
        logp = torch.full((T,), 7.0, device="cuda")
        lse = torch.full((T,), 7.0, device="cuda")
        B.arrol_token_logprob(ctx, hidden, W, targets, T, d, V, logp, ws, lse=lse)
        torch.cuda.synchronize()
        return logp, lse

    want_logp, want_lse = run()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0

    B.arrol_test_hook(ctx, B.HOOK_SPIN_LIMIT, 2000)
    B.arrol_test_hook(ctx, B.HOOK_MUTE_LOGPROB_PRODUCER, 1)
    run()                                                        # returns: every wait gives up after 2000 tries
    assert B.arrol_poll_status(ctx, raise_on_error=False) & B.DEV_WAIT_EXPIRED
    with pytest.raises(B.ArrolError) as e:                       # and the public call reports it as an error
        run()
        B.arrol_poll_status(ctx)
    assert e.value.code == -6

    B.arrol_test_hook(ctx, B.HOOK_MUTE_LOGPROB_PRODUCER, 0)
    B.arrol_test_hook(ctx, B.HOOK_SPIN_LIMIT, 0)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0   # the status word was cleared by the poll above
    logp, lse = run()
    assert torch.equal(logp, want_logp) and torch.equal(lse, want_lse)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0

    with pytest.raises(B.ArrolError):
        B.arrol_test_hook(ctx, 99, 0)
    ctx.close()
