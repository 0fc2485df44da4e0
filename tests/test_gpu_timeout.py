"""A bounded device-side wait that really runs out.

Every wait inside the library's kernels (on a TMA transfer, on an MMA commit, on a partner
block) carries a time limit; when it expires the kernel records FB_ERR_TIMEOUT in the device
status word and leaves through its normal exit.  Nothing traps, so the context and the GPU stay
usable.  Here the wait is made to expire in the only safe way: a tiny kernel waits for at most
a millisecond on a barrier at which nobody ever arrives.
"""
import pytest
import torch

from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from tests import parity_util as P

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_the_status_word_and_leaves_the_context_usable():
    wl = I.WORKLOADS["tiny"]
    T = 300
    dev = torch.device("cuda", 0)
    ctx = P.make_context(wl, T)
    li = I.make_layer(wl, 0, 0, T=T)
    bkw = P.budget_kwargs(wl, T)
    assert ctx.fb_device_status() == 0
    waited = torch.zeros(1, dtype=torch.int64, device=dev)
    limit_ns = 1_000_000                                   # one millisecond
    ctx.fb_selftest_wait_timeout(limit_ns, waited)
    assert ctx.fb_device_status() == B.FB_ERR_TIMEOUT      # reported ...
    assert ctx.fb_device_status() == 0                     # ... once, then cleared
    t = int(waited.item())
    assert limit_ns <= t < 50 * limit_ns, t                # it waited for the limit, not for ever
    # the next normal calls are clean and correct
    gpu = P.run_gpu_layer(ctx, wl, li, bkw)
    P.compare_layer(wl, li, bkw, gpu)
    # a shorter limit, twice in a row, on another stream
    side = torch.cuda.Stream()
    for _ in range(2):
        ctx.fb_selftest_wait_timeout(10_000, None, stream=side)
    assert ctx.fb_device_status(stream=side) == B.FB_ERR_TIMEOUT
    assert ctx.fb_device_status() == 0
    ctx.close()


def test_selftest_rejects_unbounded_limits():
    ctx = P.make_context(I.WORKLOADS["tiny"], 128)
    for bad in (0, 10**9):
        with pytest.raises(B.FbError) as e:
            ctx.fb_selftest_wait_timeout(bad)
        assert e.value.status == B.FB_ERR_INVALID_ARG
    ctx.close()
