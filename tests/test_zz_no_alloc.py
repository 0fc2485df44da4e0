"""The allocation-free prediction entry point.

Some callers may not allocate device memory at all: a serving engine that has frozen
its memory pool, or a host that is not allowed to create a library context because
creating one calls cudaMalloc.  For them the library offers fb_predict_load_static,
whose kernel scratch is a fixed array inside the library image.  This file checks,
through the C ABI, that it returns exactly what fb_predict_load returns - twice in a
row, because the second call finds the array as the first one left it.

The file name sorts last so that a run that stops at the first failure has already
been through every other test.
"""
import pytest
import torch

from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from tests import parity_util as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,T", [("dsv3", 1000), ("qwen3", 777), ("tiny", 512)])
def test_static_entry_matches_context_entry_twice(name, T):
    wl = I.WORKLOADS[name]
    dev = torch.device("cuda", 0)
    layers = [I.make_layer(wl, layer, 0, T=T) for layer in (0, 1)]
    cfg = B.FbConfig(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    prepared = []
    for li in layers:                                   # two calls in a row, different inputs
        W = li.W.to(dev)
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        router = B.make_router(W, None, sb)
        x = li.h_prev.to(dev)
        want_counts = torch.full((wl.E,), -1, dtype=torch.int32, device=dev)
        want_ids = torch.full((T * wl.k,), -1, dtype=torch.int32, device=dev)
        got_counts = torch.full((wl.E,), -2, dtype=torch.int32, device=dev)
        got_ids = torch.full((T * wl.k,), -2, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        prepared.append((router, x, want_counts, want_ids, got_counts, got_ids, status))
    # The first call comes before any context of this shape exists (when this file runs alone
    # it is the first launch of these kernels in the process: the driver may load the kernel
    # image onto the device during it, which is the one thing the entry point cannot avoid).
    router, x, _, _, got_counts, got_ids, status = prepared[0]
    B.fb_predict_load_static(cfg, 0, router, x, T, got_counts, got_ids, status)
    torch.cuda.synchronize(dev)
    # From the second call on, nothing is taken from the device: free memory stays where it was.
    free_before = torch.cuda.mem_get_info(dev)[0]
    router, x, _, _, got_counts, got_ids, status = prepared[1]
    B.fb_predict_load_static(cfg, 0, router, x, T, got_counts, got_ids, status)
    torch.cuda.synchronize(dev)
    assert torch.cuda.mem_get_info(dev)[0] >= free_before
    # the reference results, through a context running the same kernel (the static entry has no
    # room for the partial tiles of the k-range split, so the context switches its split off)
    ctx = P.make_context(wl, T)
    ctx.fb_set_split(0)
    for router, x, want_counts, want_ids, _, _, _ in prepared:
        ctx.fb_predict_load(router, x, T, want_counts, want_ids)
    assert ctx.fb_device_status() == 0
    torch.cuda.synchronize(dev)
    for router, x, want_counts, want_ids, got_counts, got_ids, status in prepared:
        assert int(status.item()) == 0
        assert torch.equal(got_counts, want_counts)     # integer outputs: bit-exact
        assert torch.equal(got_ids, want_ids)
        assert int(got_counts.sum().item()) == T * wl.k
    ctx.close()


def test_static_entry_rejects_sizes_beyond_its_array():
    dev = torch.device("cuda", 0)
    W = torch.zeros(8, 64, dtype=torch.bfloat16, device=dev)
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device=dev)
    counts = torch.zeros(512, dtype=torch.int32, device=dev)
    too_many = B.FbConfig(16, 64, 300, 2, 4, 0, 1, 1, 1, 1.0)          # E = 300 > FB_STATIC_MAX_EXPERTS
    with pytest.raises(B.FbError) as e:
        B.fb_predict_load_static(too_many, 0, B.make_router(W), x, 16, counts)
    assert e.value.status == B.FB_ERR_UNSUPPORTED_SHAPE
    ok = B.FbConfig(16, 64, 8, 2, 4, 0, 1, 1, 1, 1.0)
    with pytest.raises(B.FbError) as e:
        B.fb_predict_load_static(ok, 0, B.make_router(W), x, 17, counts)   # T > T_max
    assert e.value.status == B.FB_ERR_UNSUPPORTED_SHAPE
    B.fb_predict_load_static(ok, 0, B.make_router(W), x, 16, counts)        # all logits equal: experts 0 and 1
    torch.cuda.synchronize(dev)
    assert counts[:8].tolist() == [16, 16, 0, 0, 0, 0, 0, 0]


def test_static_entry_beside_contexts_of_other_shapes():
    """The static entry keeps no context, but it shares its kernels with every live context.
    Calls with three shapes alternate with calls through a context of yet another shape; the
    static entry changes shape from one call to the next (its shape-dependent set-up runs
    again within this one test) and each result must equal the context entry's."""
    dev = torch.device("cuda", 0)
    T = 600
    big = P.make_context(I.WORKLOADS["dsv3"], T)                       # alive throughout
    big.fb_set_split(0)                                                # like with like: see the test above
    big_li = I.make_layer(I.WORKLOADS["dsv3"], 0, 0, T=T)
    big_router = B.make_router(big_li.W.to(dev), None, big_li.select_bias.to(dev))
    big_x = big_li.h_prev.to(dev)
    big_want = torch.zeros(256, dtype=torch.int32, device=dev)
    big.fb_predict_load(big_router, big_x, T, big_want)
    for name in ("tiny", "qwen3", "dsv3", "tiny"):
        wl = I.WORKLOADS[name]
        li = I.make_layer(wl, 1, 0, T=T)
        cfg = B.FbConfig(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
        router = B.make_router(li.W.to(dev), None, li.select_bias.to(dev) if li.select_bias is not None else None)
        x = li.h_prev.to(dev)
        ctx = P.make_context(wl, T)
        ctx.fb_set_split(0)
        want = torch.full((wl.E,), -1, dtype=torch.int32, device=dev)
        ctx.fb_predict_load(router, x, T, want)
        got = torch.full((wl.E,), -2, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.fb_predict_load_static(cfg, 0, router, x, T, got, None, status)
        again = torch.full((256,), -3, dtype=torch.int32, device=dev)
        big.fb_predict_load(big_router, big_x, T, again)               # the other shape still launches
        torch.cuda.synchronize(dev)
        assert int(status.item()) == 0 and ctx.fb_device_status() == 0 and big.fb_device_status() == 0
        assert torch.equal(got, want), name
        assert torch.equal(again, big_want), name
        ctx.close()
    big.close()
