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
    ctx = P.make_context(wl, T)
    cfg = B.FbConfig(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    prepared = []
    for li in layers:                                   # two calls in a row, different inputs
        W = li.W.to(dev)
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        router = B.make_router(W, None, sb)
        x = li.h_prev.to(dev)
        want_counts = torch.full((wl.E,), -1, dtype=torch.int32, device=dev)
        want_ids = torch.full((T * wl.k,), -1, dtype=torch.int32, device=dev)
        ctx.fb_predict_load(router, x, T, want_counts, want_ids)
        assert ctx.fb_device_status() == 0
        got_counts = torch.full((wl.E,), -2, dtype=torch.int32, device=dev)
        got_ids = torch.full((T * wl.k,), -2, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        prepared.append((router, x, want_counts, want_ids, got_counts, got_ids, status))
    torch.cuda.synchronize(dev)
    free_before = torch.cuda.mem_get_info(dev)[0]
    for router, x, want_counts, want_ids, got_counts, got_ids, status in prepared:
        B.fb_predict_load_static(cfg, 0, router, x, T, got_counts, got_ids, status)
    torch.cuda.synchronize(dev)
    # the two calls took nothing from the device allocator (small slack for lazy driver state)
    assert torch.cuda.mem_get_info(dev)[0] >= free_before - (4 << 20)
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
