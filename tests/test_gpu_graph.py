"""The library's calls inside a CUDA graph: captured once, replayed on new inputs.

The calls allocate nothing, never synchronise and keep no per-launch state on the host that a kernel
depends on (the k-range split's partial-tile flags are put back by the kernel that consumed them), so a
captured sequence can be replayed; every replay must give the bits the same calls give when made directly.
"""
import numpy as np
import pytest
import torch

from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from tests import parity_util as P

pytestmark = pytest.mark.gpu


def _buffers(wl, T, dev):
    i32 = lambda n: torch.full((max(1, n),), -3, dtype=torch.int32, device=dev)
    return dict(counts=i32(wl.E), pi_out=i32(wl.E), swaps=i32(4 * max(1, wl.E // 2)), n=i32(1), lb=i32(wl.R), la=i32(wl.R),
                l_counts=i32(wl.E), l_pi_out=i32(wl.E), l_swaps=i32(4 * max(1, wl.E // 2)), l_n=i32(1), l_lb=i32(wl.R),
                l_la=i32(wl.R), ids=i32(T * wl.k), w=torch.zeros(max(1, T * wl.k), device=dev), so=i32(wl.E + 1),
                ro=i32(wl.R + 1), perm=i32(T * wl.k), inv=i32(T * wl.k), rl=i32(wl.R))


def _calls(ctx, router, x, H, T, pi, budget, o):
    ctx.fb_predict_and_plan(router, x, T, pi, budget, 0, o["counts"], o["pi_out"], o["swaps"], o["n"], o["lb"], o["la"])
    ctx.fb_layer_step(router, x, H, T, pi, budget, 0, o["l_counts"], o["l_pi_out"], o["l_swaps"], o["l_n"], o["l_lb"],
                      o["l_la"], o["ids"], o["w"], o["so"], o["ro"], o["perm"], o["inv"], o["rl"])


@pytest.mark.parametrize("name,T,pair_limit", [("qwen3", 2000, 0), ("mixtral", 1000, 0), ("dsv3", 1500, 0),
                                                ("dsv3", 1500, 2)])
def test_captured_calls_replay_bit_for_bit(name, T, pair_limit):
    # qwen3 / mixtral at these sizes run with the k-range split (helper pairs and their flags),
    # dsv3 with a pair limit runs the persistent kernel; every form must survive a replay.
    wl = I.WORKLOADS[name]
    layers = [I.make_layer(wl, l, 0, T=T) for l in range(3)]
    ctx = P.make_context(wl, T)
    ctx.fb_set_pair_limit(pair_limit)
    dev = torch.device("cuda", ctx.device)
    W = layers[0].W.to(dev)
    sb = layers[0].select_bias.to(dev) if layers[0].select_bias is not None else None
    router = B.make_router(W, None, sb)
    pi = layers[0].expert_to_slot.to(dev)
    budget = B.make_budget(**P.budget_kwargs(wl, T))
    x, H = layers[0].h_prev.to(dev).clone(), layers[0].H.to(dev).clone()

    eager = _buffers(wl, T, dev)
    want = []
    for li in layers:                       # the same calls made directly, on each input in turn
        x.copy_(li.h_prev.to(dev)); H.copy_(li.H.to(dev))
        _calls(ctx, router, x, H, T, pi, budget, eager)
        torch.cuda.synchronize(dev)
        want.append({k: v.clone() for k, v in eager.items()})
    assert ctx.fb_device_status() == 0

    out = _buffers(wl, T, dev)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            _calls(ctx, router, x, H, T, pi, budget, out)
    torch.cuda.current_stream(dev).wait_stream(side)
    for rep in range(2):
        for li, ref in zip(layers, want):
            x.copy_(li.h_prev.to(dev)); H.copy_(li.H.to(dev))
            graph.replay()
            torch.cuda.synchronize(dev)
            n, ln = int(ref["n"].item()), int(ref["l_n"].item())
            for key in out:
                a, b = out[key], ref[key]
                if key == "swaps":
                    a, b = a[:4 * n], b[:4 * n]
                if key == "l_swaps":
                    a, b = a[:4 * ln], b[:4 * ln]
                assert torch.equal(a, b), (rep, key)
            assert int(out["counts"].sum().item()) == T * wl.k
    assert ctx.fb_device_status() == 0
    ctx.fb_set_pair_limit(0)
    ctx.close()
