"""Token sharding on one GPU: the shards' histograms, summed (what the all-reduce does), give
the whole batch's histogram and therefore the same plan as the unsharded call."""
import pytest
import torch

from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from paper_2608_14205_b200.sharded import ShardedPredictor, shard_bounds
from tests import parity_util as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,T,world", [("tiny", 500, 2), ("qwen3", 1000, 3), ("dsv3", 2049, 4)])
def test_shards_sum_to_the_whole_batch(name, T, world):
    wl = I.WORKLOADS[name]
    dev = torch.device("cuda")
    li = I.make_layer(wl, 1, 0, T=T)
    ctx = P.make_context(wl, T)
    budget = B.make_budget(**P.budget_kwargs(wl, T))
    sb = li.select_bias.to(dev) if li.select_bias is not None else None
    router = B.make_router(li.W.to(dev), None, sb)
    h = li.h_prev.to(dev)
    pi = li.expert_to_slot.to(dev)
    i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
    ms = max(1, budget.max_swaps)
    # unsharded
    c0, p0, s0, n0, lb0, la0 = i32(wl.E), i32(wl.E), i32(4 * ms), i32(1), i32(wl.R), i32(wl.R)
    ctx.fb_predict_and_plan(router, h, T, pi, budget, 0, c0, p0, s0, n0, lb0, la0)
    # the ranks' local passes one after the other, then the sum, then the planner every rank would run
    total = i32(wl.E)
    part = i32(wl.E)
    for r in range(world):
        lo, hi = shard_bounds(T, world, r)
        ctx.fb_predict_load(router, h[lo:hi].contiguous(), hi - lo, part)
        total += part
    c1, p1, s1, n1, lb1, la1 = total, i32(wl.E), i32(4 * ms), i32(1), i32(wl.R), i32(wl.R)
    ctx.fb_plan_swaps(c1, pi, budget, 0, p1, s1, n1, lb1, la1)
    torch.cuda.synchronize()
    assert torch.equal(c0, c1) and torch.equal(p0, p1) and int(n0) == int(n1)
    assert torch.equal(s0[:4 * int(n0)], s1[:4 * int(n1)]) and torch.equal(la0, la1)
    # a single process is the degenerate group: ShardedPredictor reduces to the two calls
    c2, p2, s2, n2, lb2, la2 = i32(wl.E), i32(wl.E), i32(4 * ms), i32(1), i32(wl.R), i32(wl.R)
    ShardedPredictor(ctx).predict_and_plan(router, h, T, pi, budget, 0, c2, p2, s2, n2, lb2, la2)
    torch.cuda.synchronize()
    assert torch.equal(c0, c2) and torch.equal(p0, p2) and torch.equal(la0, la2)
    ctx.close()
