"""Attention profiling for the budget of Eq. 10, through the library: the first layer of each
attention type is measured (CUDA events around the caller's region), later layers of the type
reuse the measurement, and B_l = max(0, T_attn[r(l)] - delta)."""
import pytest
import torch

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from tests import parity_util as P

pytestmark = pytest.mark.gpu


def _stand_in_attention(x, reps):
    for _ in range(reps):
        x = x @ x.T @ x * 1e-3
    return x


def test_budget_arithmetic_and_reuse_match_the_oracle():
    ctx = P.make_context(I.WORKLOADS["tiny"], 128)
    types = ["full", "linear", "linear", "full", "sparse", "full"]
    type_id = {"full": 0, "linear": 1, "sparse": 2}
    times = {0: 700_000, 1: 150_000, 4: 90_000}
    first = {}
    got = []
    for l, t in enumerate(types):
        if t not in first:                              # r(l): install the measurement of the first layer of the type
            first[t] = l
            ctx.fb_attention_set_time_ns(type_id[t], l, times[l])
        budget, r_l = ctx.fb_layer_budget_ns(type_id[t], 100_000)
        assert r_l == first[t]
        got.append(budget)
    assert got == O.budgets_by_attention_type(types, times, 100_000) == [600_000, 50_000, 50_000, 600_000, 0, 600_000]
    with pytest.raises(B.FbError) as e:                  # a type that was never profiled has no budget
        ctx.fb_layer_budget_ns(5, 0)
    assert e.value.status == B.FB_ERR_INVALID_ARG
    ctx.fb_attention_reset()
    with pytest.raises(B.FbError):
        ctx.fb_layer_budget_ns(0, 0)
    ctx.close()


def test_measured_region_and_first_layer_reuse():
    dev = torch.device("cuda", 0)
    ctx = P.make_context(I.WORKLOADS["tiny"], 128)
    x = torch.randn(2048, 2048, device=dev)
    _stand_in_attention(x, 2)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # layer 0 (type 0, long region), layer 1 (type 1, short region), layers 2, 3 (type 0 again, short regions)
    plan = [(0, 0, 6), (1, 1, 1), (2, 0, 1), (3, 0, 1)]
    ref_ms = {}
    for layer, typ, reps in plan:
        ctx.fb_attention_begin(layer, typ)
        e0.record()
        _stand_in_attention(x, reps)
        e1.record()
        ctx.fb_attention_end(layer, typ)
        torch.cuda.synchronize()
        ref_ms[layer] = e0.elapsed_time(e1)
    b0, r0 = ctx.fb_layer_budget_ns(0, 0)
    b1, r1 = ctx.fb_layer_budget_ns(1, 0)
    assert (r0, r1) == (0, 1)                            # later layers of type 0 did not replace layer 0's time
    assert abs(b0 - ref_ms[0] * 1e6) <= 0.1 * ref_ms[0] * 1e6 + 20_000
    assert abs(b1 - ref_ms[1] * 1e6) <= 0.1 * ref_ms[1] * 1e6 + 20_000
    assert b0 > 3 * b1                                   # 6 repetitions against 1
    delta = b0 // 2
    assert ctx.fb_layer_budget_ns(0, delta)[0] == b0 - delta             # Eq. 10
    assert ctx.fb_layer_budget_ns(0, 2 * b0)[0] == 0                      # never negative
    assert B.fb_budget_ns(b0, delta) == O.budget_ns(b0, delta)
    ctx.close()
