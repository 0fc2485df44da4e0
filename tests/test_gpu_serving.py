"""GPU parity of the multi-step serving loop and the quality metrics against the oracle."""
import numpy as np
import pytest
import torch

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I
from paper_2608_14205_b200 import serving as S
from tests.test_oracle_serving import _budget, _gate, bits

pytestmark = pytest.mark.gpu


def _oracle_trace(layers_cpu):
    for (s, l), li in layers_cpu.items():
        sb = li.select_bias.numpy().astype(np.float64) if li.select_bias is not None else None
        yield s, l, bits(li.h_prev), bits(li.H), bits(li.W), sb, None


@pytest.mark.parametrize("name,T,steps,layers,sys_drift,quality", [
    ("tiny", 300, 3, 2, 0.0, True), ("tiny", 300, 3, 2, 0.0, False),
    ("qwen3", 700, 3, 2, 0.25, True),
    ("dsv3", 640, 3, 2, 0.25, True), ("dsv3", 640, 3, 2, 0.5, False),
])
def test_serving_loop_matches_the_oracle(name, T, steps, layers, sys_drift, quality):
    wl = I.WORKLOADS[name]
    cpu = {(s, l): I.make_step_layer(wl, l, s, 0, T=T, sys_drift=sys_drift)
           for s in range(steps) for l in range(layers)}
    records, summary, placements = O.serving_loop(_oracle_trace(cpu), _gate(wl), wl.R, _budget(wl, T))
    loop = S.ServingLoop(wl, T)
    budget = S.make_budget_for(wl, T)
    dev = loop.dev
    for rec, ((s, l), li) in zip(records, cpu.items()):
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        router = B.make_router(li.W.to(dev), None, sb)
        r = loop.layer_step(l, router, li.h_prev.to(dev), li.H.to(dev), budget, quality=quality)
        torch.cuda.synchronize(dev)
        o = r["out"]
        assert loop.ctx.fb_device_status() == 0
        assert r["pi_old"].cpu().tolist() == rec["pi_old"], "placement carried over from the previous step"
        n = int(o["n_swaps"].item())
        swaps = [tuple(x) for x in o["swaps"].cpu().numpy().reshape(-1, 4)[:n].tolist()]
        assert o["counts"].cpu().tolist() == rec["counts"].tolist()
        assert swaps == rec["swaps"] and r["pi_new"].cpu().tolist() == rec["pi_new"]
        realized, before, after, vanilla = loop.realised_loads(r, budget)
        assert realized == rec["realized"].tolist()
        assert O.max_over_mean(before) == rec["real_before"] and O.max_over_mean(after) == rec["real_after"]
        assert O.max_over_mean(vanilla) == rec["real_vanilla"]
        if quality:
            assert r["hit_rate"] == rec["hit_rate"]
            assert r["cos_hidden"] == pytest.approx(rec["cos_hidden"], abs=1e-12)     # same bf16 inputs, fp64 sums
            assert r["cos_logits"] == pytest.approx(rec["cos_logits"], abs=1e-5)      # fp32 vs fp64 logits
    for l in range(layers):
        assert loop.placement_of(l).cpu().tolist() == placements[l]
    loop.close()


def test_metric_kernels_on_constructed_inputs():
    dev = torch.device("cuda")
    a = torch.tensor([[1.0, 0.0, 0.0], [0.0, 0.0, 0.0], [1.0, 1.0, 0.0], [2.0, 0.0, 0.0]], device=dev)
    b = torch.tensor([[0.0, 3.0, 0.0], [1.0, 2.0, 3.0], [1.0, 0.0, 0.0], [-5.0, 0.0, 0.0]], device=dev)
    rows = torch.zeros(4, dtype=torch.float64, device=dev)
    mean = torch.zeros(1, dtype=torch.float64, device=dev)
    B.fb_row_cosine_mean(a, b, rows, mean)
    assert rows.cpu().tolist() == pytest.approx([0.0, 0.0, 2 ** -0.5, -1.0], abs=1e-15)
    assert mean.item() == pytest.approx((2 ** -0.5 - 1.0) / 4, abs=1e-15)
    ab, bb = a.to(torch.bfloat16), b.to(torch.bfloat16)
    B.fb_row_cosine_mean(ab, bb, rows, mean)
    assert mean.item() == pytest.approx((2 ** -0.5 - 1.0) / 4, abs=1e-15)
    B.fb_row_cosine_mean(a[:0], b[:0], rows, mean)
    assert mean.item() == 0.0
    # ragged width, many rows: against the oracle's definition
    g = torch.Generator().manual_seed(5)
    x, y = torch.randn(1000, 77, generator=g), torch.randn(1000, 77, generator=g)
    rows = torch.zeros(1000, dtype=torch.float64, device=dev)
    B.fb_row_cosine_mean(x.to(dev), y.to(dev), rows, mean)
    assert mean.item() == pytest.approx(O.row_cosine_mean(x.numpy(), y.numpy()), abs=1e-13)

    ids_a = torch.tensor([[0, 1, 2], [3, 4, 5], [6, 7, 8]], dtype=torch.int32, device=dev)
    ids_b = torch.tensor([[2, 1, 0], [5, 9, 10], [11, 12, 13]], dtype=torch.int32, device=dev)
    hits = torch.zeros(1, dtype=torch.int32, device=dev)
    B.fb_topk_hits(ids_a, ids_b, 3, 3, hits)
    assert hits.item() == 4
    assert O.topk_hit_rate(ids_a.cpu().numpy(), ids_b.cpu().numpy()) == pytest.approx(4 / 9)
    B.fb_topk_hits(ids_a, ids_b, 0, 3, hits)
    assert hits.item() == 0
    with pytest.raises(B.FbError):
        B.fb_topk_hits(ids_a, ids_b, 3, 9, hits)
