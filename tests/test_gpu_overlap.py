"""The two-stream overlap experiment of bench.py (--overlap) on a reduced size: it runs, the
stand-in attention takes the SMs it was given, and the figures are consistent with each other."""
import pytest
import torch

import bench
from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_standin_attention_scales_with_iterations_not_with_blocks():
    dev = torch.device("cuda", 0)
    sink = torch.zeros(1024 * 1024, device=dev)

    def t(blocks, iters):
        B.fb_standin_attention(sink, blocks, iters)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        B.fb_standin_attention(sink, blocks, iters)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    base = t(n_sm, 4000)
    assert 1.6 < t(n_sm, 8000) / base < 2.4            # time follows the iteration count
    assert 0.7 < t(n_sm // 2, 4000) / base < 1.3       # one block per SM: fewer blocks, same time
    with pytest.raises(B.FbError):
        B.fb_standin_attention(sink, 0, 10)


def test_overlap_experiment_is_consistent():
    wl = I.WORKLOADS["dsv3"]
    rep = bench.run_overlap(wl, B, torch.device("cuda", 0), window_us=300.0, reps=3, pair_limits=(8, 32), T=8192,
                            expert_bytes=4 * 2**20)
    assert rep["device_status"] == 0 and len(rep["rows"]) == 2
    for row in rep["rows"]:
        assert row["attention_sms"] == rep["sms"] - 2 * row["router_pairs"]
        assert 0.5 * 300 < row["attention_us"] < 2.0 * 300
        assert abs(row["window_us"] - row["attention_us"]) < 0.25 * row["attention_us"]      # the library's own profile
        assert abs(row["budget_us"] - 0.9 * row["window_us"]) < 1.0
        for key in ("exchange_kernel", "exchange_copies"):
            r = row[key]
            # together is never shorter than either part alone (within timing noise) ...
            assert r["together_us"] > 0.9 * max(row["attention_us"], r["auxiliary_alone_us"])
            # ... and never longer than running them one after the other
            assert r["together_us"] < 1.15 * (row["attention_us"] + r["auxiliary_alone_us"]) + 30
        assert row["swaps"] >= 0
