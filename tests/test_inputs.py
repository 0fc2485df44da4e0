"""The synthetic workload generators: determinism and the statistics they promise."""
import math

import torch

from paper_2608_14205_b200 import inputs as I


def test_layers_are_deterministic_and_distinct():
    wl = I.WORKLOADS["tiny"]
    a = I.make_layer(wl, 0, 0)
    b = I.make_layer(wl, 0, 0)
    c = I.make_layer(wl, 1, 0)
    assert torch.equal(a.h_prev, b.h_prev) and torch.equal(a.H, b.H) and torch.equal(a.W, b.W)
    assert not torch.equal(a.h_prev, c.h_prev) and not torch.equal(a.W, c.W)
    assert a.h_prev.dtype == torch.bfloat16 and a.h_prev.shape == (wl.T, wl.d) and a.W.shape == (wl.E, wl.d)


def test_drift_has_the_requested_relative_norm_and_cosine():
    wl = I.WORKLOADS["qwen3"]
    li = I.make_layer(wl, 0, 0, T=256)
    h, H = li.h_prev.double(), li.H.double()
    ratio = (H - h).norm(dim=1) / h.norm(dim=1)
    assert abs(ratio.mean().item() - wl.rho) < 2e-3
    cos = torch.nn.functional.cosine_similarity(h, H, dim=1).mean().item()
    assert abs(cos - 1 / math.sqrt(1 + wl.rho ** 2)) < 3e-3      # drift is nearly orthogonal at d=2048


def test_cluster_workload_has_bias_and_sequences():
    wl = I.WORKLOADS["dsv3"]
    li = I.make_layer(wl, 0, 0, T=64)
    assert li.select_bias is not None and li.select_bias.shape == (wl.E,)
    assert li.expert_to_slot.tolist() == list(range(wl.E))
    assert I.make_layer(wl, 0, 0, T=0).h_prev.shape == (0, wl.d)


def test_random_counts_and_placement():
    c = I.random_counts(16, 1000, seed=3)
    assert c.sum().item() == 1000 and c.shape == (16,)
    p = I.random_placement(16, seed=3)
    assert sorted(p.tolist()) == list(range(16))
