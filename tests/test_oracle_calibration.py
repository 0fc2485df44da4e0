"""Pins for the cost-model fit (Eq. 9) and the per-attention-type budgets (Eq. 10)."""
import pytest

from oracle import freebalance_oracle as O


def test_fit_recovers_alpha_and_beta_of_eq9():
    # timings generated from Eq. 9 itself with alpha = 2000 ns and 900 GB/s (1/beta = 10^6/900 fs per byte)
    for alpha, gbps in ((2000, 900), (0, 6000), (15000, 50)):
        c = lambda S: alpha + round(2 * S / gbps)               # ns: bytes / (GB/s) = ns
        a, fs = O.fit_cost_model(c(1 << 20), c(64 << 20), 1 << 20, 64 << 20)
        assert abs(a - alpha) <= 1
        assert 0 <= fs - 1e6 / gbps < 1 + 1e-3, "1/beta in whole femtoseconds per byte, rounded up"
    # exact small case: 100 ns + 2 S * 3 ns per byte  ->  alpha 100, 3 000 000 fs per byte
    assert O.fit_cost_model(100 + 6 * 10, 100 + 6 * 50, 10, 50) == (100, 3_000_000)
    # a fitted alpha below zero is clamped
    assert O.fit_cost_model(5, 100, 10, 50)[0] == 0


def test_fit_rejects_timings_that_do_not_grow():
    with pytest.raises(ValueError):
        O.fit_cost_model(100, 100, 10, 50)
    with pytest.raises(ValueError):
        O.fit_cost_model(100, 200, 50, 50)


def test_fitted_model_feeds_the_planner_cost():
    a, fs = O.fit_cost_model(2000 + 2330, 2000 + 97867, 1 << 20, 44_040_192)
    bud = O.Budget(max_swaps=8, global_ns=500_000, rank_ns=500_000, link_ns=500_000, tau_tokens=0, gamma_num=0,
                   gamma_den=1, alpha_ns=(a, a), fs_per_byte=(fs, fs), ranks_per_node=0, expert_bytes=44_040_192)
    cost = O.swap_cost_ns(bud, 0, 1)
    # never below the measured time, above it by less than one femtosecond per byte moved (+ ceilings)
    assert 0 <= cost - (2000 + 97867) <= 2 * 44_040_192 // 1_000_000 + 3


def test_budgets_reuse_the_first_layer_of_each_attention_type():
    # homogeneous model: layer 0's time is reused throughout
    assert O.budgets_by_attention_type(["full"] * 4, {0: 700_000}, 200_000) == [500_000] * 4
    # hybrid model: the first occurrence of each type is the one profiled
    types = ["full", "linear", "linear", "full", "sparse"]
    got = O.budgets_by_attention_type(types, {0: 700_000, 1: 150_000, 4: 90_000}, 100_000)
    assert got == [600_000, 50_000, 50_000, 600_000, 0]          # max(0, .) at the last one
