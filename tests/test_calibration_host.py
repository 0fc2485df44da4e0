"""Host arithmetic of the cost-model calibration and the attention-profile bookkeeping,
against the oracle (no GPU: the library's host functions run anywhere)."""
import numpy as np
import pytest

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B


def test_fit_matches_the_oracle_on_random_timings():
    rng = np.random.default_rng(0)
    for _ in range(300):
        s_small = int(rng.integers(1, 1 << 22)) * 16
        s_large = s_small + int(rng.integers(1, 1 << 24)) * 16
        t_small = int(rng.integers(1, 1 << 24))
        t_large = t_small + int(rng.integers(1, 1 << 28))
        assert B.fb_fit_cost_model(t_small, t_large, s_small, s_large) == O.fit_cost_model(t_small, t_large, s_small, s_large)
    # extreme magnitudes stay exact (128-bit intermediate products)
    big = (2**40, 2**50, 16, 2**44)
    assert B.fb_fit_cost_model(*big) == O.fit_cost_model(*big)


def test_fit_rejects_what_the_oracle_rejects():
    for args in ((100, 100, 16, 32), (100, 200, 32, 32), (200, 100, 16, 32)):
        with pytest.raises(B.FbError):
            B.fb_fit_cost_model(*args)
        with pytest.raises(ValueError):
            O.fit_cost_model(*args)
