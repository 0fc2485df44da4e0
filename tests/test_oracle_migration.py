"""Pins for the oracle's weight exchange (stage 3 on one device)."""
import numpy as np
import pytest

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import inputs as I


def _weights(E, S, seed=0):
    return np.random.default_rng(seed).integers(0, 256, size=(E, S), dtype=np.uint8)


def test_hand_worked_exchange():
    # 4 experts, expert e in slot e; slot p holds bytes (10 p, 10 p + 1).  Swap experts 0 and 3.
    w = np.array([[0, 1], [10, 11], [20, 21], [30, 31]], dtype=np.uint8)
    new, pi = O.apply_swaps(w, [0, 1, 2, 3], [(0, 1, 0, 3)])
    assert new.tolist() == [[30, 31], [10, 11], [20, 21], [0, 1]]
    assert pi == [3, 1, 2, 0]
    assert w.tolist() == [[0, 1], [10, 11], [20, 21], [30, 31]], "the input is not modified"


@pytest.mark.parametrize("seed", range(6))
def test_every_expert_ends_where_the_new_placement_says(seed):
    rng = np.random.default_rng(seed)
    E, R, S = 16, 4, 24
    pi0 = I.random_placement(E, seed).tolist()
    counts = I.random_counts(E, 4000, seed, zipf_s=1.2).tolist()
    bud = O.Budget(max_swaps=int(rng.integers(0, 8)), global_ns=2**64 - 1, rank_ns=2**64 - 1, link_ns=2**64 - 1,
                   tau_tokens=0, gamma_num=1, gamma_den=50, alpha_ns=(0, 0), fs_per_byte=(0, 0),
                   ranks_per_node=0, expert_bytes=0)
    swaps, pi_new, _, _ = O.plan_swaps(counts, pi0, R, bud)
    w = _weights(E, S, seed)
    new, pi_after = O.apply_swaps(w, pi0, swaps)
    assert pi_after == pi_new, "the exchange implies the planner's own new placement"
    for e in range(E):                                   # the definition of a correct migration
        assert np.array_equal(new[pi_new[e]], w[pi0[e]])
    assert sorted(map(bytes, new)) == sorted(map(bytes, w)), "slot images are permuted, nothing else"
    back, pi_back = O.apply_swaps(new, pi_after, swaps)
    assert np.array_equal(back, w) and pi_back == pi0, "the same exchanges again restore everything"


def test_empty_plan_is_the_identity():
    w = _weights(8, 16)
    new, pi = O.apply_swaps(w, list(range(8)), [])
    assert np.array_equal(new, w) and pi == list(range(8))
