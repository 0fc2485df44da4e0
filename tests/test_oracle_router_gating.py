"""Pins for the oracle's router (Eq. 4), gating / top-k rule and histogram (Eq. 5)."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import freebalance_oracle as O


def _bf16_bits(x):
    """Round-to-nearest-even float32 -> bf16 bit patterns (test helper)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def _bits_to_fraction(b):
    b = int(b)
    sign = -1 if b >> 15 else 1
    exp = (b >> 7) & 0xFF
    man = b & 0x7F
    if exp == 0:
        return sign * Fraction(man, 128) * Fraction(2) ** (-126)
    return sign * (1 + Fraction(man, 128)) * Fraction(2) ** (exp - 127)


def test_bf16_widening_known_patterns():
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x3E00, 0x4049], dtype=np.uint16)
    got = O.bf16_bits_to_f64(bits)
    assert got.tolist() == [1.0, -2.0, 0.0, 0.125, 3.140625]


def test_logits_equal_exact_rational_dot_products():
    rng = np.random.default_rng(1)
    T, d, E = 3, 7, 5
    xb = _bf16_bits(rng.standard_normal((T, d)))
    wb = _bf16_bits(rng.standard_normal((E, d)) * 0.02)
    bias = rng.standard_normal(E)
    z = O.router_logits(xb, wb, bias)
    assert z.shape == (T, E)
    for i in range(T):
        for e in range(E):
            exact = sum(_bits_to_fraction(xb[i, j]) * _bits_to_fraction(wb[e, j]) for j in range(d))
            exact += Fraction(float(bias[e]))
            assert abs(Fraction(float(z[i, e])) - exact) < Fraction(1, 10**12)


def test_logits_integer_inputs_are_exact_and_not_transposed():
    # small integers are exact in bf16; the product is then an exact integer matrix
    X = np.array([[1, 2, 3], [0, -1, 4]], dtype=np.float32)          # T=2, d=3
    W = np.array([[1, 0, 0], [0, 1, 0], [1, 1, 1], [2, -2, 1]], dtype=np.float32)  # E=4
    z = O.router_logits(_bf16_bits(X), _bf16_bits(W))
    assert z.tolist() == [[1, 2, 6, 1], [0, -1, 3, 6]]


def test_logits_without_bias_is_plain_product():
    rng = np.random.default_rng(2)
    xb = _bf16_bits(rng.standard_normal((4, 8)))
    wb = _bf16_bits(rng.standard_normal((3, 8)))
    z0 = O.router_logits(xb, wb)
    z1 = O.router_logits(xb, wb, np.array([1.0, -2.0, 0.5]))
    assert np.allclose(z1 - z0, [[1.0, -2.0, 0.5]] * 4, atol=1e-12)


@pytest.mark.parametrize("E,k", [(5, 2), (6, 3), (4, 4), (7, 1)])
def test_softmax_topk_is_the_max_probability_subset(E, k):
    rng = np.random.default_rng(E * 10 + k)
    z = rng.standard_normal((20, E))
    g = O.Gate(E=E, k=k)
    ids, w = O.select_topk(z, g)
    for i in range(z.shape[0]):
        p = [math.exp(v) for v in z[i]]
        s = sum(p)
        p = [v / s for v in p]
        best = max(itertools.combinations(range(E), k), key=lambda c: sum(p[e] for e in c))
        assert set(ids[i].tolist()) == set(best)
        # descending by key inside the chosen set
        assert all(z[i, ids[i, j]] >= z[i, ids[i, j + 1]] for j in range(k - 1))
        # renormalised weights = softmax restricted to the chosen experts
        zs = [math.exp(z[i, e]) for e in ids[i]]
        for j in range(k):
            assert abs(w[i, j] - zs[j] / sum(zs)) < 1e-12
        assert abs(w[i].sum() - 1.0) < 1e-12


def test_softmax_weights_without_renorm_are_full_softmax():
    z = np.array([[0.0, math.log(2.0), math.log(5.0)]])
    ids, w = O.select_topk(z, O.Gate(E=3, k=2, renorm=0))
    assert ids.tolist() == [[2, 1]]
    assert np.allclose(w, [[5 / 8, 2 / 8]])


def test_exact_ties_pick_lowest_ids():
    z = np.zeros((4, 8))
    ids, _ = O.select_topk(z, O.Gate(E=8, k=3))
    assert ids.tolist() == [[0, 1, 2]] * 4
    counts = O.expert_histogram(ids, 8)
    assert counts.tolist() == [4, 4, 4, 0, 0, 0, 0, 0]
    gs = O.Gate(E=8, k=2, gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=4, topk_group=2)
    ids, w = O.select_topk(z, gs)
    assert ids.tolist() == [[0, 1]] * 4            # groups 0,1 kept; experts 0,1 first
    assert np.allclose(w, 0.5)


def test_group_limited_worked_example(golden):
    gd = golden("group_limited_topk.json")
    q = np.array([gd["keys"]])
    # choose logits so that sigmoid(z) equals the keys (bias zero); key 0.0 -> very negative logit
    with np.errstate(divide="ignore"):
        z = np.log(q) - np.log1p(-q)
    z[np.isneginf(z)] = -700.0
    g = O.Gate(E=gd["E"], k=gd["k"], gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=gd["n_group"],
               topk_group=gd["topk_group"])
    qq, elig, score = O.selection_keys(z, g)
    assert np.allclose(qq, q, atol=1e-12)
    assert np.allclose(score[0], gd["group_score"], atol=1e-12)
    ids, w = O.select_topk(z, g)
    assert ids[0].tolist() == gd["ids"]
    assert np.allclose(w[0], [0.9 / 1.5, 0.6 / 1.5])


def _group_topk_bruteforce(q_row, n_group, topk_group, k):
    E = len(q_row)
    gs = E // n_group
    scores = []
    for g in range(n_group):
        vals = sorted(q_row[g * gs:(g + 1) * gs], reverse=True)
        scores.append(sum(vals[:min(2, gs)]))
    groups = sorted(range(n_group), key=lambda g: (-scores[g], g))[:topk_group]
    cand = [e for e in range(E) if e // gs in groups]
    return sorted(cand, key=lambda e: (-q_row[e], e))[:k]


@pytest.mark.parametrize("E,G,KG,k", [(16, 4, 2, 3), (32, 8, 4, 8), (12, 12, 5, 4), (8, 2, 1, 4)])
def test_group_limited_topk_matches_loop_implementation(E, G, KG, k):
    rng = np.random.default_rng(E + G + k)
    z = rng.standard_normal((25, E)) * 2
    bias = rng.standard_normal(E) * 0.3
    g = O.Gate(E=E, k=k, gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=G, topk_group=KG, route_scale=2.5)
    ids, w = O.select_topk(z, g, bias)
    for i in range(z.shape[0]):
        s = [1 / (1 + math.exp(-v)) for v in z[i]]
        q = [s[e] + bias[e] for e in range(E)]
        want = _group_topk_bruteforce(q, G, KG, k)
        assert ids[i].tolist() == want
        tot = sum(s[e] for e in want)
        for j, e in enumerate(want):                      # weights use the unbiased score
            assert abs(w[i, j] - 2.5 * s[e] / tot) < 1e-12


def test_selection_bias_changes_the_selected_set_but_not_the_weights_formula():
    z = np.array([[2.0, 1.0, 0.0, -1.0]])
    g = O.Gate(E=4, k=1, gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=1, topk_group=1, renorm=0)
    ids0, w0 = O.select_topk(z, g, np.zeros(4))
    ids1, w1 = O.select_topk(z, g, np.array([0.0, 0.0, 0.0, 5.0]))
    assert ids0.tolist() == [[0]] and ids1.tolist() == [[3]]
    assert abs(w1[0, 0] - 1 / (1 + math.e)) < 1e-12       # sigmoid(-1), bias not included


def test_sigmoid_closed_form_points():
    z = np.array([[0.0, math.log(3.0)]])
    q, _, _ = O.selection_keys(z, O.Gate(E=2, k=1, gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=1, topk_group=1))
    assert np.allclose(q, [[0.5, 0.75]])


def test_histogram_bruteforce_and_sum():
    rng = np.random.default_rng(5)
    T, E, k = 40, 9, 3
    ids = np.stack([rng.choice(E, size=k, replace=False) for _ in range(T)])
    counts = O.expert_histogram(ids, E)
    for e in range(E):
        assert counts[e] == sum(1 for i in range(T) if e in set(ids[i].tolist()))
    assert counts.sum() == T * k


def test_near_tie_margins():
    z = np.array([[3.0, 2.0, 1.9995, 0.0], [5.0, 4.0, 1.0, 0.0]])
    key_gap, group_gap = O.near_tie_margins(z, O.Gate(E=4, k=2))
    assert abs(key_gap[0] - 0.0005) < 1e-12 and abs(key_gap[1] - 3.0) < 1e-12
    assert np.isinf(group_gap).all()
    key_gap, _ = O.near_tie_margins(z, O.Gate(E=4, k=4))
    assert np.isinf(key_gap).all()


def test_near_tie_margins_group_gap_hand_worked():
    """The group-score gap decides which tokens a parity check may exempt, so it is pinned to
    hand-worked numbers: zero logits make every sigmoid exactly 0.5 and the key 0.5 + bias."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "near_tie_group_gap.json")) as f:
        g = json.load(f)
    keys = np.array(g["keys"], dtype=np.float64)
    gate = O.Gate(E=g["E"], k=g["k"], gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=g["n_group"],
                  topk_group=g["topk_group"])
    all_kept = O.Gate(E=g["E"], k=g["k"], gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=g["n_group"],
                      topk_group=g["n_group"])
    for r in range(keys.shape[0]):               # one token at a time: its keys as the per-expert bias
        z1 = np.zeros((1, g["E"]))
        key_gap, group_gap = O.near_tie_margins(z1, gate, keys[r] - 0.5)
        assert abs(key_gap[0] - g["key_gap"][r]) < 1e-12
        assert abs(group_gap[0] - g["group_gap"][r]) < 1e-12
        # every group kept: no dropped group, every expert eligible
        key_gap3, group_gap3 = O.near_tie_margins(z1, all_kept, keys[r] - 0.5)
        assert np.isinf(group_gap3).all()
        assert abs(key_gap3[0] - g["key_gap_all_groups_kept"][r]) < 1e-12
    # both tokens in one call, the keys reached through the logits (sigmoid of the logit of a
    # key returns it to rounding error); then with the rows swapped: the gaps travel with
    # their rows, which catches a sort along the wrong axis
    z = np.log(keys.clip(1e-300) / (1.0 - keys))
    z[keys == 0.0] = -800.0                      # sigmoid(-800) == 0 in float64
    key_gap, group_gap = O.near_tie_margins(z, gate)
    assert np.allclose(key_gap, g["key_gap"], atol=1e-9) and np.allclose(group_gap, g["group_gap"], atol=1e-9)
    key_gap2, group_gap2 = O.near_tie_margins(z[::-1], gate)
    assert np.allclose(key_gap2, g["key_gap"][::-1], atol=1e-9)
    assert np.allclose(group_gap2, g["group_gap"][::-1], atol=1e-9)


def test_near_tie_margins_bound_actual_flips():
    """Property: perturbing every logit by less than half the smaller margin (scaled to key
    units) never changes a token's expert set; a token whose set changes under a perturbation
    has a margin below twice that perturbation."""
    rng = np.random.default_rng(11)
    T, E = 400, 16
    gate = O.Gate(E=E, k=4, gate=O.GATE_SIGMOID_GROUP_TOPK, n_group=4, topk_group=2)
    z = rng.standard_normal((T, E))
    bias = 0.02 * rng.standard_normal(E)
    ids, _ = O.select_topk(z, gate, bias)
    key_gap, group_gap = O.near_tie_margins(z, gate, bias)
    eps = 2e-2                                   # logit perturbation; keys move by at most eps / 4
    ids2, _ = O.select_topk(z + rng.uniform(-eps, eps, size=z.shape), gate, bias)
    changed = (np.sort(ids, axis=1) != np.sort(ids2, axis=1)).any(axis=1)
    assert changed.any()                         # the perturbation is large enough to matter
    dk = eps / 4                                 # |d sigmoid| <= |dz| / 4
    safe = (key_gap > 2 * dk) & (group_gap > 4 * dk)
    assert not (changed & safe).any()
