"""Pins for the oracle's cost model (Eqs. 9, 10), greedy planner (Eqs. 6-8,
Algorithm 1) and dispatch index."""
import itertools
import random
from fractions import Fraction

import numpy as np
import pytest

from oracle import freebalance_oracle as O


def _bud(**kw):
    kw.setdefault("gamma_num", 1)
    kw.setdefault("gamma_den", 8)
    return O.Budget(**kw)


# ---------------------------------------------------------------- Eq. 9 / 10
def test_budget_eq10():
    assert O.budget_ns(500_000, 100_000) == 400_000
    assert O.budget_ns(100, 100) == 0
    assert O.budget_ns(100, 250) == 0


def test_swap_cost_hand_value(golden):
    gd = golden("swap_cost.json")
    b = O.Budget(alpha_ns=(gd["alpha_ns"],) * 2, fs_per_byte=(gd["fs_per_byte"],) * 2,
                 expert_bytes=gd["expert_bytes"])
    c = O.swap_cost_ns(b, 0, 1)
    assert c == gd["cost_ns"]
    assert gd["swaps_that_fit"] * c <= gd["window_ns"] < (gd["swaps_that_fit"] + 1) * c


def test_swap_cost_classes_ceiling_and_floor_of_one():
    b = O.Budget(alpha_ns=(10, 1000), fs_per_byte=(1000, 4000), expert_bytes=500, ranks_per_node=2)
    assert O.swap_cost_ns(b, 0, 1) == 10 + 1          # 1000 B * 1000 fs = 1e6 fs = exactly 1 ns
    assert O.swap_cost_ns(b, 1, 2) == 1000 + 4        # other node: 1000 B * 4000 fs = 4 ns
    b2 = O.Budget(alpha_ns=(0, 0), fs_per_byte=(1, 1), expert_bytes=1)
    assert O.swap_cost_ns(b2, 0, 1) == 1              # ceil(2e-6) = 1
    assert O.swap_cost_ns(O.Budget(), 0, 1) == 1      # never zero
    b3 = O.Budget(alpha_ns=(5, 5), fs_per_byte=(10**6, 10**6), expert_bytes_table=(1, 2, 3, 4))
    assert O.swap_cost_ns(b3, 0, 1, 1, 3) == 5 + 6


def test_link_ids():
    assert O.link_id(3, 1, 0) == ("rank", 1, 3)
    assert O.link_id(3, 1, 4) == ("rank", 1, 3)
    assert O.link_id(5, 1, 4) == ("node", 0, 1)
    assert O.link_id(1, 6, 4) == O.link_id(7, 0, 4)


# ---------------------------------------------------------------- Eq. 8
def test_objective_closed_form_points():
    assert O.objective([4, 4, 4], Fraction(3)) == 4
    assert O.objective([6, 2], Fraction(1, 2)) == 6 + Fraction(1, 2) * (4 + 4)
    assert O.objective([5, 1, 0], Fraction(0)) == 5


def test_rank_loads_bruteforce():
    rng = random.Random(3)
    E, R = 12, 4
    counts = [rng.randrange(50) for _ in range(E)]
    pi = list(range(E))
    rng.shuffle(pi)
    L = O.rank_loads(counts, pi, R)
    for r in range(R):
        assert L[r] == sum(counts[e] for e in range(E) if pi[e] in range(r * 3, r * 3 + 3))
    assert sum(L) == sum(counts)


# ---------------------------------------------------------------- worked plans
@pytest.mark.parametrize("name", ["planner_two_swaps_one_tie.json", "planner_tie_then_stop.json"])
def test_planner_worked_examples(golden, name):
    gd = golden(name)
    b = O.Budget(max_swaps=gd["max_swaps"], gamma_num=gd["gamma_num"], gamma_den=gd["gamma_den"],
                 tau_tokens=gd["tau_tokens"])
    swaps, pi, before, after = O.plan_swaps(gd["counts"], gd["expert_to_slot"], gd["R"], b)
    assert [list(s) for s in swaps] == gd["swaps"]
    assert pi == gd["expert_to_slot_out"]
    assert before == gd["load_before"] and after == gd["load_after"]


# ---------------------------------------------------------------- independent replay
def _replay_check(counts, pi0, R, bud, swaps, pi_out, before, after, layer_id=0):
    """Re-derive every accepted swap by exhaustive enumeration with integer
    arithmetic only (the sum of squares of the loads replaces the variance: the
    mean is swap-invariant), and check the paper's invariants on the way."""
    E = len(counts)
    m = E // R
    pi = list(pi0)
    L = [0] * R
    for e in range(E):
        L[pi[e] // m] += counts[e]
    assert L == before
    moved = set()
    spent_rank = [0] * R
    spent_link = {}
    spent = 0
    gn, gd = bud.gamma_num, (bud.gamma_den or 1)
    if not bud.gamma_den:
        gn = 0
    for it in range(len(swaps) + 1):
        hi = max(L)
        a = L.index(hi)
        lo = min(L)
        b = L.index(lo)
        cands = []
        if it < bud.max_swaps and hi - lo > bud.tau_tokens:
            for ea in range(E):
                for eb in range(E):
                    if pi[ea] // m != a or pi[eb] // m != b or ea in moved or eb in moved:
                        continue
                    Ln = list(L)
                    Ln[a] += counts[eb] - counts[ea]
                    Ln[b] += counts[ea] - counts[eb]
                    # gd * (Phi - Phi') with the mean cancelled
                    ben = gd * (max(L) - max(Ln)) + gn * (sum(x * x for x in L) - sum(x * x for x in Ln))
                    if ben <= 0:
                        continue
                    c = O.swap_cost_ns(bud, a, b, ea, eb)
                    lk = O.link_id(a, b, bud.ranks_per_node)
                    if bud.global_ns != O.U64_OFF and spent + c > bud.global_ns:
                        continue
                    if bud.rank_ns != O.U64_OFF and max(spent_rank[a], spent_rank[b]) + c > bud.rank_ns:
                        continue
                    if bud.link_ns != O.U64_OFF and spent_link.get(lk, 0) + c > bud.link_ns:
                        continue
                    cands.append((Fraction(-ben, c), (layer_id, a, b, ea, eb), c, Ln))
        if it == len(swaps):
            assert not cands, "planner stopped although a feasible beneficial swap remained"
            break
        assert cands, "planner accepted a swap where none was feasible"
        cands.sort(key=lambda t: (t[0], t[1]))
        _, (_, a2, b2, ea, eb), c, Ln = cands[0]
        assert swaps[it] == (a2, b2, ea, eb)
        assert max(Ln) <= max(L)                       # never raises the maximum rank load
        L = Ln
        pi[ea], pi[eb] = pi[eb], pi[ea]
        moved |= {ea, eb}
        spent += c
        spent_rank[a2] += c
        spent_rank[b2] += c
        lk = O.link_id(a2, b2, bud.ranks_per_node)
        spent_link[lk] = spent_link.get(lk, 0) + c
    assert pi == pi_out and L == after
    assert sorted(pi_out) == list(range(E))             # still a bijection onto the slots
    assert len(swaps) <= bud.max_swaps
    assert len(moved) == 2 * len(swaps)                 # every expert moves at most once
    assert sum(after) == sum(before)


@pytest.mark.parametrize("seed", range(40))
def test_planner_matches_exhaustive_replay(seed):
    rng = random.Random(seed)
    R = rng.choice([2, 3, 4, 8])
    m = rng.choice([1, 2, 3, 4])
    E = R * m
    counts = [rng.randrange(0, 60) ** rng.choice([1, 2]) for _ in range(E)]
    pi = list(range(E))
    if seed % 2:
        rng.shuffle(pi)
    kw = dict(max_swaps=rng.choice([0, 1, 2, 5, E]), gamma_num=rng.choice([0, 1, 3]),
              gamma_den=rng.choice([1, 8, 1000]), tau_tokens=rng.choice([0, 0, 10, 500]))
    if seed % 3 == 0:
        kw.update(alpha_ns=(100, 700), fs_per_byte=(2000, 9000), expert_bytes=rng.randrange(1, 10**6),
                  ranks_per_node=rng.choice([0, 2]), global_ns=rng.choice([O.U64_OFF, 10**4, 10**5]),
                  rank_ns=rng.choice([O.U64_OFF, 5000, 10**5]), link_ns=rng.choice([O.U64_OFF, 3000, 10**5]))
    if seed % 5 == 0:
        kw.update(alpha_ns=(50, 50), fs_per_byte=(10**6, 10**6),
                  expert_bytes_table=tuple(rng.randrange(1, 500) for _ in range(E)))
    bud = O.Budget(**kw)
    swaps, pi_out, before, after = O.plan_swaps(counts, pi, R, bud, layer_id=seed)
    _replay_check(counts, pi, R, bud, swaps, pi_out, before, after, layer_id=seed)
    again = O.plan_swaps(counts, pi, R, bud, layer_id=seed)
    assert again == (swaps, pi_out, before, after)       # deterministic


# ---------------------------------------------------------------- planner variants
def _random_plan_case(seed):
    rng = random.Random(1000 + seed)
    R = rng.choice([2, 3, 4, 6, 8])
    m = rng.choice([1, 2, 3, 4])
    E = R * m
    counts = [rng.randrange(0, 60) ** rng.choice([1, 2]) for _ in range(E)]
    pi = list(range(E))
    if seed % 2:
        rng.shuffle(pi)
    kw = dict(max_swaps=rng.choice([1, 2, 5, E]), gamma_num=rng.choice([0, 1, 3]),
              gamma_den=rng.choice([1, 8, 1000]), tau_tokens=rng.choice([0, 0, 10, 500]))
    if seed % 3 == 0:
        kw.update(alpha_ns=(100, 700), fs_per_byte=(2000, 9000), expert_bytes=rng.randrange(1, 10**6),
                  ranks_per_node=rng.choice([0, 2]), global_ns=rng.choice([O.U64_OFF, 10**4, 10**5]),
                  rank_ns=rng.choice([O.U64_OFF, 5000, 10**5]), link_ns=rng.choice([O.U64_OFF, 3000, 10**5]))
    if seed % 5 == 0:
        kw.update(alpha_ns=(50, 50), fs_per_byte=(10**6, 10**6),
                  expert_bytes_table=tuple(rng.randrange(1, 500) for _ in range(E)))
    return counts, pi, R, kw


def _int_benefit(L, Ln, gn, gd):
    """gd * (Phi(L) - Phi(Ln)) in integers: the mean is swap-invariant, so the variance term is
    a difference of sums of squares."""
    return gd * (max(L) - max(Ln)) + gn * (sum(x * x for x in L) - sum(x * x for x in Ln))


def test_sweep_worked_example(golden):
    gd = golden("planner_sweep_overshoots.json")
    b = O.Budget(max_swaps=gd["max_swaps"], gamma_num=gd["gamma_num"], gamma_den=gd["gamma_den"],
                 tau_tokens=gd["tau_tokens"], mode=O.PLAN_SWEEP)
    swaps, pi, before, after = O.plan(gd["counts"], gd["expert_to_slot"], gd["R"], b)
    assert [list(s) for s in swaps] == gd["swaps"]
    assert pi == gd["expert_to_slot_out"] and before == gd["load_before"] and after == gd["load_after"]
    assert max(after) >= max(before)          # the recorded weakness of the one-pass reading


@pytest.mark.parametrize("seed", range(30))
def test_sweep_matches_independent_sort_and_sweep(seed):
    counts, pi0, R, kw = _random_plan_case(seed)
    bud = O.Budget(mode=O.PLAN_SWEEP, **kw)
    swaps, pi_out, before, after = O.plan(counts, pi0, R, bud, layer_id=seed)
    # independent restatement: integers only, Python's sort on exact keys
    E, m = len(counts), len(counts) // R
    L = [sum(counts[e] for e in range(E) if pi0[e] // m == r) for r in range(R)]
    assert L == before
    gn, gd = (bud.gamma_num, bud.gamma_den) if bud.gamma_den else (0, 1)
    a, b = L.index(max(L)), L.index(min(L))
    expect, pi, sel, spent = [], list(pi0), set(), 0
    if L[a] - L[b] > bud.tau_tokens:
        cands = []
        for ea in range(E):
            for eb in range(E):
                if pi0[ea] // m != a or pi0[eb] // m != b:
                    continue
                Ln = list(L)
                Ln[a] += counts[eb] - counts[ea]
                Ln[b] += counts[ea] - counts[eb]
                ben = _int_benefit(L, Ln, gn, gd)
                if ben > 0:
                    c = O.swap_cost_ns(bud, a, b, ea, eb)
                    cands.append((Fraction(-ben, c), ea, eb, c))
        Lc = list(L)
        for _, ea, eb, c in sorted(cands):
            if len(expect) == bud.max_swaps:
                break
            if ea in sel or eb in sel:
                continue
            # one source, one destination and one link throughout: all three residuals see `spent`
            if any(lim != O.U64_OFF and spent + c > lim for lim in (bud.global_ns, bud.rank_ns, bud.link_ns)):
                continue
            expect.append((a, b, ea, eb))
            sel |= {ea, eb}
            spent += c
            Lc[a] += counts[eb] - counts[ea]
            Lc[b] += counts[ea] - counts[eb]
            pi[ea], pi[eb] = pi[eb], pi[ea]
        L = Lc
    assert swaps == expect and pi_out == pi and after == L
    assert sorted(pi_out) == list(range(E)) and sum(after) == sum(before) and len(swaps) <= bud.max_swaps
    # with room for one swap only, the sweep and Algorithm 1's loop take the same pair
    one = dict(kw, max_swaps=1)
    assert O.plan(counts, pi0, R, O.Budget(mode=O.PLAN_SWEEP, **one), seed) == \
        O.plan_swaps(counts, pi0, R, O.Budget(**one), seed)


def test_wide_frontier_worked_example(golden):
    gd = golden("planner_wide_frontier.json")
    kw = dict(max_swaps=gd["max_swaps"], gamma_num=gd["gamma_num"], gamma_den=gd["gamma_den"],
              tau_tokens=gd["tau_tokens"])
    swaps, pi, before, after = O.plan(gd["counts"], gd["expert_to_slot"], gd["R"],
                                      O.Budget(mode=O.PLAN_WIDE, frontier_width=gd["frontier_width"], **kw))
    assert [list(s) for s in swaps] == gd["swaps"]
    assert pi == gd["expert_to_slot_out"] and before == gd["load_before"] and after == gd["load_after"]
    narrow = O.plan_swaps(gd["counts"], gd["expert_to_slot"], gd["R"], O.Budget(**kw))
    assert [list(s) for s in narrow[0]] == gd["narrow_frontier_swaps"]


@pytest.mark.parametrize("seed", range(30))
def test_wide_frontier_matches_exhaustive_replay(seed):
    counts, pi0, R, kw = _random_plan_case(seed)
    W = 1 + seed % 3
    bud = O.Budget(mode=O.PLAN_WIDE, frontier_width=W, **kw)
    swaps, pi_out, before, after = O.plan(counts, pi0, R, bud, layer_id=seed)
    if W == 1:
        assert (swaps, pi_out, before, after) == O.plan_swaps(counts, pi0, R, O.Budget(**kw), seed)
    E, m = len(counts), len(counts) // R
    gn, gd = (bud.gamma_num, bud.gamma_den) if bud.gamma_den else (0, 1)
    pi, L = list(pi0), list(before)
    moved, spent, spent_rank, spent_link = set(), 0, [0] * R, {}
    for it in range(len(swaps) + 1):
        order = sorted(range(R), key=lambda r: (-L[r], r))
        top = order[:min(W, R)]
        bottom = sorted(range(R), key=lambda r: (L[r], r))[:min(W, R)]
        cands = []
        if it < bud.max_swaps and max(L) - min(L) > bud.tau_tokens:
            for a in top:
                for b in bottom:
                    if a == b or L[a] <= L[b]:
                        continue
                    for ea in range(E):
                        for eb in range(E):
                            if pi[ea] // m != a or pi[eb] // m != b or ea in moved or eb in moved:
                                continue
                            Ln = list(L)
                            Ln[a] += counts[eb] - counts[ea]
                            Ln[b] += counts[ea] - counts[eb]
                            ben = _int_benefit(L, Ln, gn, gd)
                            if ben <= 0:
                                continue
                            c = O.swap_cost_ns(bud, a, b, ea, eb)
                            lk = O.link_id(a, b, bud.ranks_per_node)
                            if bud.global_ns != O.U64_OFF and spent + c > bud.global_ns:
                                continue
                            if bud.rank_ns != O.U64_OFF and max(spent_rank[a], spent_rank[b]) + c > bud.rank_ns:
                                continue
                            if bud.link_ns != O.U64_OFF and spent_link.get(lk, 0) + c > bud.link_ns:
                                continue
                            cands.append((Fraction(-ben, c), (seed, a, b, ea, eb), c, Ln))
        if it == len(swaps):
            assert not cands
            break
        assert cands
        _, (_, a, b, ea, eb), c, Ln = min(cands, key=lambda t: (t[0], t[1]))
        assert swaps[it] == (a, b, ea, eb)
        L = Ln
        pi[ea], pi[eb] = pi[eb], pi[ea]
        moved |= {ea, eb}
        spent += c
        spent_rank[a] += c
        spent_rank[b] += c
        lk = O.link_id(a, b, bud.ranks_per_node)
        spent_link[lk] = spent_link.get(lk, 0) + c
    assert pi == pi_out and L == after and sorted(pi_out) == list(range(E))


def test_ratio_prefers_cheap_swap_over_larger_benefit():
    # experts 0,1 on rank 0, experts 2,3 on rank 1; per-expert sizes make the
    # largest-benefit pair expensive enough to lose on benefit / cost
    counts = [20, 12, 2, 0]
    sizes = (1000, 10, 1000, 10)
    bud = O.Budget(max_swaps=1, gamma_num=0, gamma_den=1, alpha_ns=(0, 0), fs_per_byte=(10**6, 10**6),
                   expert_bytes_table=sizes)
    # loads [32, 2]; (0,3): moves 20 -> max 22, benefit 10, cost 1010; (1,3): moves 12 -> max 20,
    # benefit 12, cost 20; (0,2): moves 18 -> max 20, benefit 12, cost 2000; (1,2): moves 10 -> 22, cost 1010
    swaps, _, _, after = O.plan_swaps(counts, [0, 1, 2, 3], 2, bud)
    assert swaps == [(0, 1, 1, 3)] and after == [20, 14]


# ---------------------------------------------------------------- degenerate plans
def test_zero_budget_keeps_placement():
    counts = [9, 1, 1, 1]
    pi = [3, 0, 1, 2]
    for bud in (_bud(max_swaps=0), _bud(max_swaps=4, global_ns=0), _bud(max_swaps=4, rank_ns=0),
                _bud(max_swaps=4, link_ns=0), _bud(max_swaps=4, tau_tokens=10**6)):
        swaps, pi_out, before, after = O.plan_swaps(counts, pi, 2, bud)
        assert swaps == [] and pi_out == pi and before == after


def test_uniform_counts_and_one_expert_per_rank_give_empty_plans():
    assert O.plan_swaps([5] * 8, list(range(8)), 4, _bud(max_swaps=4))[0] == []
    # one expert per rank: a swap only permutes the rank loads, Phi cannot drop
    assert O.plan_swaps([50, 3, 9, 1], list(range(4)), 4, _bud(max_swaps=4))[0] == []


def test_time_budget_admits_exactly_five_swaps():
    rng = random.Random(7)
    E, R = 256, 32
    counts = [int(4000 / (1 + rng.randrange(E)) ** 1.1) + rng.randrange(30) for _ in range(E)]
    bud = O.Budget(max_swaps=128, global_ns=500_000, rank_ns=500_000, link_ns=500_000, gamma_num=1,
                   gamma_den=2 * 4096, alpha_ns=(2000, 2000), fs_per_byte=(1111, 1111),
                   expert_bytes=44_040_192)
    swaps, pi_out, before, after = O.plan_swaps(counts, list(range(E)), R, bud)
    assert len(swaps) == 5
    assert max(after) < max(before)
    _replay_check(counts, list(range(E)), R, bud, swaps, pi_out, before, after)


def test_rank_budget_blocks_a_busy_rank():
    # loads [90,3,6]: rank 0 is the heaviest twice in a row (swaps with rank 1, then rank 2),
    # then ranks 2 and 1 level out.  A per-rank window that fits one 10 ns swap stops the
    # second swap of rank 0 and with it the loop; a window of two swaps lets all three through.
    counts = [30, 30, 30, 1, 1, 1, 2, 2, 2]
    one = _bud(max_swaps=3, rank_ns=15, alpha_ns=(10, 10))
    assert O.plan_swaps(counts, list(range(9)), 3, one)[0] == [(0, 1, 0, 3)]
    two = _bud(max_swaps=3, rank_ns=25, alpha_ns=(10, 10))
    swaps, _, _, after = O.plan_swaps(counts, list(range(9)), 3, two)
    assert swaps == [(0, 1, 0, 3), (0, 2, 1, 6), (2, 1, 7, 4)] and after == [33, 33, 33]


# ---------------------------------------------------------------- dispatch
def test_dispatch_worked_example(golden):
    gd = golden("dispatch_small.json")
    so, ro, perm, inv, rl = O.dispatch_index(np.array(gd["ids"]), gd["expert_to_slot"], gd["R"])
    assert so.tolist() == gd["slot_offsets"] and ro.tolist() == gd["rank_offsets"]
    assert perm.tolist() == gd["perm"] and inv.tolist() == gd["inv_perm"] and rl.tolist() == gd["rank_load"]


@pytest.mark.parametrize("seed", range(6))
def test_dispatch_matches_lexsort_and_invariants(seed):
    rng = np.random.default_rng(seed)
    T, E, k, R = 37, 12, 3, 4
    ids = np.stack([rng.choice(E, size=k, replace=False) for _ in range(T)])
    pi = rng.permutation(E)
    so, ro, perm, inv, rl = O.dispatch_index(ids, pi, R)
    slot = pi[ids.reshape(-1)]
    tok = np.repeat(np.arange(T), k)
    want = np.lexsort((tok, slot))                       # library routine: by slot, then token
    assert perm.tolist() == want.tolist()
    assert sorted(perm.tolist()) == list(range(T * k))
    assert inv[perm].tolist() == list(range(T * k))
    assert so[0] == 0 and so[-1] == T * k and (np.diff(so) >= 0).all()
    assert np.diff(so).tolist() == np.bincount(slot, minlength=E).tolist()
    m = E // R
    assert ro.tolist() == [so[r * m] for r in range(R)] + [T * k]
    assert rl.tolist() == np.diff(ro).tolist()
    for p in range(E):                                   # tokens ascending inside a slot
        seg = perm[so[p]:so[p + 1]] // k
        assert (np.diff(seg) > 0).all()
    counts = O.expert_histogram(ids, E)
    assert rl.tolist() == O.rank_loads(counts, pi, R)


@pytest.mark.parametrize("seed", range(8))
def test_sharded_dispatch_equals_the_whole_batch_cut_into_shards(seed):
    rng = random.Random(70 + seed)
    R = rng.choice([2, 4])
    E = R * rng.choice([1, 2, 4])
    k = rng.choice([1, 2, min(3, E)])
    world = rng.choice([1, 2, 3, 5])
    T = rng.choice([0, 1, 7, 40])
    ids = np.array([rng.sample(range(E), k) for _ in range(T)], dtype=np.int64).reshape(T, k)
    pi = list(range(E))
    rng.shuffle(pi)
    so, ro, perm, inv, rl = O.dispatch_index(ids, pi, R)
    cuts = sorted(rng.randrange(0, T + 1) for _ in range(world - 1))
    bounds = [0] + cuts + [T]                                     # uneven, possibly empty shards
    local = [O.dispatch_index(ids[bounds[r]:bounds[r + 1]], pi, R) for r in range(world)]
    counts_all = [np.diff(loc[0]).tolist() for loc in local]
    for r in range(world):
        g_so, g_ro, g_rl, g_inv = O.globalize_dispatch(counts_all, r, local[r][0], local[r][3], R)
        assert g_so.tolist() == so.tolist() and g_ro.tolist() == ro.tolist() and g_rl.tolist() == rl.tolist()
        assert g_inv.tolist() == inv[bounds[r] * k:bounds[r + 1] * k].tolist()


def test_dispatch_empty():
    so, ro, perm, inv, rl = O.dispatch_index(np.zeros((0, 2), dtype=np.int32), [0, 1, 2, 3], 2)
    assert so.tolist() == [0] * 5 and ro.tolist() == [0] * 3 and perm.size == 0 and rl.tolist() == [0, 0]


# ---------------------------------------------------------------- metrics
def test_metrics():
    assert O.max_over_mean([4, 4, 4, 4]) == 1.0
    assert O.max_over_mean([6, 2]) == 1.5
    a = np.array([[0, 1], [2, 3]])
    b = np.array([[1, 0], [2, 4]])
    assert O.topk_hit_rate(a, b) == 0.75
