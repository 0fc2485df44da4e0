"""CPU oracle for the FreeBalance per-layer hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain restatement of what the paper's method computes,
written from the paper's equations and Algorithm 1.  It exists so the CUDA
library can be checked against something that is not itself.  Nothing in the
product may import it: only the tests, the smoke check and the benchmark's
CPU-baseline leg do.  It shares no code with the CUDA path.

Precision: router logits are accumulated in float64 from the same bf16 bit
patterns the GPU reads.  Everything after top-k is exact integer / rational
arithmetic (``int`` and ``fractions.Fraction``).

Pinning status (the tests that hold each function to something other than
itself live in ``tests/test_oracle_*.py``):

* ``router_logits``      pinned: exact rational dot products on tiny inputs, and
                          integer-valued inputs whose product is exact.
* ``select_topk``        pinned: brute-force subset search, monotonicity of
                          softmax, the all-equal tie case, a hand-worked
                          group-limited example.
* ``expert_histogram``   pinned: brute-force counting, sum = T*k.
* ``rank_loads``         pinned: brute force, sum invariant.
* ``swap_cost_ns``       pinned: hand-computed value for the DeepSeek-V3-shaped
                          budget (99 858 ns) and exact rational ceiling.
* ``plan_swaps``         pinned: two hand-worked plans, exhaustive enumeration of
                          every iteration's choice, the paper's invariants
                          (budget, no max-load increase, permutation, once per
                          expert), degenerate cases with known empty plans.
* ``plan_swaps_sweep``   pinned: a hand-worked plan (the first worked example's counts, where
                          the one pass accepts a second pair that raises the maximum), an
                          independent integer-only sort-and-sweep on random cases, its
                          invariants (budget, bijection, once per expert), and agreement with
                          ``plan_swaps`` whenever at most one swap is allowed.
* ``plan_swaps_wide``    pinned: a hand-worked plan in which only the second most loaded rank
                          offers a beneficial swap, exhaustive integer-only replay over the
                          widened frontier on random cases, equality with ``plan_swaps`` at
                          width 1.
* ``dispatch_index``     pinned: brute-force ``sorted`` on tiny inputs, a
                          hand-worked example, permutation/offset invariants.
* ``globalize_dispatch`` pinned: the whole batch's ``dispatch_index`` cut into the shards' token
                          ranges (positions, offsets and loads must coincide), on random cases
                          with uneven and empty shards.
* ``budget_ns``          pinned: Eq. 10 special cases.
* ``row_cosine_mean``    pinned: closed forms (equal, opposite, orthogonal rows,
                          a 45-degree pair, scale invariance, the zero-row rule).
* ``apply_swaps``        pinned: the placement definition (the slot the new placement
                          names holds the expert's original bytes, for every expert),
                          a hand-worked exchange, identity on the empty plan, twice =
                          identity, agreement with ``plan_swaps``' own new placement.
* ``fit_cost_model``     pinned: exact recovery of alpha and beta from synthetic timings that
                          follow Eq. 9, the rounding directions, rejection of a non-increasing pair.
* ``budgets_by_attention_type`` pinned: hand-worked homogeneous and hybrid layer lists (Eq. 10).
* ``serving_loop``       pinned: placement carry-over checked step by step against
                          ``layer_step`` started from the carried placement, a
                          hand-worked two-step example of the realised-load
                          figures, and the empty-budget case (nothing ever moves).
"""
from __future__ import annotations

import dataclasses
import math
from fractions import Fraction
from typing import List, Optional, Sequence, Tuple

import numpy as np

GATE_SOFTMAX_TOPK = 0
GATE_SIGMOID_GROUP_TOPK = 1
U64_OFF = 2**64 - 1          # a residual budget with this initial value is not enforced
GROUP_SCORE_TOP = 2          # a group's score is the sum of its 2 largest selection keys


# ----------------------------------------------------------------------------
# Eq. 4: the linear router
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float64 exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def router_logits(x_bits: np.ndarray, W_bits: np.ndarray,
                  logit_bias: Optional[np.ndarray] = None) -> np.ndarray:
    """g(X) = X W + 1 b^T (Eq. 4), in float64.

    ``x_bits`` is [T, d] and ``W_bits`` is [E, d] (one row per expert, i.e. the
    paper's W transposed), both bf16 bit patterns.  Used for the early pass on
    h_{l-1} (Eq. 2) and for the normal pass on H_l (Eq. 3) alike.
    """
    X = bf16_bits_to_f64(x_bits)
    W = bf16_bits_to_f64(W_bits)
    z = X @ W.T
    if logit_bias is not None:
        z = z + np.asarray(logit_bias, dtype=np.float64)[None, :]
    return z


# ----------------------------------------------------------------------------
# "the original top-k rule" (text after Eq. 4; the rule itself is the model's)
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Gate:
    E: int
    k: int
    gate: int = GATE_SOFTMAX_TOPK
    n_group: int = 1
    topk_group: int = 1
    renorm: int = 1
    route_scale: float = 1.0


def _topk_desc(key: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries per row, descending; equal keys -> lower index first."""
    order = np.argsort(-key, axis=1, kind="stable")
    return order[:, :k]


def selection_keys(z: np.ndarray, g: Gate, select_bias: Optional[np.ndarray] = None
                   ) -> Tuple[np.ndarray, np.ndarray, Optional[np.ndarray]]:
    """Return (q, eligible, group_score).

    softmax gate: q = z (softmax is strictly increasing in z for a fixed row, so
    the top-k of the probabilities is the top-k of the logits); all experts eligible.
    sigmoid gate: s = 1/(1+exp(-z)); q = s + select_bias; experts form n_group
    contiguous groups; a group's score is the sum of its two largest q; only the
    topk_group best groups (ties -> lower group) stay eligible.
    """
    T, E = z.shape
    if g.gate == GATE_SOFTMAX_TOPK:
        return z, np.ones((T, E), dtype=bool), None
    s = 1.0 / (1.0 + np.exp(-z))
    q = s if select_bias is None else s + np.asarray(select_bias, dtype=np.float64)[None, :]
    gs = E // g.n_group
    qg = q.reshape(T, g.n_group, gs)
    n_top = min(GROUP_SCORE_TOP, gs)
    part = -np.sort(-qg, axis=2)[:, :, :n_top]
    group_score = part.sum(axis=2)
    kept = _topk_desc(group_score, g.topk_group)
    elig_g = np.zeros((T, g.n_group), dtype=bool)
    np.put_along_axis(elig_g, kept, True, axis=1)
    eligible = np.repeat(elig_g, gs, axis=1)
    return q, eligible, group_score


def select_topk(z: np.ndarray, g: Gate, select_bias: Optional[np.ndarray] = None
                ) -> Tuple[np.ndarray, np.ndarray]:
    """Top-k expert ids (descending key, ties -> lower id) and routing weights.

    Weights: softmax gate -> softmax probabilities of the chosen experts,
    renormalised over the k chosen when ``renorm``; sigmoid gate -> the unbiased
    sigmoid scores of the chosen experts, divided by their sum when ``renorm``,
    times ``route_scale``.
    """
    T, E = z.shape
    q, eligible, _ = selection_keys(z, g, select_bias)
    masked = np.where(eligible, q, -np.inf)
    ids = _topk_desc(masked, g.k).astype(np.int32)
    if g.gate == GATE_SOFTMAX_TOPK:
        zmax = z.max(axis=1, keepdims=True) if E else z
        p = np.exp(z - zmax)
        p = p / p.sum(axis=1, keepdims=True)
        w = np.take_along_axis(p, ids, axis=1)
        if g.renorm:
            w = w / w.sum(axis=1, keepdims=True)
    else:
        s = 1.0 / (1.0 + np.exp(-z))
        w = np.take_along_axis(s, ids, axis=1)
        if g.renorm:
            w = w / w.sum(axis=1, keepdims=True)
        w = w * g.route_scale
    return ids, w


def near_tie_margins(z: np.ndarray, g: Gate, select_bias: Optional[np.ndarray] = None
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """Per token: (key gap between the k-th and (k+1)-th eligible expert,
    score gap between the last kept and first dropped group).  +inf where there
    is no (k+1)-th candidate / no dropped group.  A token whose gaps are below a
    threshold may legitimately route differently under fp32 arithmetic."""
    T, E = z.shape
    q, eligible, group_score = selection_keys(z, g, select_bias)
    masked = np.where(eligible, q, -np.inf)
    srt = -np.sort(-masked, axis=1)
    if g.k < E:
        nxt = srt[:, g.k]
        key_gap = np.where(np.isfinite(nxt), srt[:, g.k - 1] - nxt, np.inf)
    else:
        key_gap = np.full(T, np.inf)
    if group_score is not None and g.topk_group < g.n_group:
        gs = -np.sort(-group_score, axis=1)
        group_gap = gs[:, g.topk_group - 1] - gs[:, g.topk_group]
    else:
        group_gap = np.full(T, np.inf)
    return key_gap, group_gap


# ----------------------------------------------------------------------------
# Eq. 5: predicted expert workload; Algorithm 1 line 2: rank loads
# ----------------------------------------------------------------------------
def expert_histogram(ids: np.ndarray, E: int) -> np.ndarray:
    """n_e = number of tokens whose assignment set contains e (Eq. 5)."""
    counts = np.zeros(E, dtype=np.int64)
    for e in np.asarray(ids).reshape(-1):
        counts[int(e)] += 1
    return counts


def rank_of_slot(slot: int, m: int) -> int:
    return slot // m


def rank_loads(counts: Sequence[int], expert_to_slot: Sequence[int], R: int) -> List[int]:
    """L_r = sum of n_e over the experts placed on rank r (Algorithm 1, line 2).
    Slot p belongs to rank p // m with m = E / R expert slots per rank."""
    E = len(counts)
    m = E // R
    L = [0] * R
    for e in range(E):
        L[rank_of_slot(int(expert_to_slot[e]), m)] += int(counts[e])
    return L


# ----------------------------------------------------------------------------
# Eqs. 9, 10: cost model and budget
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Budget:
    max_swaps: int = 0
    global_ns: int = U64_OFF
    rank_ns: int = U64_OFF
    link_ns: int = U64_OFF
    tau_tokens: int = 0
    gamma_num: int = 0
    gamma_den: int = 1
    alpha_ns: Tuple[int, int] = (0, 0)          # [intra-node, inter-node]
    fs_per_byte: Tuple[int, int] = (0, 0)       # 1/beta in femtoseconds per byte
    ranks_per_node: int = 0                     # 0 -> every rank in one node
    expert_bytes: int = 0                       # S(e), uniform ...
    expert_bytes_table: Optional[Tuple[int, ...]] = None   # ... or one size per expert
    mode: int = 0                               # PLAN_LOOP, PLAN_SWEEP or PLAN_WIDE (see plan())
    frontier_width: int = 1                     # PLAN_WIDE: ranks taken from each end of the load order


PLAN_LOOP = 0        # Algorithm 1: re-enumerate the frontier after every accepted swap
PLAN_SWEEP = 1       # the planner prose: enumerate once, sort once, one pass over the sorted list
PLAN_WIDE = 2        # Algorithm 1 with the frontier widened to several ranks at each end


def budget_ns(t_attn_ns: int, delta_ns: int) -> int:
    """B = max(0, T_attn - delta) (Eq. 10)."""
    return max(0, int(t_attn_ns) - int(delta_ns))


def link_class(a: int, b: int, ranks_per_node: int) -> int:
    if ranks_per_node <= 0:
        return 0
    return 0 if a // ranks_per_node == b // ranks_per_node else 1


def link_id(a: int, b: int, ranks_per_node: int):
    """Intra-node: the unordered rank pair.  Inter-node: the unordered node pair."""
    if link_class(a, b, ranks_per_node) == 0:
        return ("rank", min(a, b), max(a, b))
    na, nb = a // ranks_per_node, b // ranks_per_node
    return ("node", min(na, nb), max(na, nb))


def swap_cost_ns(bud: Budget, a: int, b: int, e_a: int = 0, e_b: int = 0) -> int:
    """C(s) = alpha_ab + (S(e_a) + S(e_b)) / beta_ab (Eq. 9) in whole nanoseconds:
    the transfer term is rounded up and the total is at least 1 ns."""
    cls = link_class(a, b, bud.ranks_per_node)
    if bud.expert_bytes_table is not None:
        size = int(bud.expert_bytes_table[e_a]) + int(bud.expert_bytes_table[e_b])
    else:
        size = 2 * bud.expert_bytes
    transfer = Fraction(size * bud.fs_per_byte[cls], 10**6)
    ceil_transfer = -((-transfer.numerator) // transfer.denominator)
    return max(1, bud.alpha_ns[cls] + ceil_transfer)


# ----------------------------------------------------------------------------
# Eq. 8 and Algorithm 1 lines 3-8: the deterministic greedy planner
# ----------------------------------------------------------------------------
def objective(L: Sequence[int], gamma: Fraction) -> Fraction:
    """Phi(L) = max_r L_r + gamma * sum_r (L_r - mean)^2 (Eq. 8), exact."""
    R = len(L)
    mean = Fraction(sum(L), R)
    return Fraction(max(L)) + gamma * sum((Fraction(x) - mean) ** 2 for x in L)


def plan_swaps(counts: Sequence[int], expert_to_slot: Sequence[int], R: int, bud: Budget,
               layer_id: int = 0):
    """Budgeted greedy expert-swap planning (Algorithm 1 lines 2-8 with the
    ordering, conflict and budget rules of "Budgeted Expert-Swap Planning").

    Returns (swaps, expert_to_slot_out, load_before, load_after) where each swap
    is (src_rank a, dst_rank b, expert on a, expert on b).

    One loop iteration = one pass of: take the most and the least loaded rank
    (the frontier), enumerate their expert pairs, drop pairs containing an expert
    already moved in this call, drop pairs with non-positive benefit (Eq. 8) or a
    cost that some residual budget cannot cover, and accept the pair with the
    largest benefit / cost; ties go to the lexicographically smallest
    (layer, a, b, e_a, e_b).  Loads and residual budgets are then updated
    (Eqs. 6, 7).  The loop stops when the imbalance max-min is not above tau, the
    swap cap is reached, or no pair survives.
    """
    E = len(counts)
    m = E // R
    n = [int(c) for c in counts]
    pi = [int(p) for p in expert_to_slot]
    gamma = Fraction(bud.gamma_num, bud.gamma_den) if bud.gamma_den else Fraction(0)
    L = rank_loads(n, pi, R)
    load_before = list(L)
    selected = [False] * E
    g_res = bud.global_ns
    r_res = [bud.rank_ns] * R
    l_res = {}
    swaps = []
    while len(swaps) < bud.max_swaps:
        a = max(range(R), key=lambda r: (L[r], -r))      # most loaded, lowest index on ties
        b = min(range(R), key=lambda r: (L[r], r))       # least loaded, lowest index on ties
        if L[a] - L[b] <= bud.tau_tokens:
            break
        phi = objective(L, gamma)
        lk = link_id(a, b, bud.ranks_per_node)
        lres = l_res.get(lk, bud.link_ns)
        on_a = [e for e in range(E) if rank_of_slot(pi[e], m) == a and not selected[e]]
        on_b = [e for e in range(E) if rank_of_slot(pi[e], m) == b and not selected[e]]
        best = None          # (benefit/cost, tie-break tuple, cost, new loads)
        for ea in on_a:
            for eb in on_b:
                Ln = list(L)
                Ln[a] = L[a] - n[ea] + n[eb]                      # Eq. 6
                Ln[b] = L[b] - n[eb] + n[ea]                      # Eq. 7
                benefit = phi - objective(Ln, gamma)
                if benefit <= 0:
                    continue
                cost = swap_cost_ns(bud, a, b, ea, eb)            # Eq. 9
                if bud.global_ns != U64_OFF and cost > g_res:
                    continue
                if bud.rank_ns != U64_OFF and (cost > r_res[a] or cost > r_res[b]):
                    continue
                if bud.link_ns != U64_OFF and cost > lres:
                    continue
                ratio = benefit / cost
                tie = (layer_id, a, b, ea, eb)
                if best is None or ratio > best[0] or (ratio == best[0] and tie < best[1]):
                    best = (ratio, tie, cost, Ln)
        if best is None:
            break
        _, (_, _, _, ea, eb), cost, L = best
        pi[ea], pi[eb] = pi[eb], pi[ea]
        selected[ea] = selected[eb] = True
        if bud.global_ns != U64_OFF:
            g_res -= cost
        if bud.rank_ns != U64_OFF:
            r_res[a] -= cost
            r_res[b] -= cost
        if bud.link_ns != U64_OFF:
            l_res[lk] = lres - cost
        swaps.append((a, b, ea, eb))
    return swaps, pi, load_before, list(L)


def plan_swaps_sweep(counts: Sequence[int], expert_to_slot: Sequence[int], R: int, bud: Budget,
                     layer_id: int = 0):
    """The one-pass reading of the planner's ordering paragraph ("Budgeted Expert-Swap
    Planning"): on the frontier of the given placement (most and least loaded rank)
    every expert pair is enumerated ONCE, pairs with non-positive benefit (Eq. 8,
    evaluated under the initial loads) are removed, the rest is sorted ONCE by
    decreasing benefit / cost (ties: layer, source rank, destination rank, expert
    ids), and the sorted list is swept: a pair is accepted if neither expert has been
    selected and every residual budget covers its cost; loads (Eqs. 6, 7) and residual
    budgets are updated after each accepted pair, the order is not.  Same return value
    as plan_swaps.  Unlike Algorithm 1's loop, later pairs were scored against loads
    that earlier acceptances have since changed, so the maximum rank load can rise."""
    E = len(counts)
    m = E // R
    n = [int(c) for c in counts]
    pi = [int(p) for p in expert_to_slot]
    gamma = Fraction(bud.gamma_num, bud.gamma_den) if bud.gamma_den else Fraction(0)
    L = rank_loads(n, pi, R)
    load_before = list(L)
    swaps = []
    a = max(range(R), key=lambda r: (L[r], -r))
    b = min(range(R), key=lambda r: (L[r], r))
    if bud.max_swaps == 0 or L[a] - L[b] <= bud.tau_tokens:
        return swaps, pi, load_before, list(L)
    phi = objective(L, gamma)
    cands = []
    for ea in (e for e in range(E) if rank_of_slot(pi[e], m) == a):
        for eb in (e for e in range(E) if rank_of_slot(pi[e], m) == b):
            Ln = list(L)
            Ln[a] = L[a] - n[ea] + n[eb]
            Ln[b] = L[b] - n[eb] + n[ea]
            benefit = phi - objective(Ln, gamma)
            if benefit <= 0:
                continue
            cost = swap_cost_ns(bud, a, b, ea, eb)
            cands.append((-(benefit / cost), (layer_id, a, b, ea, eb), cost))
    cands.sort()                                   # decreasing ratio, then the tie-break tuple
    selected = [False] * E
    g_res, ra_res, rb_res, l_res = bud.global_ns, bud.rank_ns, bud.rank_ns, bud.link_ns
    for _, (_, _, _, ea, eb), cost in cands:
        if len(swaps) == bud.max_swaps:
            break
        if selected[ea] or selected[eb]:
            continue
        if bud.global_ns != U64_OFF and cost > g_res:
            continue
        if bud.rank_ns != U64_OFF and (cost > ra_res or cost > rb_res):
            continue
        if bud.link_ns != U64_OFF and cost > l_res:
            continue
        L[a] += n[eb] - n[ea]                       # Eq. 6
        L[b] += n[ea] - n[eb]                       # Eq. 7
        pi[ea], pi[eb] = pi[eb], pi[ea]
        selected[ea] = selected[eb] = True
        if bud.global_ns != U64_OFF:
            g_res -= cost
        if bud.rank_ns != U64_OFF:
            ra_res -= cost
            rb_res -= cost
        if bud.link_ns != U64_OFF:
            l_res -= cost
        swaps.append((a, b, ea, eb))
    return swaps, pi, load_before, list(L)


def plan_swaps_wide(counts: Sequence[int], expert_to_slot: Sequence[int], R: int, bud: Budget,
                    layer_id: int = 0):
    """Algorithm 1's loop with a wider frontier: instead of only the most and the
    least loaded rank (the restriction the end of "Budgeted Expert-Swap Planning"
    describes as the practical choice), every iteration considers the
    ``frontier_width`` most loaded ranks as sources and the ``frontier_width`` least
    loaded ranks as destinations (lowest index on equal loads; a source must carry
    strictly more than its destination).  Benefit (Eq. 8), cost (Eq. 9), budgets,
    conflicts and the ordering rule are those of plan_swaps; the source and
    destination rank now take part in the tie-break.  Width 1 is plan_swaps."""
    E = len(counts)
    m = E // R
    W = max(1, min(int(bud.frontier_width), R))
    n = [int(c) for c in counts]
    pi = [int(p) for p in expert_to_slot]
    gamma = Fraction(bud.gamma_num, bud.gamma_den) if bud.gamma_den else Fraction(0)
    L = rank_loads(n, pi, R)
    load_before = list(L)
    selected = [False] * E
    g_res = bud.global_ns
    r_res = [bud.rank_ns] * R
    l_res = {}
    swaps = []
    while len(swaps) < bud.max_swaps:
        top = sorted(range(R), key=lambda r: (-L[r], r))[:W]
        bottom = sorted(range(R), key=lambda r: (L[r], r))[:W]
        if L[top[0]] - L[bottom[0]] <= bud.tau_tokens:
            break
        phi = objective(L, gamma)
        best = None
        for a in top:
            for b in bottom:
                if a == b or L[a] <= L[b]:
                    continue
                lk = link_id(a, b, bud.ranks_per_node)
                lres = l_res.get(lk, bud.link_ns)
                for ea in (e for e in range(E) if rank_of_slot(pi[e], m) == a and not selected[e]):
                    for eb in (e for e in range(E) if rank_of_slot(pi[e], m) == b and not selected[e]):
                        Ln = list(L)
                        Ln[a] = L[a] - n[ea] + n[eb]
                        Ln[b] = L[b] - n[eb] + n[ea]
                        benefit = phi - objective(Ln, gamma)
                        if benefit <= 0:
                            continue
                        cost = swap_cost_ns(bud, a, b, ea, eb)
                        if bud.global_ns != U64_OFF and cost > g_res:
                            continue
                        if bud.rank_ns != U64_OFF and (cost > r_res[a] or cost > r_res[b]):
                            continue
                        if bud.link_ns != U64_OFF and cost > lres:
                            continue
                        ratio = benefit / cost
                        tie = (layer_id, a, b, ea, eb)
                        if best is None or ratio > best[0] or (ratio == best[0] and tie < best[1]):
                            best = (ratio, tie, cost, Ln)
        if best is None:
            break
        _, (_, a, b, ea, eb), cost, L = best
        pi[ea], pi[eb] = pi[eb], pi[ea]
        selected[ea] = selected[eb] = True
        if bud.global_ns != U64_OFF:
            g_res -= cost
        if bud.rank_ns != U64_OFF:
            r_res[a] -= cost
            r_res[b] -= cost
        if bud.link_ns != U64_OFF:
            lk = link_id(a, b, bud.ranks_per_node)
            l_res[lk] = l_res.get(lk, bud.link_ns) - cost
        swaps.append((a, b, ea, eb))
    return swaps, pi, load_before, list(L)


def plan(counts: Sequence[int], expert_to_slot: Sequence[int], R: int, bud: Budget, layer_id: int = 0):
    """The planner in the mode the budget names: Algorithm 1's loop (default), the one-pass
    sorted sweep, or the loop with a widened frontier."""
    if bud.mode == PLAN_SWEEP:
        return plan_swaps_sweep(counts, expert_to_slot, R, bud, layer_id)
    if bud.mode == PLAN_WIDE:
        return plan_swaps_wide(counts, expert_to_slot, R, bud, layer_id)
    return plan_swaps(counts, expert_to_slot, R, bud, layer_id)


# ----------------------------------------------------------------------------
# Stage 4: dispatch index under the committed placement
# ----------------------------------------------------------------------------
def dispatch_index(ids: np.ndarray, expert_to_slot: Sequence[int], R: int):
    """Token -> expert dispatch order under placement pi'.

    Assignment (i, j) (token i, j-th chosen expert) goes to physical slot
    p = pi'[ids[i, j]].  Assignments are laid out by (p, i) ascending, so the
    tokens of one slot are contiguous, the slots of one rank are contiguous and
    tokens keep their order inside a slot.

    Returns (slot_offsets [E+1], rank_offsets [R+1], perm [T*k], inv_perm [T*k],
    rank_load [R]); perm[pos] = i*k + j and inv_perm[i*k + j] = pos.
    """
    ids = np.asarray(ids)
    T, k = ids.shape
    E = len(expert_to_slot)
    m = E // R
    flat = [(int(expert_to_slot[int(ids[i, j])]), i, i * k + j) for i in range(T) for j in range(k)]
    flat.sort(key=lambda t: (t[0], t[1]))
    perm = np.array([f for (_, _, f) in flat], dtype=np.int64).reshape(-1)
    inv_perm = np.zeros(T * k, dtype=np.int64)
    for pos, f in enumerate(perm):
        inv_perm[f] = pos
    slot_count = [0] * E
    for (p, _, _) in flat:
        slot_count[p] += 1
    slot_offsets = [0] * (E + 1)
    for p in range(E):
        slot_offsets[p + 1] = slot_offsets[p] + slot_count[p]
    rank_offsets = [slot_offsets[r * m] for r in range(R)] + [slot_offsets[E]]
    rank_load = [rank_offsets[r + 1] - rank_offsets[r] for r in range(R)]
    return (np.array(slot_offsets, dtype=np.int64), np.array(rank_offsets, dtype=np.int64),
            perm, inv_perm, np.array(rank_load, dtype=np.int64))


def globalize_dispatch(slot_counts_all: Sequence[Sequence[int]], rank: int, slot_offsets_local: Sequence[int],
                       inv_perm_local: Sequence[int], R: int):
    """Token-sharded dispatch: from a shard's own dispatch index to positions in the dispatch
    order of the whole batch.

    The ranks hold contiguous token ranges in rank order, and the order of the whole batch is by
    (slot, token), so inside slot p the assignments of earlier ranks come first.  With
    ``slot_counts_all[r][p]`` the number of assignments rank r sends to slot p (the exchange
    step: an all-gather of E counts per rank), the position of a local assignment whose local
    position is ``q`` in slot p is  G[p] + sum_{r' < rank} slot_counts_all[r'][p] + (q -
    slot_offsets_local[p]),  where G is the exclusive prefix over the slots of the counts summed
    over all ranks.  Returns (slot_offsets [E+1], rank_offsets [R+1], rank_load [R]) of the whole
    batch and the shard's inv_perm in whole-batch positions."""
    world = len(slot_counts_all)
    E = len(slot_counts_all[0])
    m = E // R
    total = [sum(int(slot_counts_all[r][p]) for r in range(world)) for p in range(E)]
    G = [0] * (E + 1)
    for p in range(E):
        G[p + 1] = G[p] + total[p]
    before = [sum(int(slot_counts_all[r][p]) for r in range(rank)) for p in range(E)]
    out = []
    for q in inv_perm_local:
        q = int(q)
        p = max(s for s in range(E) if int(slot_offsets_local[s]) <= q and int(slot_offsets_local[s + 1]) > q)
        out.append(G[p] + before[p] + q - int(slot_offsets_local[p]))
    rank_offsets = [G[r * m] for r in range(R)] + [G[E]]
    rank_load = [rank_offsets[r + 1] - rank_offsets[r] for r in range(R)]
    return (np.array(G, dtype=np.int64), np.array(rank_offsets, dtype=np.int64),
            np.array(rank_load, dtype=np.int64), np.array(out, dtype=np.int64))


# ----------------------------------------------------------------------------
# Evaluation metrics (Evaluation, "Metrics")
# ----------------------------------------------------------------------------
def max_over_mean(L: Sequence[int]) -> float:
    s = sum(int(x) for x in L)
    return float(max(L)) * len(L) / s if s else 1.0


def topk_hit_rate(ids_early: np.ndarray, ids_final: np.ndarray) -> float:
    """Fraction of final top-k assignments recovered by the early pass."""
    T, k = ids_final.shape
    hit = 0
    for i in range(T):
        hit += len(set(ids_early[i].tolist()) & set(ids_final[i].tolist()))
    return hit / (T * k) if T * k else 1.0


# ----------------------------------------------------------------------------
# One layer end to end, in the order of Algorithm 1
# ----------------------------------------------------------------------------
def layer_step(h_prev_bits, H_bits, W_bits, gate: Gate, R: int, expert_to_slot, bud: Budget,
               select_bias=None, logit_bias=None, layer_id: int = 0):
    """predict -> plan -> (placement committed) -> normal routing -> dispatch index."""
    z_early = router_logits(h_prev_bits, W_bits, logit_bias)                   # Eq. 2
    ids_early, _ = select_topk(z_early, gate, select_bias)
    counts = expert_histogram(ids_early, gate.E)                               # Eq. 5
    swaps, pi_new, load_before, load_after = plan_swaps(counts, expert_to_slot, R, bud, layer_id)
    z = router_logits(H_bits, W_bits, logit_bias)                              # Eq. 3
    ids, w = select_topk(z, gate, select_bias)
    disp = dispatch_index(ids, pi_new, R)
    return dict(z_early=z_early, ids_early=ids_early, counts=counts, swaps=swaps, pi_new=pi_new,
                load_before=load_before, load_after=load_after, z=z, ids=ids, w=w, dispatch=disp)


# ----------------------------------------------------------------------------
# Prediction / planning quality over a sequence of prefill steps
# (Evaluation, "Metrics" and "Prediction and Planning Quality")
# ----------------------------------------------------------------------------
def row_cosine_mean(a: np.ndarray, b: np.ndarray) -> float:
    """Cosine similarity between corresponding rows (tokens) of a and b, averaged over
    the rows; a row with a zero vector on either side contributes 0."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    if a.shape[0] == 0:
        return 0.0
    total = 0.0
    for i in range(a.shape[0]):
        na = math.sqrt(float(np.dot(a[i], a[i])))
        nb = math.sqrt(float(np.dot(b[i], b[i])))
        if na > 0.0 and nb > 0.0:
            total += float(np.dot(a[i], b[i])) / (na * nb)
    return total / a.shape[0]


def serving_loop(trace, gate: Gate, R: int, bud: Budget, with_cosines: bool = True):
    """Run layer_step over a sequence of prefill steps with the placement of every layer
    carried from one step to the next (a committed swap plan stays in force until a later
    plan changes it), and record the paper's quality metrics per (step, layer).

    ``trace`` yields ``(step, layer, h_prev_bits, H_bits, W_bits, select_bias, logit_bias)``
    in execution order.  Returns ``(records, summary, placements)``.
    """
    placements = {}
    records = []
    for step, layer, h_prev_bits, H_bits, W_bits, select_bias, logit_bias in trace:
        pi_old = placements.get(layer, list(range(gate.E)))
        out = layer_step(h_prev_bits, H_bits, W_bits, gate, R, pi_old, bud, select_bias, logit_bias, layer)
        realized = expert_histogram(out["ids"], gate.E)
        real_before = rank_loads(realized, pi_old, R)
        real_after = rank_loads(realized, out["pi_new"], R)
        real_vanilla = rank_loads(realized, list(range(gate.E)), R)      # the fixed initial placement
        rec = dict(step=step, layer=layer, pi_old=list(pi_old), pi_new=list(out["pi_new"]), swaps=out["swaps"],
                   counts=out["counts"], realized=realized,
                   pred_before=max_over_mean(out["load_before"]), pred_after=max_over_mean(out["load_after"]),
                   real_before=max_over_mean(real_before), real_after=max_over_mean(real_after),
                   real_vanilla=max_over_mean(real_vanilla),
                   hit_rate=topk_hit_rate(out["ids_early"], out["ids"]),
                   improved=max_over_mean(real_after) < max_over_mean(real_before))
        if with_cosines:
            rec["cos_hidden"] = row_cosine_mean(bf16_bits_to_f64(h_prev_bits), bf16_bits_to_f64(H_bits))
            rec["cos_logits"] = row_cosine_mean(out["z_early"], out["z"])
        records.append(rec)
        placements[layer] = list(out["pi_new"])
    moved = [r for r in records if len(r["swaps"]) > 0]
    n = max(1, len(records))
    summary = dict(
        layers_run=len(records),
        swaps_per_layer=sum(len(r["swaps"]) for r in records) / n,
        hit_rate=sum(r["hit_rate"] for r in records) / n,
        real_max_over_mean_vanilla=max((r["real_vanilla"] for r in records), default=1.0),
        real_max_over_mean_balanced=max((r["real_after"] for r in records), default=1.0),
        layers_with_migration=len(moved),
        improved_fraction=(sum(1 for r in moved if r["improved"]) / len(moved)) if moved else None,
    )
    if with_cosines and records:
        summary["cos_hidden"] = sum(r["cos_hidden"] for r in records) / n
        summary["cos_logits"] = sum(r["cos_logits"] for r in records) / n
    return records, summary, placements


# ----------------------------------------------------------------------------
# Stage 3 on one device: the accepted swaps applied to the expert weights
# (Method overview, "Weight Transfer"; "Budgeted Expert-Swap Planning", pairwise exchange)
# ----------------------------------------------------------------------------
def apply_swaps(slot_weights: np.ndarray, expert_to_slot: Sequence[int], swaps):
    """Exchange, swap by swap, the weights of the two experts of each accepted swap between
    the physical slots that hold them.  ``slot_weights[p]`` is the byte image of the expert
    in slot p.  Returns ``(new_slot_weights, expert_to_slot_after)``."""
    w = np.array(slot_weights, copy=True)
    pi = [int(p) for p in expert_to_slot]
    for _, _, e_a, e_b in swaps:
        pa, pb = pi[e_a], pi[e_b]
        tmp = w[pa].copy()
        w[pa] = w[pb]
        w[pb] = tmp
        pi[e_a], pi[e_b] = pb, pa
    return w, pi


# ----------------------------------------------------------------------------
# Cost-model calibration and per-attention-type budgets ("Budgeted Expert-Swap Planning")
# ----------------------------------------------------------------------------
def fit_cost_model(t_small_ns: int, t_large_ns: int, bytes_small: int, bytes_large: int):
    """Eq. 9 fitted through two timed exchanges of experts of two sizes:
    C = alpha + (S(e_a) + S(e_b)) / beta with S(e_a) = S(e_b) = bytes.  Returns
    ``(alpha_ns, fs_per_byte)`` in the planner's integer units: 1/beta rounded up to whole
    femtoseconds per byte, alpha rounded down to whole nanoseconds and clamped at 0."""
    d_bytes = 2 * (bytes_large - bytes_small)
    d_t = t_large_ns - t_small_ns
    if d_bytes <= 0 or d_t <= 0:
        raise ValueError("the larger exchange must move more bytes and take longer")
    inv_beta = Fraction(d_t * 1_000_000, d_bytes)                       # femtoseconds per byte
    fs_per_byte = -((-inv_beta.numerator) // inv_beta.denominator)      # ceiling
    alpha = Fraction(t_small_ns) - Fraction(2 * bytes_small) * inv_beta / 1_000_000
    return max(0, alpha.numerator // alpha.denominator), fs_per_byte


def budgets_by_attention_type(layer_types: Sequence[str], profiled_ns: dict, delta_ns: int) -> List[int]:
    """Eq. 10 per layer: B_l = max(0, T_attn[r(l)] - delta), where r(l) is the first layer with
    the attention type of layer l and ``profiled_ns`` maps that first layer to its measured time."""
    first = {}
    out = []
    for l, t in enumerate(layer_types):
        first.setdefault(t, l)
        out.append(budget_ns(profiled_ns[first[t]], delta_ns))
    return out
