"""Run one layer through the CUDA library and through the CPU oracle on the same
seeded inputs and compare them.  Used by the GPU tests and the smoke check.

Comparison rules
* logits: |gpu - oracle| <= LOGIT_TOL everywhere.
* top-k: per-token expert sets must be equal, except for tokens whose oracle margin
  (gap between the k-th and (k+1)-th eligible key, or between the last kept and first
  dropped group score) is below the near-tie threshold; those are counted.  Two
  thresholds are asserted: 2e-3 (the stated one) and a tight one, 1e-4 or - when it is
  larger - the bound that the measured logit error of this very comparison implies
  (two keys can only change order if their gap is below twice the key error).
* everything integer (counts, plan, placement, loads, dispatch index) is rechecked
  bit-exactly by feeding the GPU's own top-k to the oracle, and must additionally equal
  the oracle's own pipeline when no token differed.
* the one-call layer step is checked the same way, on its own outputs (not against the
  separate calls: the kernel variants differ in the order of their fp32 sums).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I

LOGIT_TOL = 2e-3
NEAR_TIE = 2e-3
NEAR_TIE_TIGHT = 1e-4
WEIGHT_TOL = 2e-3


def budget_kwargs(wl: I.Workload, T: int, **override):
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    kw = dict(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
              link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
              alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
              ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)
    kw.update(override)
    return kw


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_gate(wl: I.Workload) -> O.Gate:
    return O.Gate(E=wl.E, k=wl.k, gate=wl.gate, n_group=wl.n_group, topk_group=wl.topk_group,
                  renorm=wl.renorm, route_scale=wl.route_scale)


def make_context(wl: I.Workload, T_max: int) -> B.Context:
    return B.Context(T_max, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm,
                     wl.route_scale)


GUARD_WORDS = 64                      # 256 bytes of known pattern before and after every output
GUARD_PATTERN = 0x5A5AA5A5


class GuardedOutputs:
    """Output buffers with guard regions.  compute-sanitizer is not available to these tests, so
    every output the library writes sits between two 256-byte regions of a known pattern; a write
    past either end of a buffer shows up as a damaged guard."""

    def __init__(self, dev):
        self.dev = dev
        self._all = []

    def _alloc(self, n, dtype, fill):
        n = max(1, int(n))
        whole = torch.full((n + 2 * GUARD_WORDS,), GUARD_PATTERN, dtype=torch.int32, device=self.dev)
        body = whole[GUARD_WORDS:GUARD_WORDS + n]
        view = body.view(dtype)
        view.fill_(fill)
        self._all.append((whole, n))
        return view

    def i32(self, n):
        return self._alloc(n, torch.int32, 0x7FFFFFFF)

    def f32(self, n):
        return self._alloc(n, torch.float32, float("nan"))

    def check(self):
        for whole, n in self._all:
            front = whole[:GUARD_WORDS]
            back = whole[GUARD_WORDS + n:]
            assert bool((front == GUARD_PATTERN).all()) and bool((back == GUARD_PATTERN).all()), \
                f"a kernel wrote outside an output buffer of {n} words"


def run_gpu_layer(ctx: B.Context, wl: I.Workload, li: I.LayerInputs, bkw: dict, want_logits=True,
                  placement=None, pair_limit=0):
    """All entry points on one layer; returns numpy copies of every output.

    ``pair_limit`` > 0 caps the SM pairs of the router kernel for these calls, which sends
    calls with more tile pairs than that through the persistent kernel."""
    ctx.fb_set_pair_limit(pair_limit)
    dev = torch.device("cuda", ctx.device)
    T = li.h_prev.shape[0]
    E, R, k = wl.E, wl.R, wl.k
    W = li.W.to(dev)
    lb = li.logit_bias.to(dev) if li.logit_bias is not None else None
    sb = li.select_bias.to(dev) if li.select_bias is not None else None
    router = B.make_router(W, lb, sb)
    h_prev = li.h_prev.to(dev)
    H = li.H.to(dev)
    pi = (li.expert_to_slot if placement is None else placement).to(dev)
    table = bkw.get("expert_bytes_table")
    bkw = dict(bkw)
    if table is not None:
        bkw["expert_bytes_table"] = torch.as_tensor(np.asarray(table, dtype=np.int64)).to(dev)
    budget = B.make_budget(**bkw)
    ms = max(1, budget.max_swaps)

    guarded = GuardedOutputs(dev)
    u32 = guarded.i32
    counts, ids_early = u32(E), u32(max(1, T * k)).view(-1)
    logits_early = guarded.f32(T * E) if want_logits else None
    ctx.fb_predict_load(router, h_prev, T, counts, ids_early, logits_early)
    pi_out, swaps, n_swaps, lb4, la4 = u32(E), u32(4 * ms), u32(1), u32(R), u32(R)
    ctx.fb_plan_swaps(counts, pi, budget, 0, pi_out, swaps, n_swaps, lb4, la4)
    # fused entry point into separate buffers
    f_counts, f_pi_out, f_swaps, f_n, f_lb, f_la = u32(E), u32(E), u32(4 * ms), u32(1), u32(R), u32(R)
    ctx.fb_predict_and_plan(router, h_prev, T, pi, budget, 0, f_counts, f_pi_out, f_swaps, f_n, f_lb, f_la)
    ids = u32(max(1, T * k))
    w = guarded.f32(T * k)
    slot_offsets, rank_offsets, rank_load = u32(E + 1), u32(R + 1), u32(R)
    perm, inv_perm = u32(max(1, T * k)), u32(max(1, T * k))
    logits = guarded.f32(T * E) if want_logits else None
    ctx.fb_route_dispatch(router, H, T, f_pi_out, ids, w, slot_offsets, rank_offsets, perm, inv_perm, rank_load,
                          logits)
    # the whole layer in one call, into buffers of its own
    l_counts, l_pi_out, l_swaps, l_n, l_lb, l_la = u32(E), u32(E), u32(4 * ms), u32(1), u32(R), u32(R)
    l_ids, l_w = u32(max(1, T * k)), guarded.f32(T * k)
    l_so, l_ro, l_rl = u32(E + 1), u32(R + 1), u32(R)
    l_perm, l_inv = u32(max(1, T * k)), u32(max(1, T * k))
    ctx.fb_layer_step(router, h_prev, H, T, pi, budget, 0, l_counts, l_pi_out, l_swaps, l_n, l_lb, l_la,
                      l_ids, l_w, l_so, l_ro, l_perm, l_inv, l_rl)
    status = ctx.fb_device_status()
    torch.cuda.synchronize(dev)
    guarded.check()
    ctx.fb_set_pair_limit(0)
    n = int(n_swaps.item())
    fn = int(f_n.item())
    ln = int(l_n.item())
    out = dict(
        status=status,
        counts=counts.cpu().numpy().astype(np.int64),
        ids_early=ids_early.cpu().numpy()[:T * k].reshape(T, k),
        logits_early=logits_early.cpu().numpy()[:T * E].reshape(T, E).astype(np.float64) if want_logits else None,
        swaps=[tuple(r) for r in swaps.cpu().numpy().reshape(-1, 4)[:n].tolist()],
        pi_out=pi_out.cpu().numpy().tolist(), load_before=lb4.cpu().numpy().tolist(),
        load_after=la4.cpu().numpy().tolist(),
        fused=dict(counts=f_counts.cpu().numpy().astype(np.int64),
                   swaps=[tuple(r) for r in f_swaps.cpu().numpy().reshape(-1, 4)[:fn].tolist()],
                   pi_out=f_pi_out.cpu().numpy().tolist(), load_before=f_lb.cpu().numpy().tolist(),
                   load_after=f_la.cpu().numpy().tolist()),
        ids=ids.cpu().numpy()[:T * k].reshape(T, k), w=w.cpu().numpy()[:T * k].reshape(T, k).astype(np.float64),
        logits=logits.cpu().numpy()[:T * E].reshape(T, E).astype(np.float64) if want_logits else None,
        slot_offsets=slot_offsets.cpu().numpy().astype(np.int64),
        rank_offsets=rank_offsets.cpu().numpy().astype(np.int64),
        perm=perm.cpu().numpy()[:T * k].astype(np.int64), inv_perm=inv_perm.cpu().numpy()[:T * k].astype(np.int64),
        rank_load=rank_load.cpu().numpy().astype(np.int64),
        layer=dict(counts=l_counts.cpu().numpy().astype(np.int64),
                   swaps=[tuple(r) for r in l_swaps.cpu().numpy().reshape(-1, 4)[:ln].tolist()],
                   pi_out=l_pi_out.cpu().numpy().tolist(), load_before=l_lb.cpu().numpy().tolist(),
                   load_after=l_la.cpu().numpy().tolist(),
                   ids=l_ids.cpu().numpy()[:T * k].reshape(T, k),
                   w=l_w.cpu().numpy()[:T * k].reshape(T, k).astype(np.float64),
                   slot_offsets=l_so.cpu().numpy().astype(np.int64),
                   rank_offsets=l_ro.cpu().numpy().astype(np.int64),
                   perm=l_perm.cpu().numpy()[:T * k].astype(np.int64),
                   inv_perm=l_inv.cpu().numpy()[:T * k].astype(np.int64),
                   rank_load=l_rl.cpu().numpy().astype(np.int64)),
    )
    return out


def oracle_budget(bkw: dict) -> O.Budget:
    kw = dict(bkw)
    if kw.get("expert_bytes_table") is not None:
        kw["expert_bytes_table"] = tuple(int(x) for x in kw["expert_bytes_table"])
    return O.Budget(**kw)


def _set_mismatch(ids_gpu: np.ndarray, ids_ref: np.ndarray) -> np.ndarray:
    return (np.sort(ids_gpu, axis=1) != np.sort(ids_ref, axis=1)).any(axis=1)


def compare_routing(name, z_gpu, ids_gpu, z_ref, ids_ref, gate, select_bias, report):
    T = z_ref.shape[0]
    if z_gpu is not None and T:
        err = float(np.abs(z_gpu - z_ref).max())
        report[f"{name}_logit_max_err"] = err
        assert err <= LOGIT_TOL, f"{name}: logit error {err}"
    assert ids_gpu.min(initial=0) >= 0 and ids_gpu.max(initial=0) < gate.E
    if T:
        srt = np.sort(ids_gpu, axis=1)
        assert (np.diff(srt, axis=1) > 0).all() if gate.k > 1 else True, f"{name}: duplicate expert in a token"
    key_gap, group_gap = O.near_tie_margins(z_ref, gate, select_bias)
    mism = _set_mismatch(ids_gpu, ids_ref)
    # How far a selection key can be off, given the logit error measured above: a softmax key
    # is the logit; a sigmoid key moves by at most a quarter of the logit error, plus the
    # kernel's approximate exp / reciprocal and the fp32 rounding of the key (< 1e-6 together).
    tight = NEAR_TIE_TIGHT
    if z_gpu is not None and T:
        key_err = err if gate.gate == O.GATE_SOFTMAX_TOPK else 0.25 * err + 1e-6
        tight = max(tight, 2.0 * key_err)
    report[f"{name}_tight_eps"] = tight
    for tag, eps in (("", NEAR_TIE), ("_tight", tight)):
        flagged = (key_gap < eps) | (group_gap < 2 * eps)
        report[f"{name}_flagged{tag}"] = int(flagged.sum())
        report[f"{name}_mismatch_flagged{tag}"] = int((mism & flagged).sum())
        report[f"{name}_mismatch_unflagged{tag}"] = int((mism & ~flagged).sum())
    assert report[f"{name}_mismatch_unflagged"] == 0, f"{name}: {report}"
    assert report[f"{name}_mismatch_unflagged_tight"] == 0, f"{name}: {report}"
    return mism


def compare_layer(wl: I.Workload, li: I.LayerInputs, bkw: dict, gpu: dict, placement=None,
                  sample_rows=None) -> dict:
    """Assert parity of every output; returns a report of counts and error figures.

    With ``sample_rows`` (an index array) the float64 router product, and with it the
    logit / top-k comparison, is restricted to those tokens; every integer output is
    still checked in full from the GPU's own top-k."""
    report = {}
    rows = slice(None) if sample_rows is None else np.asarray(sample_rows)
    full = sample_rows is None
    gate = oracle_gate(wl)
    bud = oracle_budget(bkw)
    R, E, k = wl.R, wl.E, wl.k
    pi0 = (li.expert_to_slot if placement is None else placement).numpy().tolist()
    sb = li.select_bias.numpy().astype(np.float64) if li.select_bias is not None else None
    lb = li.logit_bias.numpy().astype(np.float64) if li.logit_bias is not None else None
    assert gpu["status"] == 0, f"device status {gpu['status']}"

    # ---- early pass (Eqs. 2, 4, 5)
    z_early = O.router_logits(bits(li.h_prev)[rows], bits(li.W), lb)
    ids_early, _ = O.select_topk(z_early, gate, sb)
    mism_early = compare_routing("early", None if gpu["logits_early"] is None else gpu["logits_early"][rows],
                                 gpu["ids_early"][rows], z_early, ids_early, gate, sb, report)
    counts_from_gpu_ids = O.expert_histogram(gpu["ids_early"], E)
    assert gpu["counts"].tolist() == counts_from_gpu_ids.tolist(), "histogram != histogram of the GPU's own top-k"
    assert int(gpu["counts"].sum()) == li.h_prev.shape[0] * k
    if full and not mism_early.any():
        assert gpu["counts"].tolist() == O.expert_histogram(ids_early, E).tolist()

    # ---- planner (Algorithm 1), recomputed from the GPU's own counts
    swaps, pi_new, before, after = O.plan_swaps(gpu["counts"].tolist(), pi0, R, bud)
    assert gpu["swaps"] == swaps, f"plan differs: gpu {gpu['swaps']} oracle {swaps}"
    assert gpu["pi_out"] == pi_new and gpu["load_before"] == before and gpu["load_after"] == after
    f = gpu["fused"]
    assert f["counts"].tolist() == gpu["counts"].tolist(), "fused counts differ from the two-call path"
    assert f["swaps"] == swaps and f["pi_out"] == pi_new and f["load_before"] == before and f["load_after"] == after
    report["n_swaps"] = len(swaps)
    report["pred_max_over_mean_before"] = O.max_over_mean(before)
    report["pred_max_over_mean_after"] = O.max_over_mean(after)

    # ---- normal routing pass (Eq. 3) and dispatch index under pi'
    z = O.router_logits(bits(li.H)[rows], bits(li.W), lb)
    ids, w = O.select_topk(z, gate, sb)
    mism = compare_routing("final", None if gpu["logits"] is None else gpu["logits"][rows], gpu["ids"][rows],
                           z, ids, gate, sb, report)
    T = z.shape[0]
    if T:
        same = ~mism
        order_g = np.argsort(gpu["ids"][rows], axis=1)
        order_r = np.argsort(ids, axis=1)
        wg = np.take_along_axis(gpu["w"][rows], order_g, axis=1)[same]
        wr = np.take_along_axis(w, order_r, axis=1)[same]
        werr = float(np.abs(wg - wr).max()) if wg.size else 0.0
        report["weight_max_err"] = werr
        assert werr <= WEIGHT_TOL, f"routing weight error {werr}"
    so, ro, perm, inv, rl = O.dispatch_index(gpu["ids"], pi_new, R)
    assert gpu["slot_offsets"].tolist() == so.tolist()
    assert gpu["rank_offsets"].tolist() == ro.tolist()
    assert gpu["rank_load"].tolist() == rl.tolist()
    assert np.array_equal(gpu["perm"], perm), "perm differs"
    assert np.array_equal(gpu["inv_perm"], inv), "inv_perm differs"
    # ---- the one-call layer step, checked on its own against the oracle.  Its router passes may
    # run another kernel variant than the separate calls (persistent kernel, k-range split), whose
    # fp32 sums are formed in another order: logits agree to rounding, so a token at a near tie
    # may be routed differently by the two and everything downstream follows the call's own top-k.
    ly = gpu["layer"]
    T_all = li.h_prev.shape[0]
    assert int(ly["counts"].sum()) == T_all * k
    moved = int(np.abs(ly["counts"] - gpu["counts"]).sum()) // 2
    if full:
        assert moved <= k * report["early_flagged_tight"], "layer step: counts differ beyond the near-tie tokens"
    report["layer_counts_moved"] = moved
    l_swaps, l_pi, l_before, l_after = O.plan_swaps(ly["counts"].tolist(), pi0, R, bud)
    assert ly["swaps"] == l_swaps and ly["pi_out"] == l_pi, "layer step: plan differs from the oracle's on its counts"
    assert ly["load_before"] == l_before and ly["load_after"] == l_after
    mism_l = compare_routing("layer", None, ly["ids"][rows], z, ids, gate, sb, report)
    if T:
        same = ~mism_l
        wg = np.take_along_axis(ly["w"][rows], np.argsort(ly["ids"][rows], axis=1), axis=1)[same]
        wr = np.take_along_axis(w, np.argsort(ids, axis=1), axis=1)[same]
        assert (float(np.abs(wg - wr).max()) if wg.size else 0.0) <= WEIGHT_TOL, "layer step: routing weights"
    l_so, l_ro, l_perm, l_inv, l_rl = O.dispatch_index(ly["ids"], l_pi, R)
    assert ly["slot_offsets"].tolist() == l_so.tolist() and ly["rank_offsets"].tolist() == l_ro.tolist()
    assert ly["rank_load"].tolist() == l_rl.tolist()
    assert np.array_equal(ly["perm"], l_perm) and np.array_equal(ly["inv_perm"], l_inv), "layer step: dispatch index"
    realized = O.expert_histogram(gpu["ids"], E)
    report["real_max_over_mean_before"] = O.max_over_mean(O.rank_loads(realized, pi0, R))
    report["real_max_over_mean_after"] = O.max_over_mean(O.rank_loads(realized, pi_new, R))
    report["hit_rate"] = O.topk_hit_rate(gpu["ids_early"], gpu["ids"])
    return report
