"""Pins for the oracle's quality metrics and its multi-step serving loop
(Evaluation, "Metrics"; "Prediction and Planning Quality")."""
import math

import numpy as np
import pytest

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import inputs as I


def bits(t):
    import torch
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------ row_cosine_mean: closed forms
def test_cosine_closed_forms():
    a = np.array([[1.0, 0.0], [0.0, 2.0], [3.0, 3.0]])
    assert O.row_cosine_mean(a, a) == pytest.approx(1.0, abs=1e-15)
    assert O.row_cosine_mean(a, -a) == pytest.approx(-1.0, abs=1e-15)
    assert O.row_cosine_mean(a, 7.5 * a) == pytest.approx(1.0, abs=1e-15)          # scale invariance
    orth = np.array([[0.0, 1.0], [5.0, 0.0], [1.0, -1.0]])
    assert O.row_cosine_mean(a, orth) == pytest.approx(0.0, abs=1e-15)
    # one row at 45 degrees, one equal, one opposite: (1/sqrt2 + 1 - 1) / 3
    x = np.array([[1.0, 0.0], [2.0, 1.0], [1.0, 1.0]])
    y = np.array([[1.0, 1.0], [4.0, 2.0], [-2.0, -2.0]])
    assert O.row_cosine_mean(x, y) == pytest.approx((1 / math.sqrt(2)) / 3, abs=1e-15)


def test_cosine_is_a_mean_over_rows_and_zero_rows_count_as_zero():
    x = np.array([[1.0, 0.0], [0.0, 0.0], [0.0, 1.0], [1.0, 0.0]])
    y = np.array([[1.0, 0.0], [3.0, 4.0], [0.0, 0.0], [0.0, 1.0]])
    assert O.row_cosine_mean(x, y) == pytest.approx(1.0 / 4, abs=1e-15)
    assert O.row_cosine_mean(np.zeros((0, 3)), np.zeros((0, 3))) == 0.0
    # a dropped normalisation or a sum instead of a mean would both show here
    z = np.array([[3.0, 4.0]] * 5)
    assert O.row_cosine_mean(z, np.array([[4.0, 3.0]] * 5)) == pytest.approx(24 / 25, abs=1e-15)


# ------------------------------------------------------------------ serving_loop
def _trace(wl, steps, layers, T, seed=0, sys_drift=0.0):
    for s in range(steps):
        for l in layers:
            li = I.make_step_layer(wl, l, s, seed, T=T, sys_drift=sys_drift)
            sb = li.select_bias.numpy().astype(np.float64) if li.select_bias is not None else None
            yield s, l, bits(li.h_prev), bits(li.H), bits(li.W), sb, None


def _gate(wl):
    return O.Gate(E=wl.E, k=wl.k, gate=wl.gate, n_group=wl.n_group, topk_group=wl.topk_group,
                  renorm=wl.renorm, route_scale=wl.route_scale)


def _budget(wl, T, **kw):
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    base = dict(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
                link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
                alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
                ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)
    base.update(kw)
    return O.Budget(**base)


def test_placement_is_carried_from_step_to_step_per_layer():
    wl = I.WORKLOADS["tiny"]
    T, steps, layers = 256, 3, (0, 1)
    gate, bud = _gate(wl), _budget(wl, T)
    records, summary, placements = O.serving_loop(_trace(wl, steps, layers, T), gate, wl.R, bud)
    assert len(records) == steps * len(layers) and summary["layers_run"] == 6
    carried = {l: list(range(wl.E)) for l in layers}
    for rec, item in zip(records, _trace(wl, steps, layers, T)):
        s, l, hb, Hb, Wb, sb, lb = item
        assert (rec["step"], rec["layer"]) == (s, l)
        assert rec["pi_old"] == carried[l], "a layer starts from the placement its previous step committed"
        ref = O.layer_step(hb, Hb, Wb, gate, wl.R, carried[l], bud, sb, lb, l)
        assert rec["swaps"] == ref["swaps"] and rec["pi_new"] == ref["pi_new"]
        assert sorted(rec["pi_new"]) == list(range(wl.E))
        carried[l] = ref["pi_new"]
    assert placements == carried


def test_realised_load_figures_hand_worked():
    # E = 4 experts on R = 2 ranks (slots 0,1 -> rank 0; 2,3 -> rank 1), k = 1.
    # Step A realises counts n = (6, 2, 1, 1): under the contiguous placement the rank loads are
    # (8, 2): max/mean 1.6.  Exchanging experts 1 and 2 (placement (0, 2, 1, 3)) gives (7, 3): 1.4.
    n = [6, 2, 1, 1]
    assert O.max_over_mean(O.rank_loads(n, [0, 1, 2, 3], 2)) == pytest.approx(1.6)
    assert O.max_over_mean(O.rank_loads(n, [0, 2, 1, 3], 2)) == pytest.approx(1.4)
    # the loop reports exactly these two figures for a layer whose tokens realise n
    E, d = 4, 4
    import torch
    W = torch.eye(E, d).to(torch.bfloat16)                      # logit e = x[e]
    rows = [e for e, c in enumerate(n) for _ in range(c)]
    h = torch.zeros(len(rows), d)
    h[torch.arange(len(rows)), torch.tensor(rows)] = 1.0        # token picks expert rows[i]
    hb = bits(h.to(torch.bfloat16))
    gate = O.Gate(E=E, k=1, gate=0, n_group=1, topk_group=1, renorm=1, route_scale=1.0)
    bud = O.Budget(max_swaps=1, global_ns=2**64 - 1, rank_ns=2**64 - 1, link_ns=2**64 - 1, tau_tokens=0,
                   gamma_num=0, gamma_den=1, alpha_ns=(0, 0), fs_per_byte=(0, 0), ranks_per_node=0, expert_bytes=0)
    trace = [(0, 0, hb, hb, bits(W), None, None), (1, 0, hb, hb, bits(W), None, None)]
    records, summary, _ = O.serving_loop(trace, gate, 2, bud)
    r0, r1 = records
    assert r0["realized"].tolist() == n and r0["hit_rate"] == 1.0
    assert r0["real_vanilla"] == pytest.approx(1.6) and r0["real_before"] == pytest.approx(1.6)
    # one swap with gamma = 0 minimises the maximum load: (6+1, 2+1) = (7, 3) is the best reachable
    assert len(r0["swaps"]) == 1 and r0["real_after"] == pytest.approx(1.4) and r0["improved"]
    # step 1 starts from the committed placement: its "before" is step 0's "after", vanilla stays 1.6
    assert r1["pi_old"] == r0["pi_new"]
    assert r1["real_before"] == pytest.approx(1.4) and r1["real_vanilla"] == pytest.approx(1.6)
    assert r0["cos_hidden"] == pytest.approx(1.0) and r0["cos_logits"] == pytest.approx(1.0)
    assert summary["real_max_over_mean_vanilla"] == pytest.approx(1.6)


def test_empty_budget_never_moves_anything():
    wl = I.WORKLOADS["tiny"]
    T = 200
    records, summary, placements = O.serving_loop(_trace(wl, 2, (0,), T), _gate(wl), wl.R,
                                                  _budget(wl, T, max_swaps=0))
    assert all(r["swaps"] == [] and r["pi_new"] == list(range(wl.E)) for r in records)
    assert summary["layers_with_migration"] == 0 and summary["improved_fraction"] is None
    assert all(r["real_before"] == r["real_after"] == r["real_vanilla"] for r in records)


def test_step_layers_change_the_task_but_not_the_router():
    wl = I.WORKLOADS["dsv3"]
    a = I.make_step_layer(wl, 3, 0, T=64)
    b = I.make_step_layer(wl, 3, 1, T=64)
    ref = I.make_layer(wl, 3, 0, T=64)
    import torch
    assert torch.equal(a.W, b.W) and torch.equal(a.W, ref.W) and torch.equal(a.select_bias, ref.select_bias)
    assert not torch.equal(a.h_prev, b.h_prev)
    # relative drift of the normal router input: rho without the systematic part, larger with it
    def rel(li):
        hf, Hf = li.h_prev.float(), li.H.float()
        return float(((Hf - hf).norm(dim=1) / hf.norm(dim=1)).mean())
    assert rel(a) == pytest.approx(wl.rho, abs=0.01)
    # the systematic part moves the mean logit of expert e by about sys_drift * o_e
    c = I.make_step_layer(wl, 3, 0, T=64, sys_drift=0.5)
    o = I._zipf_log_weights(wl.E, max(wl.zipf_s, 1.0), I._gen(0, 3, 9)).numpy()
    shift = ((c.H.float() - a.H.float()) @ a.W.float().T).mean(dim=0).numpy()
    assert np.corrcoef(shift, 0.5 * o)[0, 1] > 0.95
    assert np.abs(shift - 0.5 * o).max() < 0.25          # cross-talk between router rows and bf16 rounding
