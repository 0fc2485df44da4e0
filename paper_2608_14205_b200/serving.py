"""Multi-step serving loop over the C-ABI library: the placement of every MoE layer is
carried from one prefill step to the next (a committed swap plan stays in force until a
later plan changes it), as in the paper's changing-task serving experiment.

This module only owns buffers and passes pointers: prediction, planning, routing, the
dispatch index and the quality metrics all run in the library's kernels.  The normal mode
makes one `fb_layer_step` call per layer; with ``quality=True`` it makes the three separate
calls instead, with logit dumps, and evaluates the paper's prediction-quality metrics
(hidden-state and logit cosine similarity, top-k hit rate) on the device.

    python -m paper_2608_14205_b200.serving --workload dsv3 --steps 4 --layers 2

prints one JSON report per run (synthetic changing-task steps, see inputs.make_step_layer).
"""
from __future__ import annotations

import argparse
import json
from typing import Dict, Optional

import torch

from . import binding as B
from . import inputs as I


def make_budget_for(wl: I.Workload, T: int, **override) -> B.FbBudget:
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    kw = dict(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
              link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
              alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
              ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)
    kw.update(override)
    return B.make_budget(**kw)


class ServingLoop:
    """Per-layer placement state plus the output buffers of one layer step."""

    def __init__(self, wl: I.Workload, T_max: int, device: int = 0):
        self.wl, self.T_max = wl, T_max
        self.dev = torch.device("cuda", device)
        self.ctx = B.Context(T_max, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm,
                             wl.route_scale, device=device)
        E, R, k = wl.E, wl.R, wl.k
        i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=self.dev)
        ms = max(1, min(wl.max_swaps, E // 2))
        self.out = dict(counts=i32(E), swaps=i32(4 * max(ms, E // 2)), n_swaps=i32(1), load_before=i32(R),
                        load_after=i32(R), ids=i32(T_max * k), w=torch.zeros(max(1, T_max * k), device=self.dev),
                        slot_offsets=i32(E + 1), rank_offsets=i32(R + 1), perm=i32(T_max * k),
                        inv_perm=i32(T_max * k), rank_load=i32(R))
        self.placement: Dict[int, torch.Tensor] = {}      # layer -> expert_to_slot in force
        self._spare = i32(E)                              # receives the next placement
        self._q: Optional[dict] = None                    # quality-mode buffers, allocated on first use

    def close(self):
        self.ctx.close()

    def placement_of(self, layer: int) -> torch.Tensor:
        if layer not in self.placement:
            self.placement[layer] = torch.arange(self.wl.E, dtype=torch.int32, device=self.dev)
        return self.placement[layer]

    def _quality_buffers(self):
        if self._q is None:
            T, E, k = self.T_max, self.wl.E, self.wl.k
            f64 = lambda n: torch.zeros(max(1, n), dtype=torch.float64, device=self.dev)
            self._q = dict(z_early=torch.zeros(max(1, T * E), device=self.dev),
                           z=torch.zeros(max(1, T * E), device=self.dev),
                           ids_early=torch.zeros(max(1, T * k), dtype=torch.int32, device=self.dev),
                           rows=f64(T), cos_hidden=f64(1), cos_logits=f64(1),
                           hits=torch.zeros(1, dtype=torch.int32, device=self.dev))
        return self._q

    def layer_step(self, layer: int, router: B.FbRouter, h_prev: torch.Tensor, H: torch.Tensor,
                   budget: B.FbBudget, quality: bool = False) -> dict:
        """Run one layer of one prefill step; commits the new placement for ``layer``.

        Returns the output buffers (device tensors, overwritten by the next call) and, with
        ``quality=True``, the metrics as Python floats."""
        T, o, ctx = h_prev.shape[0], self.out, self.ctx
        pi, pi_new = self.placement_of(layer), self._spare
        report = {}
        if not quality:
            ctx.fb_layer_step(router, h_prev, H, T, pi, budget, layer, o["counts"], pi_new, o["swaps"], o["n_swaps"],
                              o["load_before"], o["load_after"], o["ids"], o["w"], o["slot_offsets"],
                              o["rank_offsets"], o["perm"], o["inv_perm"], o["rank_load"])
        else:
            q = self._quality_buffers()
            E, k = self.wl.E, self.wl.k
            ctx.fb_predict_load(router, h_prev, T, o["counts"], q["ids_early"], q["z_early"])
            ctx.fb_plan_swaps(o["counts"], pi, budget, layer, pi_new, o["swaps"], o["n_swaps"], o["load_before"],
                              o["load_after"])
            ctx.fb_route_dispatch(router, H, T, pi_new, o["ids"], o["w"], o["slot_offsets"], o["rank_offsets"],
                                  o["perm"], o["inv_perm"], o["rank_load"], q["z"])
            B.fb_row_cosine_mean(h_prev, H, q["rows"], q["cos_hidden"])
            B.fb_row_cosine_mean(q["z_early"][:T * E].view(T, E), q["z"][:T * E].view(T, E), q["rows"],
                                 q["cos_logits"])
            B.fb_topk_hits(q["ids_early"], o["ids"], T, k, q["hits"])
            report = dict(cos_hidden=float(q["cos_hidden"].item()), cos_logits=float(q["cos_logits"].item()),
                          hit_rate=(int(q["hits"].item()) & 0xFFFFFFFF) / (T * k) if T * k else 1.0)
        # the plan is committed: the buffer that held the old placement receives the next one
        self.placement[layer], self._spare = pi_new, pi
        return dict(out=o, pi_old=pi, pi_new=pi_new, **report)

    def realised_loads(self, r: dict, budget: B.FbBudget):
        """Realised per-expert counts of the last layer step and the rank loads they give under the
        old, the new and the identity placement - all from the library: per-slot counts of the
        dispatch index, `rank_load` of the step, and the planner's own rank-load aggregation
        (fb_plan_swaps with no swap allowed) for the other two placements."""
        ctx, o, E, R = self.ctx, self.out, self.wl.E, self.wl.R
        i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=self.dev)
        slot_counts, before, vanilla, scratch = i32(E), i32(R), i32(R), i32(R)
        ctx.fb_dispatch_slot_counts(o["slot_offsets"], slot_counts)
        realised = slot_counts[r["pi_new"].long()].contiguous()          # per expert: the count of its slot
        none = type(budget).from_buffer_copy(budget)     # same fields (and the same table pointer, kept alive by `budget`)
        none.max_swaps = 0
        identity = torch.arange(E, dtype=torch.int32, device=self.dev)
        ctx.fb_plan_swaps(realised, r["pi_old"], none, 0, i32(E), None, i32(1), before, scratch)
        ctx.fb_plan_swaps(realised, identity, none, 0, i32(E), None, i32(1), vanilla, scratch)
        torch.cuda.synchronize(self.dev)
        return (realised.cpu().tolist(), before.cpu().tolist(), o["rank_load"].cpu().tolist(),
                vanilla.cpu().tolist())


def max_over_mean(loads) -> float:
    """Report formatting: the imbalance ratio of a rank-load vector the library returned."""
    L = [int(v) for v in loads]
    s = sum(L)
    return max(L) * len(L) / s if s else 1.0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="dsv3", choices=sorted(I.WORKLOADS))
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--tokens", type=int, default=0, help="0 = the workload's batch size")
    ap.add_argument("--sys-drift", type=float, default=0.25,
                    help="systematic logit shift between the two router inputs, see inputs.make_step_layer")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    wl = I.WORKLOADS[args.workload]
    T = args.tokens or wl.T
    loop = ServingLoop(wl, T)
    budget = make_budget_for(wl, T)
    recs = []
    for s in range(args.steps):
        for l in range(args.layers):
            li = I.make_step_layer(wl, l, s, args.seed, T=T, sys_drift=args.sys_drift)
            dev = loop.dev
            sb = li.select_bias.to(dev) if li.select_bias is not None else None
            router = B.make_router(li.W.to(dev), None, sb)
            r = loop.layer_step(l, router, li.h_prev.to(dev), li.H.to(dev), budget, quality=True)
            torch.cuda.synchronize(dev)
            _, before, after, vanilla = loop.realised_loads(r, budget)
            recs.append(dict(step=s, layer=l, n_swaps=int(r["out"]["n_swaps"].item()), hit_rate=r["hit_rate"],
                             cos_hidden=r["cos_hidden"], cos_logits=r["cos_logits"],
                             real_vanilla=max_over_mean(vanilla), real_before=max_over_mean(before),
                             real_after=max_over_mean(after)))
    moved = [r for r in recs if r["n_swaps"] > 0]
    n = max(1, len(recs))
    print(json.dumps(dict(
        workload=wl.name, T=T, steps=args.steps, layers=args.layers, sys_drift=args.sys_drift,
        hit_rate=sum(r["hit_rate"] for r in recs) / n, cos_hidden=sum(r["cos_hidden"] for r in recs) / n,
        cos_logits=sum(r["cos_logits"] for r in recs) / n, swaps_per_layer=sum(r["n_swaps"] for r in recs) / n,
        max_over_mean_vanilla=max(r["real_vanilla"] for r in recs),
        max_over_mean_balanced=max(r["real_after"] for r in recs),
        improved_fraction=(sum(1 for r in moved if r["real_after"] < r["real_before"]) / len(moved)) if moved else None,
        device_status=loop.ctx.fb_device_status(), records=recs)))
    loop.close()


if __name__ == "__main__":
    main()
