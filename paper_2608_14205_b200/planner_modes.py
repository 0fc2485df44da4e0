"""The planner's three candidate walks side by side on one workload.

Runs the early router pass once per layer (fb_predict_load), then fb_plan_swaps on the same
counts in each mode - Algorithm 1's loop on the narrow frontier, the one-pass sorted sweep of
the ordering paragraph, the loop with a widened frontier - and prints the predicted max / mean
rank load before and after, the number of swaps, and the realised max / mean under each new
placement (counts of the normal pass on H).

    python -m paper_2608_14205_b200.planner_modes [--workload dsv3] [--layers 4] [--tokens T]
"""
from __future__ import annotations

import argparse
import json
import sys

import torch


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="dsv3")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--tokens", type=int, default=0)
    ap.add_argument("--width", type=int, default=2)
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    from . import binding as B
    from . import inputs as I

    wl = I.WORKLOADS[args.workload]
    T = args.tokens or wl.T
    dev = torch.device("cuda", 0)
    ctx = B.Context(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    base = dict(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
                link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
                alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
                ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)
    modes = [("loop", dict(mode=B.FB_PLAN_LOOP)), ("sweep", dict(mode=B.FB_PLAN_SWEEP)),
             (f"wide{args.width}", dict(mode=B.FB_PLAN_WIDE, frontier_width=args.width))]
    i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=dev)
    mom = lambda L: max(L) * len(L) / sum(L) if sum(L) else 1.0
    rows = {name: dict(pred_before=[], pred_after=[], real_after=[], real_before=[], swaps=[]) for name, _ in modes}
    for layer in range(args.layers):
        li = I.make_layer(wl, layer, 0, T=T)
        W = li.W.to(dev)
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        router = B.make_router(W, None, sb)
        pi = li.expert_to_slot.to(dev)
        counts, real = i32(wl.E), i32(wl.E)
        ctx.fb_predict_load(router, li.h_prev.to(dev), T, counts)
        ctx.fb_predict_load(router, li.H.to(dev), T, real)          # what the normal pass will route
        for name, kw in modes:
            bud = B.make_budget(**dict(base, **kw))
            pi_out, swaps, n, lb, la = i32(wl.E), i32(4 * max(1, base["max_swaps"])), i32(1), i32(wl.R), i32(wl.R)
            ctx.fb_plan_swaps(counts, pi, bud, layer, pi_out, swaps, n, lb, la)
            # realised loads under the old and the new placement: the planner with an empty budget
            none = B.make_budget(**dict(base, max_swaps=0))
            rb, ra, dummy = i32(wl.R), i32(wl.R), i32(wl.R)
            ctx.fb_plan_swaps(real, pi, none, layer, i32(wl.E), None, i32(1), rb, dummy)
            ctx.fb_plan_swaps(real, pi_out, none, layer, i32(wl.E), None, i32(1), ra, dummy)
            torch.cuda.synchronize()
            r = rows[name]
            r["pred_before"].append(mom(lb.tolist())); r["pred_after"].append(mom(la.tolist()))
            r["real_before"].append(mom(rb.tolist())); r["real_after"].append(mom(ra.tolist()))
            r["swaps"].append(int(n.item()))
    assert ctx.fb_device_status() == 0
    mean = lambda xs: sum(xs) / len(xs)
    print(f"{wl.name} T={T}, {args.layers} layers: max / mean rank load (mean over layers)")
    print(f"{'mode':8s} {'swaps':>6s} {'predicted before':>17s} {'after':>7s} {'realised before':>16s} {'after':>7s} "
          f"{'layers improved':>16s}")
    out = {}
    for name, _ in modes:
        r = rows[name]
        improved = sum(1 for a, b in zip(r["real_after"], r["real_before"]) if a < b) / len(r["swaps"])
        out[name] = dict(swaps=mean(r["swaps"]), pred_before=mean(r["pred_before"]), pred_after=mean(r["pred_after"]),
                         real_before=mean(r["real_before"]), real_after=mean(r["real_after"]), improved=improved)
        o = out[name]
        print(f"{name:8s} {o['swaps']:6.2f} {o['pred_before']:17.3f} {o['pred_after']:7.3f} {o['real_before']:16.3f} "
              f"{o['real_after']:7.3f} {improved:16.2f}")
    if args.json:
        with open(args.json, "w") as f:
            json.dump(out, f, indent=1)
    ctx.close()


if __name__ == "__main__":
    sys.exit(main())
