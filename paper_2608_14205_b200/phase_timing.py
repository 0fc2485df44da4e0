"""Where the time of one fb_predict_and_plan launch goes, phase by phase.

Builds the library once more with -DFB_TIMING (libfreebalance_timing.so, beside the normal
one), in which one thread per role of every block of the one-tile router kernel writes the
global nanosecond timer and the SM cycle counter at its phase boundaries, runs the call on the
seeded inputs of a workload and prints, in microseconds since the first block's start:
the mean and the latest block per phase boundary, the span of the kernel (first start to last
exit), how far apart the blocks start and finish, the gap to the next launch, and the SM clock
each phase ran at (cycles per nanosecond).  The stamps cost a few stores per block.

    python -m paper_2608_14205_b200.phase_timing [--workload dsv3] [--tokens T] [--launches 12]
        [--call predict_and_plan|predict_load] [--json out.json]
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

SLOTS = {0: "block start", 1: "set-up done", 14: "first load issued", 16: "first operands landed",
         15: "last load issued", 17: "last MMA issued", 2: "accumulators complete", 3: "keys computed",
         4: "barrier", 5: "groups chosen", 7: "candidates collected", 8: "candidates ranked", 9: "top-k read back",
         10: "outputs written", 11: "counts published", 18: "planner entered", 19: "rank loads formed",
         20: "greedy loop left", 12: "planner done", 13: "block exit"}
ORDER = [0, 1, 14, 16, 15, 17, 2, 3, 4, 5, 7, 8, 9, 10, 11, 18, 19, 20, 12, 13]


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="dsv3")
    ap.add_argument("--tokens", type=int, default=0)
    ap.add_argument("--launches", type=int, default=12)
    ap.add_argument("--call", default="predict_and_plan", choices=["predict_and_plan", "predict_load"])
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)

    from . import build as fb_build
    fb_build.use_library(fb_build.build_variant("timing", ["-DFB_TIMING"]))
    from . import binding as B
    from . import inputs as I

    wl = I.WORKLOADS[args.workload]
    T = args.tokens or wl.T
    dev = torch.device("cuda", 0)
    layers = [I.make_layer(wl, l, 0, T=T) for l in range(2)]
    L = []
    for li in layers:
        W = li.W.to(dev)
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        L.append(dict(W=W, sb=sb, router=B.make_router(W, None, sb), x=li.h_prev.to(dev), pi=li.expert_to_slot.to(dev)))
    ctx = B.Context(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    budget = B.make_budget(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
                           link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
                           alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
                           ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)
    i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=dev)
    counts, pio, sw, ns, lb, la = i32(wl.E), i32(wl.E), i32(4 * 128), i32(1), i32(wl.R), i32(wl.R)
    blocks_max = 2 * ((T + 127) // 128 + 1) + 64
    n = args.launches
    stamps = torch.zeros((n, blocks_max, 64), dtype=torch.int64, device=dev)

    def call(i):
        d = L[i % 2]
        if args.call == "predict_and_plan":
            ctx.fb_predict_and_plan(d["router"], d["x"], T, d["pi"], budget, 0, counts, pio, sw, ns, lb, la)
        else:
            ctx.fb_predict_load(d["router"], d["x"], T, counts)

    for i in range(4):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):                       # back to back, each launch into its own stamp table
        ctx.fb_set_stamp_buffer(stamps[i])
        call(i)
    e1.record()
    torch.cuda.synchronize()
    ctx.fb_set_stamp_buffer(None)
    per_launch_us = e0.elapsed_time(e1) * 1e3 / n
    st = stamps.cpu().numpy()
    used = st[:, :, 0] != 0                                  # blocks that ran
    nblk = int(used[0].sum())
    st = st[:, :nblk, :]
    ns_t = st[:, :, :32].astype(np.float64)
    cyc = st[:, :, 32:].astype(np.float64)
    rows = []
    out = {"workload": wl.name, "T": T, "call": args.call, "launches": n, "blocks": nblk,
           "per_launch_us_events": per_launch_us, "phases": {}}
    start = ns_t[:, :, 0].min(axis=1, keepdims=True)         # first block start of each launch
    print(f"{args.call} on {wl.name} T={T}: {nblk} blocks, {per_launch_us:.1f} us per launch "
          f"(two events around {n} back-to-back launches)")
    print(f"{'phase boundary':26s} {'mean':>8s} {'latest':>8s}   (us since the launch's first block start; "
          f"launches 2..{n})")
    sel = slice(1, None)
    for slot in ORDER:
        t = ns_t[sel, :, slot]
        ok = t > 0
        if not ok.any():
            continue
        rel = np.where(ok, (t - start[sel]) / 1e3, np.nan)
        mean, latest = float(np.nanmean(rel)), float(np.nanmean(np.nanmax(rel, axis=1)))
        out["phases"][SLOTS[slot]] = {"mean_us": mean, "latest_us": latest, "blocks": int(ok[0].sum())}
        print(f"{SLOTS[slot]:26s} {mean:8.2f} {latest:8.2f}   [{int(ok[0].sum())} blocks]")
    end = ns_t[:, :, 13].max(axis=1)
    span = (end - start[:, 0]) / 1e3
    gap = (start[1:, 0] - end[:-1]) / 1e3
    skew_start = (ns_t[:, :, 0].max(axis=1) - start[:, 0]) / 1e3
    ends = ns_t[:, :, 13]
    skew_end = (end - np.where(ends > 0, ends, np.inf).min(axis=1)) / 1e3
    own = (ns_t[sel, :, 2] > 0) & (ns_t[sel, :, 11] > 0)          # blocks that own a tile (helper pairs have no epilogue)
    main_cyc = (cyc[sel, :, 2] - cyc[sel, :, 1])[own]
    main_ns = (ns_t[sel, :, 2] - ns_t[sel, :, 1])[own]
    epi_cyc = (cyc[sel, :, 11] - cyc[sel, :, 2])[own]
    epi_ns = (ns_t[sel, :, 11] - ns_t[sel, :, 2])[own]
    out.update(span_us=float(span[sel].mean()), gap_us=float(gap.mean()), start_skew_us=float(skew_start[sel].mean()),
               end_skew_us=float(skew_end[sel].mean()), main_loop_ghz=float(main_cyc.mean() / main_ns.mean()),
               epilogue_ghz=float(epi_cyc.mean() / epi_ns.mean()), main_loop_cycles=float(main_cyc.mean()))
    print(f"kernel span (first start .. last exit) {out['span_us']:.2f} us; gap to the next launch's first block "
          f"{out['gap_us']:.2f} us; blocks start within {out['start_skew_us']:.2f} us and exit within "
          f"{out['end_skew_us']:.2f} us")
    print(f"SM clock: main loop {out['main_loop_ghz']:.3f} GHz ({out['main_loop_cycles']:.0f} cycles), "
          f"epilogue {out['epilogue_ghz']:.3f} GHz")
    if args.json:
        with open(args.json, "w") as f:
            json.dump(out, f, indent=1)
    ctx.close()


if __name__ == "__main__":
    sys.exit(main())
