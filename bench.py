#!/usr/bin/env python
"""Benchmark of the FreeBalance per-layer hot path on B200.

One "step" = the whole hot path for one MoE layer on one prefill batch, through
fb_layer_step: the early router pass on h_{l-1} (gating, top-k, histogram, rank loads,
swap planner) and the normal router pass on H_l (top-k ids, routing weights) in ONE
kernel launch, then the dispatch index under the new placement in a second launch.
`--api separate` times the same work as fb_predict_and_plan + fb_route_dispatch (three
launches).  The metric is tokens per second through that path, per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload dsv3] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica on its own GPU - the path has no exchange step - and the time is the
maximum over ranks.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_14205_b200 import inputs as I  # noqa: E402

METRIC = "predicted-routing tokens/sec per layer"
UNIT = "tokens/s"
L2_BYTES = 126 * 2**20


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def budget_kwargs(wl: I.Workload, T: int):
    gn, gd = I.default_gamma(T, wl.k, wl.R)
    return dict(max_swaps=min(wl.max_swaps, wl.E // 2), global_ns=wl.global_ns, rank_ns=wl.rank_ns,
                link_ns=wl.link_ns, tau_tokens=0, gamma_num=gn, gamma_den=gd,
                alpha_ns=(wl.alpha_ns, wl.alpha_ns), fs_per_byte=(wl.fs_per_byte, wl.fs_per_byte),
                ranks_per_node=wl.ranks_per_node, expert_bytes=wl.expert_bytes)


def _clock_sampler_main(index, period_s, go, stop, times, mhz, reasons, count, max_mhz):
    """Body of the sampler process: polls NVML (read-only) as fast as `period_s` allows."""
    try:
        import pynvml as nv
        nv.nvmlInit()
        h = nv.nvmlDeviceGetHandleByIndex(index)
        max_mhz.value = int(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
    except Exception:
        max_mhz.value = -1
        return
    go.wait()
    n, cap = 0, len(times)
    while not stop.is_set() and n < cap:
        try:
            mhz[n] = int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
            reasons[n] = int(get_reasons(h)) if get_reasons is not None else 0
            times[n] = time.perf_counter()
            n += 1
            count.value = n
        except Exception:
            pass
        if period_s > 0:
            time.sleep(period_s)


class ClockSampler:
    """SM clock and throttle reasons through NVML (read-only) while the timed region runs.

    The polling loop lives in a process of its own: a thread of this process would share the
    interpreter lock with the loop that launches the kernels and get a sample every few
    milliseconds at best.  Samples carry host time stamps (the same monotonic clock in both
    processes); the caller marks the timed region with `window`."""
    REASONS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int, period_s: float = 0.0001, capacity: int = 200000):
        import multiprocessing as mp
        ctx = mp.get_context("spawn")
        self.window = [None, None]           # host times that bracket the timed region
        self._go, self._stop = ctx.Event(), ctx.Event()
        self._times = ctx.Array("d", capacity, lock=False)
        self._mhz = ctx.Array("i", capacity, lock=False)
        self._reasons = ctx.Array("q", capacity, lock=False)
        self._count = ctx.Value("i", 0, lock=False)
        self._max = ctx.Value("i", 0, lock=False)
        self._proc = ctx.Process(target=_clock_sampler_main, daemon=True,
                                 args=(index, period_s, self._go, self._stop, self._times, self._mhz, self._reasons,
                                       self._count, self._max))
        try:
            self._proc.start()
        except Exception:
            self._proc = None

    def start(self):
        self._go.set()

    def stop(self):
        self._stop.set()
        self._go.set()
        if self._proc is not None:
            self._proc.join(timeout=5)
        n = int(self._count.value)
        t0, t1 = self.window
        idx = [i for i in range(n) if t0 is not None and t1 is not None and t0 <= self._times[i] <= t1]
        use = idx if len(idx) >= 3 else list(range(n))
        mhz = [self._mhz[i] for i in use]
        bits = 0
        for i in use:
            bits |= int(self._reasons[i])
        return {"sm_mhz": statistics.median(mhz) if mhz else None,
                "sm_max_mhz": int(self._max.value) if self._max.value > 0 else None,
                "reasons": sorted(name for name, bit in self.REASONS.items() if bits & bit),
                "samples": len(use), "samples_in_timed_region": len(idx), "samples_total": n,
                "sm_mhz_min": min(mhz) if mhz else None}


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time decides: MAX all-reduce (identity when not distributed)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(world: int, tokens_per_step: int, steps: int, total_ms: float) -> float:
    """Replicas process world * tokens per step; the job takes the slowest rank's time."""
    return world * tokens_per_step * steps / (total_ms * 1e-3)


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def oracle_layer_seconds(wl, layer, bkw, steps, warmup):
    """Time the CPU oracle, as it stands, on whole layers of the workload."""
    import numpy as np
    from oracle import freebalance_oracle as O
    def bits(t): return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    gate = O.Gate(E=wl.E, k=wl.k, gate=wl.gate, n_group=wl.n_group, topk_group=wl.topk_group,
                  renorm=wl.renorm, route_scale=wl.route_scale)
    bud = O.Budget(**bkw)
    args = (bits(layer.h_prev), bits(layer.H), bits(layer.W), gate, wl.R, layer.expert_to_slot.tolist(), bud,
            None if layer.select_bias is None else layer.select_bias.numpy(),
            None if layer.logit_bias is None else layer.logit_bias.numpy())
    for _ in range(warmup):
        O.layer_step(*args)
    t0 = time.perf_counter()
    for _ in range(steps):
        O.layer_step(*args)
    return (time.perf_counter() - t0) / max(1, steps)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, wl, rank):
    if rank != 0:
        return
    # one whole layer of the workload per step is a few seconds of CPU work for the
    # 16k-token shape; longer shapes are cut to 16k tokens to keep the run bounded
    T_s = min(wl.T, 16384)
    layer = I.make_layer(wl, 0, 0, T=T_s)
    bkw = budget_kwargs(wl, T_s)
    steps = max(1, min(args.steps, 5))
    warmup = min(args.warmup, 1)
    sec = oracle_layer_seconds(wl, layer, bkw, steps, warmup)
    value = T_s / sec
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "T": T_s, "d": wl.d, "E": wl.E, "k": wl.k, "R": wl.R},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{steps} whole layer(s) of {T_s} tokens, full chain"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_overlap(wl, B, dev, window_us, reps=10, pair_limits=(8, 16, 24, 32, 48), T=None, expert_bytes=None,
                n_sm=None):
    """The method's two-stream schedule on one GPU ("Overlap Analysis"): the target layer's
    attention on one stream, and on a side stream the work it is meant to hide - early router
    pass + planner (fb_predict_and_plan), then the weight exchange of the accepted swaps
    (fb_apply_swaps, or the host-issued copies of fb_apply_swaps_staged).

    Attention is a compute-bound stand-in (fb_standin_attention) on n_sm - 2 p SMs; the router
    kernel is confined to the other p SM pairs (fb_set_pair_limit).  The window B of Eq. 10 comes
    from the library's own attention profile (fb_attention_begin / _end around the stand-in,
    fb_layer_budget_ns with a 10 % margin) and is what the planner's time budgets are set to.
    For every p: attention alone, auxiliary work alone, both together, exposed = together -
    attention alone, and whether the auxiliary work fitted into the window."""
    T = T or wl.T
    E, R, k = wl.E, wl.R, wl.k
    n_sm = n_sm or torch.cuda.get_device_properties(dev).multi_processor_count
    S = ((expert_bytes if expert_bytes is not None else wl.expert_bytes) or 16 * 2**20) // 16 * 16
    li = I.make_layer(wl, 0, 0, T=T)
    ctx = B.Context(T, wl.d, E, k, R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale,
                    device=dev.index or 0)
    sb = li.select_bias.to(dev) if li.select_bias is not None else None
    W = li.W.to(dev)
    router = B.make_router(W, None, sb)
    h_prev, pi = li.h_prev.to(dev), li.expert_to_slot.to(dev)
    i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=dev)
    cap = max(1, min(wl.max_swaps, E // 2))
    counts, pi_out, swaps, n_swaps, lb, la = i32(E), i32(E), i32(4 * cap), i32(1), i32(R), i32(R)
    weights = torch.empty(E * S, dtype=torch.uint8, device=dev)          # content is irrelevant for timing
    sink = torch.zeros(1024 * 1024, device=dev)
    side = torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream(dev)

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize(dev)
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize(dev)
            ts.append(a.elapsed_time(b) * 1e3)
        return statistics.median(ts)

    # stand-in length: iterations per microsecond from two probes
    t1 = timed(lambda: B.fb_standin_attention(sink, n_sm, 2000))
    t2 = timed(lambda: B.fb_standin_attention(sink, n_sm, 12000))
    iters = max(1, int(2000 + (window_us - t1) * 10000 / max(t2 - t1, 1e-3)))
    rows = []
    for p_lim in pair_limits:
        if 2 * p_lim >= n_sm:
            continue
        blocks = n_sm - 2 * p_lim
        ctx.fb_set_pair_limit(p_lim)
        attention = lambda: B.fb_standin_attention(sink, blocks, iters)
        # the window of Eq. 10 from the library's attention profile, 10 % margin
        ctx.fb_attention_reset()
        attention()
        ctx.fb_attention_begin(0, 0)
        attention()
        ctx.fb_attention_end(0, 0)
        window_ns, _ = ctx.fb_layer_budget_ns(0, 0)
        budget_ns, _ = ctx.fb_layer_budget_ns(0, window_ns // 10)
        bkw = budget_kwargs(wl, T)
        bkw.update(max_swaps=cap)
        if wl.global_ns != 2**64 - 1:                         # workloads with a time budget take the measured one
            bkw.update(global_ns=budget_ns, rank_ns=budget_ns, link_ns=budget_ns)
        budget = B.make_budget(**bkw)

        def predict_plan(stream=None):
            ctx.fb_predict_and_plan(router, h_prev, T, pi, budget, 0, counts, pi_out, swaps, n_swaps, lb, la,
                                    stream=stream)

        def aux_kernel(stream=None):
            predict_plan(stream)
            B.fb_apply_swaps(weights, S, E, pi, swaps, n_swaps, cap, stream=stream)

        def aux_copies(stream=None):
            predict_plan(stream)
            ctx.fb_apply_swaps_staged(weights, S, pi, swaps, n_swaps, cap, 0, plan_stream=stream, copy_stream=stream)

        def beside(work):
            def run():
                side.wait_stream(main)
                attention()                                   # main stream
                work(side)                                    # side stream, started at the same time
                main.wait_stream(side)
            return run

        row = dict(router_pairs=p_lim, attention_sms=blocks, window_us=window_ns / 1e3, budget_us=budget_ns / 1e3,
                   attention_us=timed(attention), predict_plan_us=timed(predict_plan))
        for name, work in (("exchange_kernel", aux_kernel), ("exchange_copies", aux_copies)):
            alone, both = timed(work), timed(beside(work))
            row[name] = dict(auxiliary_alone_us=alone, together_us=both,
                             exposed_us=max(0.0, both - row["attention_us"]),
                             hidden_fraction=1.0 - max(0.0, both - row["attention_us"]) / alone if alone > 0 else None,
                             fits_window=both <= row["attention_us"] * 1.05)
        row["swaps"] = int(n_swaps.item())
        row["exchange_bytes"] = 4 * S * row["swaps"]
        rows.append(row)
    ctx.fb_set_pair_limit(0)
    status = ctx.fb_device_status()
    ctx.close()
    return {"experiment": "two-stream overlap on one GPU", "workload": wl.name, "T": T, "expert_bytes": S,
            "stand_in": f"fb_standin_attention, {iters} iterations, one block per SM", "sms": n_sm,
            "device_status": status, "rows": rows}


def run_sharded(args, wl, B, dist, dev, rank, local_rank, world, sampler):
    """Strong-scaling leg: one batch of wl.T tokens split over the ranks.  Per step and rank: early
    pass on the local tokens, all-reduce of the E counts, planner, normal pass + local dispatch
    index, all-gather of the E slot counts, whole-batch positions (sharded.ShardedPredictor)."""
    from paper_2608_14205_b200.sharded import ShardedPredictor, shard_bounds
    T, E, R, k, d = wl.T, wl.E, wl.R, wl.k, wl.d
    lo, hi = shard_bounds(T, world, rank)
    Tl = hi - lo
    bkw = budget_kwargs(wl, T)                                  # gamma from the whole batch, same on every rank
    budget = B.make_budget(**bkw)
    ctx = B.Context(max(Tl, 1), d, E, k, R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale,
                    device=local_rank)
    ring = max(1, args.ring)
    layers = []
    for l in range(ring):
        li = I.make_layer(wl, layer=l, seed=0)                  # the same batch on every rank; each keeps its shard
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        W = li.W.to(dev)
        layers.append(dict(W=W, sb=sb, router=B.make_router(W, None, sb), h_prev=li.h_prev[lo:hi].contiguous().to(dev),
                           H=li.H[lo:hi].contiguous().to(dev), pi=li.expert_to_slot.to(dev)))
    i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=dev)
    out = dict(counts=i32(E), pi_out=i32(E), swaps=i32(4 * max(1, bkw["max_swaps"])), n_swaps=i32(1),
               load_before=i32(R), load_after=i32(R), ids=i32(Tl * k), w=torch.zeros(max(1, Tl * k), device=dev),
               slot_offsets=i32(E + 1), rank_offsets=i32(R + 1), perm=i32(Tl * k), inv_perm=i32(Tl * k),
               rank_load=i32(R))
    counts_all = i32(world * E)
    sp = ShardedPredictor(ctx)

    def step(L):
        sp.layer_step(L["router"], L["h_prev"], L["H"], Tl, L["pi"], budget, 0, out, counts_all)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(args.warmup):
        step(layers[i % ring])
    barrier()
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.fb_launch_count()
    sampler.start()
    sampler.window[0] = time.perf_counter()
    e0.record()
    for i in range(K):
        step(layers[i % ring])
    e1.record()
    barrier()
    sampler.window[1] = time.perf_counter()
    clocks = sampler.stop()
    total_ms = max_over_ranks(e0.elapsed_time(e1), dev)
    launches = ctx.fb_launch_count() - launches0
    status = ctx.fb_device_status()
    if rank == 0:
        mom = lambda L: (max(L) * len(L) / sum(L)) if sum(L) else 1.0
        line = {"metric": METRIC, "value": T * K / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
                "warmup": args.warmup, "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "T": T, "T_per_rank": Tl, "d": d, "E": E, "k": k, "R": R,
                           "api": "sharded.ShardedPredictor.layer_step (fb_predict_load, all-reduce, fb_plan_swaps, "
                                  "fb_route_dispatch, all-gather, fb_dispatch_globalize)",
                           "parallelism": f"token shards x{world}", "layers_in_ring": ring,
                           "l2": "inputs larger than L2" if Tl * d * 2 > L2_BYTES else
                                 "ring of layers; inputs may be L2-resident"},
                "clocks": clocks, "e2e": None, "gpu_launches": int(launches), "device_status": status,
                "collectives_per_step": 0 if world == 1 else 2,
                "load_balance": {"predicted_max_over_mean": [mom(out["load_before"].tolist()),
                                                             mom(out["load_after"].tolist())],
                                 "realized_max_over_mean_after": mom(out["rank_load"].tolist()),
                                 "n_swaps": int(out["n_swaps"].item())}}
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="dsv3", choices=sorted(I.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ring", type=int, default=2, help="distinct layers cycled through")
    ap.add_argument("--api", default="layer", choices=["layer", "separate"],
                    help="layer: fb_layer_step (default); separate: fb_predict_and_plan + fb_route_dispatch")
    ap.add_argument("--sharded", action="store_true",
                    help="strong scaling: the workload's T tokens are split over the ranks (contiguous ranges); "
                         "two small collectives per step (count all-reduce, slot-count all-gather)")
    ap.add_argument("--overlap", action="store_true",
                    help="the two-stream schedule on one GPU: prediction, planning and the weight exchange on a "
                         "side stream beside a stand-in attention; sweeps the SM pairs left to the router kernel")
    ap.add_argument("--window-us", type=float, default=500.0, help="--overlap: length of the stand-in attention")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (for profiler captures)")
    ap.add_argument("--no-probe", action="store_true",
                    help="skip the per-kernel timing passes after the bracketed region and the in-kernel clock "
                         "probe (for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = I.WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, wl, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    from paper_2608_14205_b200 import binding as B

    import torch.distributed as dist
    distributed = world > 1
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if distributed:
        dist.init_process_group("nccl", device_id=dev)

    # the clock sampler's process starts now (it needs a second to load NVML) and waits for start()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    T_global = wl.T
    if args.sharded:
        return run_sharded(args, wl, B, dist, dev, rank, local_rank, world, sampler)
    if args.overlap:
        sampler.stop()
        print(json.dumps(run_overlap(wl, B, dev, args.window_us, reps=max(3, min(args.steps, 10)))), flush=True)
        return
    T, E, R, k, d = wl.T, wl.E, wl.R, wl.k, wl.d
    bkw = budget_kwargs(wl, T)
    budget = B.make_budget(**bkw)
    ctx = B.Context(T, d, E, k, R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale, device=local_rank)

    # ---- inputs: a ring of distinct layers, resident in HBM before the timed region
    ring = max(1, args.ring)
    layers_cpu = [I.make_layer(wl, layer=l, seed=rank) for l in range(ring)]
    layers = []
    for li in layers_cpu:
        W = li.W.to(dev)
        sb = li.select_bias.to(dev) if li.select_bias is not None else None
        layers.append(dict(router=B.make_router(W, None, sb), h_prev=li.h_prev.to(dev), H=li.H.to(dev),
                           pi=li.expert_to_slot.to(dev)))
    i32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32, device=dev)
    out = dict(counts=i32(E), pi_out=i32(E), swaps=i32(4 * max(1, bkw["max_swaps"])), n_swaps=i32(1),
               load_before=i32(R), load_after=i32(R), ids=i32(T * k), w=torch.zeros(max(1, T * k), device=dev),
               slot_offsets=i32(E + 1), rank_offsets=i32(R + 1), perm=i32(T * k), inv_perm=i32(T * k),
               rank_load=i32(R))

    layer_api = args.api == "layer"

    def predict_and_plan(L):
        ctx.fb_predict_and_plan(L["router"], L["h_prev"], T, L["pi"], budget, 0, out["counts"], out["pi_out"],
                                out["swaps"], out["n_swaps"], out["load_before"], out["load_after"])

    def step(L):
        if layer_api:
            ctx.fb_layer_step(L["router"], L["h_prev"], L["H"], T, L["pi"], budget, 0, out["counts"], out["pi_out"],
                              out["swaps"], out["n_swaps"], out["load_before"], out["load_after"], out["ids"],
                              out["w"], out["slot_offsets"], out["rank_offsets"], out["perm"], out["inv_perm"],
                              out["rank_load"])
        else:
            predict_and_plan(L)
            ctx.fb_route_dispatch(L["router"], L["H"], T, out["pi_out"], out["ids"], out["w"], out["slot_offsets"],
                                  out["rank_offsets"], out["perm"], out["inv_perm"], out["rank_load"])

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(args.warmup):
        step(layers[i % ring])
    barrier()
    if ctx.fb_device_status() != 0:
        raise SystemExit("device status non-zero after warm-up")

    # ---- timed region: exactly K steps; two events on the launching (current) stream
    K = args.steps
    ev_begin, ev_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.fb_launch_count()
    persistent0 = ctx.fb_persistent_launch_count()
    # in-kernel clock probe on a side stream: (time, cycle counter) pairs every ~4 us for the
    # expected length of the region (estimated from a few untimed steps), plus one device time
    # stamp on the main stream at each end of the region
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(3):
        step(layers[i % ring])
    e1.record()
    barrier()
    est_region_ns = e0.elapsed_time(e1) / 3 * K * 1e6
    probe_period_ns = 4000
    probe_n = int(min(65536, max(64, 1.5 * est_region_ns / probe_period_ns + 64)))
    probe = torch.zeros(2 * probe_n, dtype=torch.int64, device=dev)
    marks = torch.zeros(4, dtype=torch.int64, device=dev)
    side = torch.cuda.Stream(device=dev)
    barrier()
    sampler.start()
    sampler.window[0] = time.perf_counter()
    if not args.no_probe:                    # (under a profiler the probe kernel would be serialised with the steps)
        B.fb_clock_probe(probe, probe_n, probe_period_ns, stream=side)
        B.fb_clock_probe(marks[0:2], 1, 0)
    ev_begin.record()
    for i in range(K):
        step(layers[i % ring])
    ev_end.record()
    if not args.no_probe:
        B.fb_clock_probe(marks[2:4], 1, 0)
    barrier()
    sampler.window[1] = time.perf_counter()
    launches = ctx.fb_launch_count() - launches0
    persistent_launches = ctx.fb_persistent_launch_count() - persistent0
    total_ms = ev_begin.elapsed_time(ev_end)
    total_ms = max_over_ranks(total_ms, dev)
    status = ctx.fb_device_status()

    # ---- the dominant kernel (the router kernel: the first launch of a step), timed on
    # `n_probe` further steps by a pair of events that the library records directly around that
    # launch.  Kept out of the bracketed region: an event between two launches keeps the GPU from
    # preparing the next launch early and costs about 2 us per record.  The clock sampler keeps
    # running, so short bracketed regions still get enough clock samples.
    n_probe = 0 if args.no_probe else max(16, min(K, 64))
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_probe)]
    for pair in ev:                          # torch creates the CUDA event on its first record
        for e in pair:
            e.record()
    barrier()
    for i in range(n_probe):
        ctx.fb_time_next_router_launch(ev[i][0], ev[i][1])
        step(layers[i % ring])
    barrier()
    router_ms = [a.elapsed_time(b) for a, b in ev]

    # ---- the fused predictor + planner alone (fb_predict_and_plan), the unit the roofline target
    # of the method's prediction stage refers to: (1) launches back to back between two events,
    # repeated, median of the repeats; (2) one event pair per launch
    pp_n = 0 if args.no_probe else 24
    pp_b2b = []
    for _ in range(0 if args.no_probe else 5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(pp_n):
            predict_and_plan(layers[i % ring])
        b.record()
        barrier()
        pp_b2b.append(a.elapsed_time(b) / pp_n)
    # the same launch cut down to its main loop (operands loaded only / loaded and multiplied; nothing after
    # it): what launch, set-up and the operand stream cost by themselves with this tiling
    floor_us = {}
    one_tile_launch = (T + 127) // 128 // 2 <= ctx.fb_max_pairs()       # else the call uses the persistent kernel
    if pp_n and one_tile_launch:
        for what, name in ((1, "loads_only_us"), (2, "loads_and_mma_us")):
            reps = []
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for i in range(pp_n):
                    L = layers[i % ring]
                    ctx.fb_router_floor(L["router"], L["h_prev"], T, what)
                b.record()
                barrier()
                reps.append(a.elapsed_time(b) / pp_n * 1e3)
            floor_us[name] = statistics.median(reps)
    pp_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(pp_n)]
    for i in range(pp_n):
        pp_ev[i][0].record()
        predict_and_plan(layers[i % ring])
        pp_ev[i][1].record()
    barrier()
    pp_ms = [a.elapsed_time(b) for a, b in pp_ev]
    clocks = sampler.stop()
    # SM clock seen from inside a kernel during the bracketed region
    side.synchronize()
    pr = probe.cpu().view(-1, 2).tolist()
    t_lo, t_hi = int(marks[0].item()), int(marks[2].item())
    inside = [(t, c) for t, c in pr if t_lo <= t <= t_hi]
    mhz = []
    stride = max(1, len(inside) // 64)                    # ~64 windows over the region
    for i in range(0, len(inside) - stride, stride):
        dt, dc = inside[i + stride][0] - inside[i][0], inside[i + stride][1] - inside[i][1]
        if dt > 0:
            mhz.append(dc / dt * 1e3)
    clocks["in_kernel"] = {"sm_mhz_median": statistics.median(mhz) if mhz else None,
                           "sm_mhz_min": min(mhz) if mhz else None, "sm_mhz_max": max(mhz) if mhz else None,
                           "windows": len(mhz), "samples_in_timed_region": len(inside),
                           "how": "fb_clock_probe: cycle counter / global timer of a one-thread kernel running "
                                  "beside the timed steps"}

    # ---- realised rank loads before / after the plan of the last timed step, from the library's
    # own outputs: counts of the normal pass (fb_predict_load on H), loads under the old placement
    # (fb_plan_swaps with an empty budget), loads under the new one (rank_load of the step)
    L_last = layers[(K - 1) % ring]
    step(L_last)
    real_counts, real_before, scratch_after = i32(E), i32(R), i32(R)
    ctx.fb_predict_load(L_last["router"], L_last["H"], T, real_counts)
    no_swaps = B.make_budget(**dict(bkw, max_swaps=0))
    ctx.fb_plan_swaps(real_counts, L_last["pi"], no_swaps, 0, i32(E), None, i32(1), real_before, scratch_after)
    barrier()

    # ---- stage 3 on this device (not part of the step): the plan just produced, applied to a buffer
    # of E slot images of the workload's expert size; HBM bound, 4 bytes of traffic per byte moved
    mig = None
    if not args.no_e2e and not args.no_probe and wl.expert_bytes > 0 and bkw["max_swaps"] > 0:
        S = wl.expert_bytes // 16 * 16
        weights = torch.empty(E * S, dtype=torch.uint8, device=dev)      # content does not matter for timing
        cap = int(bkw["max_swaps"])
        L0d = L_last
        run_mig = lambda: B.fb_apply_swaps(weights, S, E, L0d["pi"], out["swaps"], out["n_swaps"], cap)
        for _ in range(3):
            run_mig()
        barrier()
        m_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
        for a, b in m_ev:
            a.record()
            run_mig()
            b.record()
        barrier()
        n_sw = int(out["n_swaps"].item())
        m_us = statistics.mean(a.elapsed_time(b) for a, b in m_ev) * 1e3
        mig = {"kernel": "fb_swap_weights_kernel (fb_apply_swaps)", "swaps": n_sw, "expert_bytes": S,
               "traffic_bytes": 4 * S * n_sw, "us": m_us,
               "achieved_GBps": 4 * S * n_sw / (m_us * 1e-6) / 1e9 if m_us > 0 else None}
        del weights

    # ---- end to end through the host-buffer entry point (copies inside the timed region)
    L0 = layers_cpu[0]
    pin = lambda t: t.contiguous().pin_memory()
    h_prev_h, H_h, pi_h = pin(L0.h_prev), pin(L0.H), pin(L0.expert_to_slot)
    hi32 = lambda n: torch.zeros(max(1, n), dtype=torch.int32).pin_memory()
    hout = dict(counts=hi32(E), expert_to_slot_out=hi32(E), swaps=hi32(4 * max(1, bkw["max_swaps"])),
                n_swaps=hi32(1), load_before=hi32(R), load_after=hi32(R), topk_ids=hi32(T * k),
                topk_w=torch.zeros(max(1, T * k)).pin_memory(), slot_offsets=hi32(E + 1),
                rank_offsets=hi32(R + 1), perm=hi32(T * k), inv_perm=hi32(T * k), rank_load=hi32(R))
    h2d = h_prev_h.numel() * 2 + H_h.numel() * 2 + pi_h.numel() * 4
    d2h = sum(v.numel() * v.element_size() for v in hout.values())
    e2e_steps = 0 if args.no_e2e else max(3, min(K, 20))
    for _ in range(0 if args.no_e2e else 2):
        ctx.fb_layer_step_host(layers[0]["router"], h_prev_h, H_h, T, pi_h, budget, 0, **hout)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        ctx.fb_layer_step_host(layers[0]["router"], h_prev_h, H_h, T, pi_h, budget, 0, **hout)
    e1.record()
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), 1e-9)
    e2e_ms = max_over_ranks(e2e_ms, dev)

    if rank == 0:
        peaks = measured_peaks()
        ms_per_step = total_ms / K
        value = whole_job_throughput(world, T, K, total_ms)
        # Roofline of the dominant kernel: the router kernel of the step.  Algorithmic work per
        # launch: read each input matrix once (2 T d bytes per pass), W once, write the counts and,
        # in the normal pass, ids and weights (8 T k); 2 T d E flops per pass.
        passes = 2 if layer_api else 1
        alg_bytes = passes * 2 * T * d + 2 * d * E + 4 * E + (8 * T * k if layer_api else 0)
        alg_flops = passes * 2 * T * d * E

        def sustained_roof(ms, t_hbm, nflops, tf, gbs):
            # The same bound with the GEMM peak of a seconds-long loop (the driver's sustained figure)
            # in place of the burst figure: the regime these back-to-back launches run in (their
            # in-kernel clock sits near the one that measurement saw).  `frac` above stays on the
            # burst figure and the copy peak.
            t_tensor = nflops / (peaks["bf16_tflops_sustained"] * 1e12)
            hbm = t_hbm >= t_tensor
            return {"bound": "hbm" if hbm else "tensor", "t_roof_us": max(t_hbm, t_tensor) * 1e6,
                    "peak": peaks["hbm_gbs"] if hbm else peaks["bf16_tflops_sustained"],
                    "unit": "GB/s" if hbm else "TFLOP/s",
                    "frac": (gbs / peaks["hbm_gbs"]) if hbm else (tf / peaks["bf16_tflops_sustained"]),
                    "note": "bound recomputed with the sustained bf16 GEMM peak instead of the burst one"}

        def roofline(ms, nbytes, nflops, kernel):
            gbs = nbytes / (ms * 1e-3) / 1e9
            tf = nflops / (ms * 1e-3) / 1e12
            t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
            t_tensor = nflops / (peaks["bf16_tflops"] * 1e12)
            hbm = t_hbm >= t_tensor
            return {"kernel": kernel, "bound": "hbm" if hbm else "tensor", "achieved": gbs if hbm else tf,
                    "peak": peaks["hbm_gbs"] if hbm else peaks["bf16_tflops"], "unit": "GB/s" if hbm else "TFLOP/s",
                    "frac": (gbs / peaks["hbm_gbs"]) if hbm else (tf / peaks["bf16_tflops"]),
                    "peak_source": peaks["source"], "traffic": None, "kernel_us": ms * 1e3,
                    "t_roof_us": max(t_hbm, t_tensor) * 1e6, "algorithmic_bytes": nbytes, "algorithmic_flops": nflops,
                    "tensor_tflops": tf, "tensor_frac_of_burst": tf / peaks["bf16_tflops"],
                    "tensor_frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                    "sustained": sustained_roof(ms, t_hbm, nflops, tf, gbs)}

        def spread(xs):
            xs = sorted(xs)
            return {"min_us": xs[0] * 1e3, "median_us": statistics.median(xs) * 1e3, "max_us": xs[-1] * 1e3,
                    "n": len(xs)}

        def attach_traffic(block, key):
            # DRAM bytes per launch come from an ncu capture of the same kernel (not from this run)
            traffic_file = os.path.join(ROOT, "profiles", "router_kernel_traffic.json")
            if os.path.exists(traffic_file):
                with open(traffic_file) as f:
                    tr = json.load(f)
                if key in tr:
                    block["traffic"] = tr[key]
                    block["traffic_source"] = "profiles/router_kernel_traffic.json (ncu capture of this kernel; " \
                                              "not measured in this run)"

        persistent = persistent_launches > 0
        roof = None
        if router_ms:
            kname = ("fb_router_persistent_kernel" if persistent else "fb_router_kernel") + \
                    (" (fb_layer_step: both router passes in one launch)" if layer_api else " (fb_predict_and_plan)")
            k1_ms = statistics.median(router_ms)
            roof = roofline(k1_ms, alg_bytes, alg_flops, kname)
            roof["timing"] = "median of one event pair per launch, recorded by the library around the launch"
            roof["launches_timed"] = len(router_ms)
            roof["spread"] = spread(router_ms)
            roof["rest_of_step_us"] = ms_per_step * 1e3 - k1_ms * 1e3
            attach_traffic(roof, wl.name + ("/layer" if layer_api else ""))
        roof_pp = None
        if pp_b2b:
            pp_bytes, pp_flops = 2 * T * d + 2 * d * E + 4 * E, 2 * T * d * E
            roof_pp = roofline(statistics.median(pp_b2b), pp_bytes, pp_flops,
                               "fb_router_kernel + planner tail (fb_predict_and_plan)")
            roof_pp["timing"] = f"{pp_n} launches back to back between two events, median of {len(pp_b2b)} repeats"
            roof_pp["spread"] = spread(pp_b2b)
            roof_pp["tokens_per_s"] = T / (statistics.median(pp_b2b) * 1e-3)
            per_launch = roofline(statistics.median(pp_ms), pp_bytes, pp_flops, "")
            roof_pp["per_launch_events"] = dict(spread(pp_ms), frac=per_launch["frac"],
                                                 note="one event pair per launch: includes launch latency and "
                                                      "event granularity that back-to-back launches hide")
            attach_traffic(roof_pp, wl.name)
            if floor_us:
                roof_pp["main_loop_floor"] = dict(floor_us, how="fb_router_floor: the same launch without MMAs / with "
                                                  "them, and nothing after the main loop; timed like kernel_us")

        lb, la = out["load_before"].cpu().tolist(), out["load_after"].cpu().tolist()
        real_b, real_a = real_before.cpu().tolist(), out["rank_load"].cpu().tolist()
        mom = lambda L: (max(L) * len(L) / sum(L)) if sum(L) else 1.0

        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "T": T, "d": d, "E": E, "k": k, "R": R,
                           "gate": "sigmoid_group_topk" if wl.gate else "softmax_topk",
                           "api": "fb_layer_step" if layer_api else "fb_predict_and_plan + fb_route_dispatch",
                           "layers_in_ring": ring, "parallelism": f"replicas x{world}",
                           "l2": "each input matrix (%.0f MB) exceeds L2 (126 MB); consecutive launches read different matrices"
                                 % (T * d * 2 / 1e6) if T * d * 2 > L2_BYTES else
                                 "ring of layers; inputs may be L2-resident"},
                "clocks": clocks,
                "e2e": None if args.no_e2e else
                       {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps},
                "gpu_launches": int(launches), "device_status": status,
                "roofline": roof,
                "roofline_predict_and_plan": roof_pp,
                "roofline_note": "roofline: the dominant kernel of the timed step; roofline_predict_and_plan: the "
                                 "fused predictor + planner call by itself (the unit the 70 % target names), "
                                 "timed back to back",
                "migration": None if mig is None else dict(
                    mig, frac_of_hbm_peak=(mig["achieved_GBps"] / peaks["hbm_gbs"]) if mig["achieved_GBps"] else None),
                "load_balance": {"predicted_max_over_mean": [mom(lb), mom(la)],
                                 "realized_max_over_mean": [mom(real_b), mom(real_a)],
                                 "n_swaps": int(out["n_swaps"].item())}}
        if not args.no_cpu_baseline:
            T_s = min(T, 16384)
            sample_layer = layers_cpu[0] if T_s == T else I.make_layer(wl, 0, rank, T=T_s)
            sec = oracle_layer_seconds(wl, sample_layer, budget_kwargs(wl, T_s), 1, 0)
            line["cpu_baseline"] = {"value": T_s / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": f"1 whole layer of {T_s} tokens, full chain, {sec:.2f} s"}
        print(json.dumps(line), flush=True)
    ctx.close()
    if distributed:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
