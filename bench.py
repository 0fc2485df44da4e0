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
import threading
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


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                if get_reasons is not None:
                    r = int(get_reasons(self._h))
                    for name, bit in names.items():
                        if r & bit:
                            self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (for profiler captures)")
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

    # ---- timed region: exactly K steps; events on the launching (current) stream
    K = args.steps
    # The whole region is bracketed by two events.  The duration of the dominant kernel (the
    # router kernel: the first launch of the step) comes from a pair of events that the library
    # records directly around that launch, on every `sample_every`-th step only: an event
    # between two launches keeps the GPU from starting the next kernel's launch early and
    # costs about 2 us per record, which would otherwise be charged to every step.
    sample_every = 8 if K >= 16 else 1
    sampled = [i for i in range(K) if i % sample_every == 0]
    ev = {i: [torch.cuda.Event(enable_timing=True) for _ in range(2)] for i in sampled}
    for pair in ev.values():                 # torch creates the CUDA event on its first record
        for e in pair:
            e.record()
    ev_begin, ev_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    launches0 = ctx.fb_launch_count()
    persistent0 = ctx.fb_persistent_launch_count()
    barrier()
    sampler.start()
    ev_begin.record()
    for i in range(K):
        e2 = ev.get(i)
        if e2:
            ctx.fb_time_next_router_launch(e2[0], e2[1])
        step(layers[i % ring])
    ev_end.record()
    barrier()
    clocks = sampler.stop()
    launches = ctx.fb_launch_count() - launches0
    persistent_launches = ctx.fb_persistent_launch_count() - persistent0
    total_ms = ev_begin.elapsed_time(ev_end)
    router_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in sampled]
    total_ms = max_over_ranks(total_ms, dev)
    status = ctx.fb_device_status()

    # ---- the fused predictor + planner alone (fb_predict_and_plan), outside the timed region:
    # per-launch events, for the roofline fraction of that call by itself
    pp_n = 0 if args.no_e2e else 24
    pp_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(pp_n)]
    for i in range(pp_n):
        pp_ev[i][0].record()
        predict_and_plan(layers[i % ring])
        pp_ev[i][1].record()
    barrier()
    pp_ms = [a.elapsed_time(b) for a, b in pp_ev]

    # ---- stage 3 on this device (not part of the step): the plan just produced, applied to a buffer
    # of E slot images of the workload's expert size; HBM bound, 4 bytes of traffic per byte moved
    mig = None
    if not args.no_e2e and wl.expert_bytes > 0 and bkw["max_swaps"] > 0:
        S = wl.expert_bytes // 16 * 16
        weights = torch.empty(E * S, dtype=torch.uint8, device=dev)      # content does not matter for timing
        cap = int(bkw["max_swaps"])
        L0d = layers[(K - 1) % ring]
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
        k1_ms = statistics.mean(router_ms)

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
                    "tensor_frac_of_sustained": tf / peaks["bf16_tflops_sustained"]}

        persistent = persistent_launches > 0
        kname = ("fb_router_persistent_kernel" if persistent else "fb_router_kernel") + \
                (" (fb_layer_step: both router passes in one launch)" if layer_api else " (fb_predict_and_plan)")
        roof = roofline(k1_ms, alg_bytes, alg_flops, kname)
        roof["kernel_us_median"] = statistics.median(router_ms) * 1e3
        roof["launches_timed"] = len(router_ms)
        roof["rest_of_step_us"] = ms_per_step * 1e3 - k1_ms * 1e3
        traffic_key = wl.name + ("/layer" if layer_api else "")
        traffic_file = os.path.join(ROOT, "profiles", "router_kernel_traffic.json")
        if os.path.exists(traffic_file):
            with open(traffic_file) as f:
                tr = json.load(f)
            if traffic_key in tr:
                roof["traffic"] = tr[traffic_key]

        lb, la = out["load_before"].cpu().tolist(), out["load_after"].cpu().tolist()
        pi_new = out["pi_out"].cpu().tolist()
        so = out["slot_offsets"].cpu().tolist()
        m = E // R
        realized = [so[pi_new[e] + 1] - so[pi_new[e]] for e in range(E)]
        pi_old = layers_cpu[(K - 1) % ring].expert_to_slot.tolist()
        real_before = [0] * R
        for e in range(E):
            real_before[pi_old[e] // m] += realized[e]
        real_after = out["rank_load"].cpu().tolist()
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
                "predict_and_plan": None if not pp_ms else dict(
                    roofline(statistics.mean(pp_ms), 2 * T * d + 2 * d * E + 4 * E, 2 * T * d * E,
                             "fb_router_kernel (fb_predict_and_plan alone, one event pair per launch)"),
                    tokens_per_s=T / (statistics.mean(pp_ms) * 1e-3), launches_timed=len(pp_ms)),
                "migration": None if mig is None else dict(
                    mig, frac_of_hbm_peak=(mig["achieved_GBps"] / peaks["hbm_gbs"]) if mig["achieved_GBps"] else None),
                "load_balance": {"predicted_max_over_mean": [mom(lb), mom(la)],
                                 "realized_max_over_mean": [mom(real_before), mom(real_after)],
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
