"""Stage 3 beside attention, on one GPU: how much of the weight exchange stays hidden.

The method hides prediction, planning and weight transfer of layer l behind the attention of
layer l (two-stream schedule of the paper's "Overlap Analysis"; the budget of Eq. 10 is the
attention time minus a margin).  This script measures that schedule on one device with a
stand-in for attention (a chain of bf16 matrix products through torch, sized to a given
duration - it is not part of the library):

  stream A:  stand-in attention                                  (critical path)
  stream B:  fb_predict_and_plan -> fb_apply_swaps               (auxiliary work)

and reports the duration of A alone, of B alone, of both started together, and the exposed
time (both - A alone).  Logical EP ranks are a mapping on one GPU, so the exchange is HBM to
HBM; the figures say what the auxiliary work costs beside a compute-bound kernel on the same
device, not what an NVLink transfer would cost.

    python -m paper_2608_14205_b200.migration_overlap --workload dsv3 --window-us 500
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding as B
from . import inputs as I
from .serving import make_budget_for


def _timed(fn, reps, dev):
    for _ in range(3):
        fn()
    torch.cuda.synchronize(dev)
    out = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize(dev)
        out.append(a.elapsed_time(b) * 1e3)
    return statistics.median(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="dsv3", choices=sorted(I.WORKLOADS))
    ap.add_argument("--window-us", type=float, default=500.0, help="target duration of the stand-in attention")
    ap.add_argument("--expert-bytes", type=int, default=0, help="0 = the workload's expert size")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--exchange-only", type=int, default=0, metavar="SLOTS",
                    help="only time fb_apply_swaps: 5 swaps among SLOTS (>= 10) slot images of the expert size")
    args = ap.parse_args()
    wl = I.WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    if args.exchange_only:
        slots = max(10, args.exchange_only)
        S = (args.expert_bytes or wl.expert_bytes or 16 * 2**20) // 16 * 16
        weights = torch.empty(slots * S, dtype=torch.uint8, device=dev)
        pi = torch.arange(slots, dtype=torch.int32, device=dev)
        swaps = torch.tensor([[0, 1, 2 * i, 2 * i + 1] for i in range(5)], dtype=torch.int32, device=dev)
        n_swaps = torch.tensor([5], dtype=torch.int32, device=dev)
        us = _timed(lambda: B.fb_apply_swaps(weights, S, slots, pi, swaps, n_swaps, 5), args.reps, dev)
        print(json.dumps(dict(expert_bytes=S, swaps=5, traffic_bytes=20 * S, us=us, GBps=20 * S / us / 1e3)))
        return
    T, E = wl.T, wl.E
    S = (args.expert_bytes or wl.expert_bytes or 16 * 2**20) // 16 * 16
    li = I.make_layer(wl, 0, 0)
    ctx = B.Context(T, wl.d, E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    budget = make_budget_for(wl, T)
    sb = li.select_bias.to(dev) if li.select_bias is not None else None
    router = B.make_router(li.W.to(dev), None, sb)
    h_prev, pi = li.h_prev.to(dev), li.expert_to_slot.to(dev)
    i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
    cap = max(1, min(wl.max_swaps, E // 2))
    counts, pi_out, swaps, n_swaps, lb, la = i32(E), i32(E), i32(4 * cap), i32(1), i32(wl.R), i32(wl.R)
    weights = torch.empty(E * S, dtype=torch.uint8, device=dev)          # content is irrelevant for timing

    # stand-in attention: square bf16 products, count chosen to fill the window
    n = 4096
    xa, xb = torch.randn(n, n, device=dev).to(torch.bfloat16), torch.randn(n, n, device=dev).to(torch.bfloat16)
    one = _timed(lambda: torch.matmul(xa, xb), 5, dev)
    n_mm = max(1, round(args.window_us / one))

    side = torch.cuda.Stream(device=dev)

    def attention():
        y = xa
        for _ in range(n_mm):
            y = torch.matmul(y, xb)

    def auxiliary(stream=None):
        ctx.fb_predict_and_plan(router, h_prev, T, pi, budget, 0, counts, pi_out, swaps, n_swaps, lb, la,
                                stream=stream)
        B.fb_apply_swaps(weights, S, E, pi, swaps, n_swaps, cap, stream=stream)

    def exchange(stream=None):
        B.fb_apply_swaps(weights, S, E, pi, swaps, n_swaps, cap, stream=stream)

    def exchange_by_copies(stream=None):
        # host-issued device-to-device copies (waits for the plan on the current stream first)
        ctx.fb_apply_swaps_staged(weights, S, pi, swaps, n_swaps, cap, 0, plan_stream=None, copy_stream=stream)

    def beside_attention(work, attention_first):
        def run():
            side.wait_stream(torch.cuda.current_stream(dev))
            if attention_first:
                attention()
                work(side)
            else:
                work(side)
                attention()
            torch.cuda.current_stream(dev).wait_stream(side)
        return run

    t_attn = _timed(attention, args.reps, dev)
    t_aux = _timed(auxiliary, args.reps, dev)
    t_exch = _timed(exchange, args.reps, dev)
    t_both = min(_timed(beside_attention(auxiliary, False), args.reps, dev),
                 _timed(beside_attention(auxiliary, True), args.reps, dev))
    t_copy = _timed(exchange_by_copies, args.reps, dev)
    t_copy_both = min(_timed(beside_attention(exchange_by_copies, False), args.reps, dev),
                      _timed(beside_attention(exchange_by_copies, True), args.reps, dev))
    t_exch_both = min(_timed(beside_attention(exchange, False), args.reps, dev),
                      _timed(beside_attention(exchange, True), args.reps, dev))
    print(json.dumps(dict(
        workload=wl.name, T=T, expert_bytes=S, swaps=int(n_swaps.item()),
        exchange_bytes=4 * S * int(n_swaps.item()),
        attention_stand_in=f"{n_mm} x bf16 matmul {n}^3 (torch)", attention_us=t_attn, auxiliary_us=t_aux,
        together_us=t_both, exposed_us=max(0.0, t_both - t_attn), hidden_fraction=
        (1.0 - max(0.0, t_both - t_attn) / t_aux) if t_aux > 0 else None,
        exchange_only=dict(alone_us=t_exch, together_us=t_exch_both, exposed_us=max(0.0, t_exch_both - t_attn),
                           hidden_fraction=(1.0 - max(0.0, t_exch_both - t_attn) / t_exch) if t_exch > 0 else None),
        exchange_by_copies=dict(alone_us=t_copy, together_us=t_copy_both, exposed_us=max(0.0, t_copy_both - t_attn),
                                hidden_fraction=(1.0 - max(0.0, t_copy_both - t_attn) / t_copy) if t_copy > 0 else None),
        budget_window_us=args.window_us, device_status=ctx.fb_device_status())))
    ctx.close()


if __name__ == "__main__":
    main()
