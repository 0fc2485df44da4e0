"""Token-sharded prediction and planning over several GPUs (one process per GPU).

Tokens are independent up to the expert histogram, so data-parallel / expert-parallel ranks
each run the early router pass on their own tokens and need exactly one exchange step: a sum
all-reduce of the E x u32 count vector (at most 1 KB).  After it every rank holds the global
counts and replays the same deterministic, integer-exact planner, so all ranks arrive at the
same plan without a broadcast ("Budgeted Expert-Swap Planning": the sorted sweep and its
tie-breaks are fixed, which keeps the ranks' plans consistent).

The collective is `torch.distributed.all_reduce` on the count tensor (NCCL between GPUs;
any backend works, the tests run it over gloo).  Everything else is the single-GPU library.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


class ShardedPredictor:
    """`ctx` is a binding.Context (or any object with its fb_predict_load / fb_plan_swaps)."""

    def __init__(self, ctx, group: Optional[dist.ProcessGroup] = None):
        self.ctx = ctx
        self.group = group

    def predict_and_plan(self, router, h_prev_local, T_local: int, expert_to_slot, budget, layer_id: int, counts,
                         expert_to_slot_out, swaps, n_swaps, load_before, load_after, stream=None) -> None:
        """Same outputs as fb_predict_and_plan on the concatenation of all ranks' tokens.

        `counts` receives the GLOBAL count vector on every rank.  `budget` must be the same on
        every rank (in particular gamma, which the callers derive from the global batch)."""
        self.ctx.fb_predict_load(router, h_prev_local, T_local, counts, None, None, stream=stream)
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1:
            if stream is not None and counts.is_cuda:
                with torch.cuda.stream(stream):
                    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=self.group)
            else:
                dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=self.group)
        self.ctx.fb_plan_swaps(counts, expert_to_slot, budget, layer_id, expert_to_slot_out, swaps, n_swaps,
                               load_before, load_after, stream=stream)


def shard_bounds(T: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced token ranges: the first T % world ranks get one token more."""
    base, extra = divmod(T, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
