"""The per-layer path on several GPUs, token-sharded (one process per GPU).

Tokens are independent up to the expert histogram, so data-parallel / expert-parallel ranks
each run the router passes on their own tokens (a contiguous range of the batch, in rank order)
and need exactly two small exchanges per layer ("Budgeted Expert-Swap Planning": ranks exchange
only the compact load statistics and then reproduce the same plan locally):

1. a sum all-reduce of the E x u32 predicted counts (at most 1 KB), after which every rank
   replays the same deterministic, integer-exact planner and holds the same plan without a
   broadcast;
2. an all-gather of the E x u32 per-slot counts of the normal pass (world x E words), after
   which every rank knows where its assignments fall in the dispatch order of the whole batch.

Both collectives are `torch.distributed` calls on small tensors (NCCL between GPUs; any backend
works - the CPU tests run them over gloo).  They are pure latency, so no fused
compute + collective kernel exists for them.  Everything else is the single-GPU library: this
module only passes pointers.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def _world(group) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def _rank(group) -> int:
    return dist.get_rank(group) if dist.is_available() and dist.is_initialized() else 0


class ShardedPredictor:
    """`ctx` is a binding.Context (or any object with the same calls)."""

    def __init__(self, ctx, group: Optional[dist.ProcessGroup] = None):
        self.ctx = ctx
        self.group = group
        self._local_offsets = None         # E + 1 words: the shard's own slot offsets
        self._mine = None                  # E words: this rank's row for the all-gather

    def _collective(self, fn, stream):
        if stream is not None and torch.cuda.is_available():
            with torch.cuda.stream(stream):
                fn()
        else:
            fn()

    def predict_and_plan(self, router, h_prev_local, T_local: int, expert_to_slot, budget, layer_id: int, counts,
                         expert_to_slot_out, swaps, n_swaps, load_before, load_after, stream=None) -> None:
        """Same outputs as fb_predict_and_plan on the concatenation of all ranks' tokens.

        `counts` receives the GLOBAL count vector on every rank.  `budget` must be the same on
        every rank (in particular gamma, which the callers derive from the global batch)."""
        self.ctx.fb_predict_load(router, h_prev_local, T_local, counts, None, None, stream=stream)
        if _world(self.group) > 1:
            self._collective(lambda: dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=self.group), stream)
        self.ctx.fb_plan_swaps(counts, expert_to_slot, budget, layer_id, expert_to_slot_out, swaps, n_swaps,
                               load_before, load_after, stream=stream)

    def route_dispatch(self, router, H_local, T_local: int, expert_to_slot, topk_ids, topk_w, slot_offsets,
                       rank_offsets, perm_local, inv_perm, rank_load, slot_counts_all, stream=None) -> None:
        """fb_route_dispatch for a shard of the batch.

        topk_ids / topk_w describe the local tokens.  inv_perm[i*k + j] receives the position of
        local assignment (i, j) in the dispatch order of the WHOLE batch; slot_offsets,
        rank_offsets and rank_load describe the whole batch and are identical on every rank;
        perm_local keeps the shard's own order (local positions -> local assignments).
        slot_counts_all: scratch of world x E int32 on the same device."""
        world, rank = _world(self.group), _rank(self.group)
        E = expert_to_slot.numel()
        assert slot_counts_all.numel() == world * E, "slot_counts_all must hold world x E words"
        if self._local_offsets is None or self._local_offsets.numel() != E + 1 or \
                self._local_offsets.device != slot_counts_all.device:
            self._local_offsets = slot_counts_all.new_zeros(E + 1)
            self._mine = slot_counts_all.new_zeros(E)
        local_offsets, mine = self._local_offsets, self._mine
        self.ctx.fb_route_dispatch(router, H_local, T_local, expert_to_slot, topk_ids, topk_w, local_offsets,
                                   rank_offsets, perm_local, inv_perm, rank_load, None, stream=stream)
        if world > 1:
            self.ctx.fb_dispatch_slot_counts(local_offsets, mine, stream=stream)
            self._collective(lambda: dist.all_gather_into_tensor(slot_counts_all.view(-1), mine, group=self.group),
                             stream)
        else:
            self.ctx.fb_dispatch_slot_counts(local_offsets, slot_counts_all.view(-1), stream=stream)
        self.ctx.fb_dispatch_globalize(T_local, world, rank, slot_counts_all, local_offsets, topk_ids,
                                       expert_to_slot, inv_perm, slot_offsets, rank_offsets, rank_load, stream=stream)

    def layer_step(self, router, h_prev_local, H_local, T_local: int, expert_to_slot, budget, layer_id: int, out,
                   slot_counts_all, stream=None) -> None:
        """One whole layer on this rank's shard; `out` holds the buffers of fb_layer_step by name
        (counts, pi_out, swaps, n_swaps, load_before, load_after, ids, w, slot_offsets,
        rank_offsets, perm, inv_perm, rank_load)."""
        self.predict_and_plan(router, h_prev_local, T_local, expert_to_slot, budget, layer_id, out["counts"],
                              out["pi_out"], out["swaps"], out["n_swaps"], out["load_before"], out["load_after"],
                              stream=stream)
        self.route_dispatch(router, H_local, T_local, out["pi_out"], out["ids"], out["w"], out["slot_offsets"],
                            out["rank_offsets"], out["perm"], out["inv_perm"], out["rank_load"], slot_counts_all,
                            stream=stream)


def shard_bounds(T: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced token ranges: the first T % world ranks get one token more."""
    base, extra = divmod(T, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
