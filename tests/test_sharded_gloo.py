"""The token-sharded layer: the rank bookkeeping and the two exchange steps (count all-reduce,
slot-count all-gather), run as gloo processes on CPU.  The library's calls are replaced by the
oracle's functions (test infrastructure) so that the sharding logic itself can run without a
GPU; the same module drives the CUDA library in tests/test_gpu_sharded.py."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OracleContext:
    """Stands in for binding.Context on CPU tensors: same two calls, computed by the oracle."""

    def __init__(self, O, gate, W_bits, R, bud):
        self.O, self.gate, self.W_bits, self.R, self.bud = O, gate, W_bits, R, bud

    def fb_predict_load(self, router, x, T, counts, topk_ids=None, logits=None, stream=None):
        bits = x.contiguous().view(torch.int16).numpy().view(np.uint16)[:T]
        z = self.O.router_logits(bits, self.W_bits, None)
        ids, _ = self.O.select_topk(z, self.gate, None)
        counts.copy_(torch.from_numpy(self.O.expert_histogram(ids, self.gate.E).astype(np.int32)))

    def fb_route_dispatch(self, router, x, T, expert_to_slot, ids_out, w_out, so, ro, perm, inv, rl, logits=None,
                          stream=None):
        bits = x.contiguous().view(torch.int16).numpy().view(np.uint16)[:T]
        z = self.O.router_logits(bits, self.W_bits, None)
        ids, w = self.O.select_topk(z, self.gate, None)
        s, r, p, i, l = self.O.dispatch_index(ids, expert_to_slot.tolist(), self.R)
        k = self.gate.k
        ids_out[:T * k] = torch.from_numpy(ids.reshape(-1).astype(np.int32))
        w_out[:T * k] = torch.from_numpy(w.reshape(-1).astype(np.float32))
        so.copy_(torch.from_numpy(s.astype(np.int32)))
        ro.copy_(torch.from_numpy(r.astype(np.int32)))
        perm[:T * k] = torch.from_numpy(p.astype(np.int32))
        inv[:T * k] = torch.from_numpy(i.astype(np.int32))
        rl.copy_(torch.from_numpy(l.astype(np.int32)))

    def fb_dispatch_slot_counts(self, slot_offsets, slot_counts, stream=None):
        E = self.gate.E
        slot_counts.view(-1)[:E] = slot_offsets[1:E + 1] - slot_offsets[:E]

    def fb_dispatch_globalize(self, T, world, rank, counts_all, local_offsets, ids, expert_to_slot, inv, so, ro, rl,
                              stream=None):
        k, E = self.gate.k, self.gate.E
        g_so, g_ro, g_rl, g_inv = self.O.globalize_dispatch(counts_all.view(world, E).tolist(), rank,
                                                            local_offsets.tolist(), inv[:T * k].tolist(), self.R)
        so.copy_(torch.from_numpy(g_so.astype(np.int32)))
        ro.copy_(torch.from_numpy(g_ro.astype(np.int32)))
        rl.copy_(torch.from_numpy(g_rl.astype(np.int32)))
        inv[:T * k] = torch.from_numpy(g_inv.astype(np.int32))

    def fb_plan_swaps(self, counts, expert_to_slot, budget, layer_id, pi_out, swaps, n_swaps, lb, la, stream=None):
        sw, pi_new, before, after = self.O.plan_swaps(counts.tolist(), expert_to_slot.tolist(), self.R, self.bud, layer_id)
        pi_out.copy_(torch.tensor(pi_new, dtype=torch.int32))
        n_swaps[0] = len(sw)
        for i, s in enumerate(sw):
            swaps[4 * i:4 * i + 4] = torch.tensor(s, dtype=torch.int32)
        lb.copy_(torch.tensor(before, dtype=torch.int32))
        la.copy_(torch.tensor(after, dtype=torch.int32))


def _worker(rank, world, port, T, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import freebalance_oracle as O
    from paper_2608_14205_b200 import inputs as I
    from paper_2608_14205_b200.sharded import ShardedPredictor, shard_bounds
    from tests.test_oracle_serving import _budget, _gate, bits
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = I.WORKLOADS["tiny"]
    li = I.make_layer(wl, 0, 0, T=T)                       # every rank draws the same batch, keeps its shard
    lo, hi = shard_bounds(T, world, rank)
    ctx = OracleContext(O, _gate(wl), bits(li.W), wl.R, _budget(wl, T))
    sp = ShardedPredictor(ctx)
    i32 = lambda n: torch.zeros(n, dtype=torch.int32)
    Tl, k = hi - lo, wl.k
    o = dict(counts=i32(wl.E), pi_out=i32(wl.E), swaps=i32(4 * 8), n_swaps=i32(1), load_before=i32(wl.R),
             load_after=i32(wl.R), ids=i32(max(1, Tl * k)), w=torch.zeros(max(1, Tl * k)), slot_offsets=i32(wl.E + 1),
             rank_offsets=i32(wl.R + 1), perm=i32(max(1, Tl * k)), inv_perm=i32(max(1, Tl * k)), rank_load=i32(wl.R))
    sp.layer_step(None, li.h_prev[lo:hi], li.H[lo:hi], Tl, li.expert_to_slot, None, 0, o, i32(world * wl.E))
    dist.barrier()
    out.put((rank, lo, hi, o["counts"].tolist(), o["pi_out"].tolist(), o["swaps"][:4 * int(o["n_swaps"])].tolist(),
             o["load_after"].tolist(), o["inv_perm"][:Tl * k].tolist(), o["slot_offsets"].tolist(),
             o["rank_offsets"].tolist(), o["rank_load"].tolist(), o["ids"][:Tl * k].tolist()))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,T", [(2, 301), (3, 256)])
def test_all_ranks_reach_the_plan_of_the_whole_batch(world, T):
    sys.path.insert(0, ROOT)
    from oracle import freebalance_oracle as O
    from paper_2608_14205_b200 import inputs as I
    from tests.test_oracle_serving import _budget, _gate, bits
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, T, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = I.WORKLOADS["tiny"]
    li = I.make_layer(wl, 0, 0, T=T)
    ref = O.layer_step(bits(li.h_prev), bits(li.H), bits(li.W), _gate(wl), wl.R, li.expert_to_slot.tolist(), _budget(wl, T))
    covered = []
    k = wl.k
    d_so, d_ro, _, d_inv, d_rl = ref["dispatch"]
    for rank, lo, hi, counts, pi_out, swaps, la, inv, so, ro, rl, ids in got:
        covered += list(range(lo, hi))
        assert counts == ref["counts"].tolist(), "every rank holds the global histogram after the exchange"
        assert pi_out == ref["pi_new"] and la == ref["load_after"]
        assert [tuple(swaps[i:i + 4]) for i in range(0, len(swaps), 4)] == ref["swaps"]
        # the dispatch index of the whole batch, cut to this rank's tokens
        assert ids == ref["ids"][lo:hi].reshape(-1).tolist()
        assert inv == d_inv[lo * k:hi * k].tolist(), "whole-batch positions of the shard's assignments"
        assert so == d_so.tolist() and ro == d_ro.tolist() and rl == d_rl.tolist()
    assert covered == list(range(T)), "the shards tile the batch"


def test_shard_bounds():
    from paper_2608_14205_b200.sharded import shard_bounds
    assert [shard_bounds(10, 4, r) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]
    assert [shard_bounds(2, 4, r) for r in range(4)] == [(0, 1), (1, 2), (2, 2), (2, 2)]
    assert shard_bounds(0, 3, 1) == (0, 0)
