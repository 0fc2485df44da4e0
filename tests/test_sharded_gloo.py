"""Token-sharded prediction + planning: the rank bookkeeping and the one exchange step, run as
gloo processes on CPU.  The library's two calls are replaced by the oracle's functions (test
infrastructure) so that the sharding logic itself can run without a GPU."""
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
    counts, pi_out, swaps, n_swaps, lb, la = i32(wl.E), i32(wl.E), i32(4 * 8), i32(1), i32(wl.R), i32(wl.R)
    sp.predict_and_plan(None, li.h_prev[lo:hi], hi - lo, li.expert_to_slot, None, 0, counts, pi_out, swaps, n_swaps, lb, la)
    dist.barrier()
    out.put((rank, lo, hi, counts.tolist(), pi_out.tolist(), swaps[:4 * int(n_swaps)].tolist(), la.tolist()))
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
    for rank, lo, hi, counts, pi_out, swaps, la in got:
        covered += list(range(lo, hi))
        assert counts == ref["counts"].tolist(), "every rank holds the global histogram after the exchange"
        assert pi_out == ref["pi_new"] and la == ref["load_after"]
        assert [tuple(swaps[i:i + 4]) for i in range(0, len(swaps), 4)] == ref["swaps"]
    assert covered == list(range(T)), "the shards tile the batch"


def test_shard_bounds():
    from paper_2608_14205_b200.sharded import shard_bounds
    assert [shard_bounds(10, 4, r) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]
    assert [shard_bounds(2, 4, r) for r in range(4)] == [(0, 1), (1, 2), (2, 2), (2, 2)]
    assert shard_bounds(0, 3, 1) == (0, 0)
