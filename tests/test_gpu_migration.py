"""GPU parity of the weight exchange (stage 3 on one device) against the oracle: byte exact."""
import numpy as np
import pytest
import torch

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B
from paper_2608_14205_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _run(E, S, pi0, swaps, max_swaps=None, seed=0):
    dev = torch.device("cuda")
    w = np.random.default_rng(seed).integers(0, 256, size=(E, S), dtype=np.uint8)
    max_swaps = max(1, len(swaps)) if max_swaps is None else max_swaps
    sw = np.zeros((max(1, max_swaps), 4), dtype=np.int32)
    for i, s in enumerate(swaps):
        sw[i] = s
    w_d = torch.from_numpy(w.copy()).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.fb_apply_swaps(w_d, S, E, torch.tensor(pi0, dtype=torch.int32, device=dev), torch.from_numpy(sw).to(dev),
                     torch.tensor([len(swaps)], dtype=torch.int32, device=dev), max_swaps, status)
    torch.cuda.synchronize()
    return w, w_d.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("E,R,S,cap", [
    (8, 4, 16, 2),                 # one 16-byte unit per slot
    (16, 4, 4096 + 48, 8),         # ragged tail inside one block's span
    (64, 8, 1 << 20, 10),          # several blocks per swap
    (256, 32, 3 * 32768 * 16 + 16, 5),   # more 16-byte units than one pass of the grid covers, ragged
])
def test_planned_swaps_applied_to_weights(E, R, S, cap):
    pi0 = I.random_placement(E, 3).tolist()
    counts = I.random_counts(E, 50000, 3, zipf_s=1.2).tolist()
    bud = O.Budget(max_swaps=cap, global_ns=2**64 - 1, rank_ns=2**64 - 1, link_ns=2**64 - 1, tau_tokens=0,
                   gamma_num=1, gamma_den=100, alpha_ns=(0, 0), fs_per_byte=(0, 0), ranks_per_node=0, expert_bytes=0)
    swaps, pi_new, _, _ = O.plan_swaps(counts, pi0, R, bud)
    assert len(swaps) >= 1
    w, got, status = _run(E, S, pi0, swaps, max_swaps=cap + 3)      # unused swap entries are ignored
    ref, pi_after = O.apply_swaps(w, pi0, swaps)
    assert status == 0 and pi_after == pi_new
    assert np.array_equal(got, ref)
    for e in range(E):
        assert np.array_equal(got[pi_new[e]], w[pi0[e]])


def test_plan_from_the_library_feeds_the_exchange_without_a_host_round_trip():
    wl = I.WORKLOADS["dsv3"]
    T, S = 2048, 4096
    dev = torch.device("cuda")
    li = I.make_layer(wl, 0, 0, T=T)
    ctx = B.Context(T, wl.d, wl.E, wl.k, wl.R, wl.gate, wl.n_group, wl.topk_group, wl.renorm, wl.route_scale)
    from tests import parity_util as P
    budget = B.make_budget(**P.budget_kwargs(wl, T))
    router = B.make_router(li.W.to(dev), None, li.select_bias.to(dev))
    i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
    counts, pi_out, swaps, n_swaps, lb, la = i32(wl.E), i32(wl.E), i32(4 * 128), i32(1), i32(wl.R), i32(wl.R)
    pi = li.expert_to_slot.to(dev)
    w = np.random.default_rng(1).integers(0, 256, size=(wl.E, S), dtype=np.uint8)
    w_d = torch.from_numpy(w.copy()).to(dev)
    ctx.fb_predict_and_plan(router, li.h_prev.to(dev), T, pi, budget, 0, counts, pi_out, swaps, n_swaps, lb, la)
    B.fb_apply_swaps(w_d, S, wl.E, pi, swaps, n_swaps, 128)          # same stream, no synchronisation between
    torch.cuda.synchronize()
    assert int(n_swaps.item()) == 5
    new, old = pi_out.cpu().tolist(), pi.cpu().tolist()
    got = w_d.cpu().numpy()
    for e in range(wl.E):
        assert np.array_equal(got[new[e]], w[old[e]]), "every expert's weights sit where the new placement says"
    ctx.close()


def test_empty_plan_bad_arguments_and_bad_swaps():
    w, got, status = _run(8, 64, list(range(8)), [])
    assert np.array_equal(w, got) and status == 0
    # a swap naming an expert out of range is skipped and reported; the valid one still runs
    w, got, status = _run(8, 64, list(range(8)), [(0, 1, 0, 9), (0, 1, 2, 5)])
    ref, _ = O.apply_swaps(w, list(range(8)), [(0, 1, 2, 5)])
    assert np.array_equal(got, ref) and status == B.FB_ERR_RANGE
    dev = torch.device("cuda")
    z = torch.zeros(8 * 64, dtype=torch.uint8, device=dev)
    i = torch.zeros(8, dtype=torch.int32, device=dev)
    with pytest.raises(B.FbError):
        B.fb_apply_swaps(z, 24, 8, i, i, i, 1)                       # size not a multiple of 16
    with pytest.raises(B.FbError):
        B.fb_apply_swaps(z[1:], 16, 8, i, i, i, 1)                   # misaligned buffer
    B.fb_apply_swaps(z, 64, 8, i, i, i, 0)                           # capacity 0: nothing to do


@pytest.mark.parametrize("S,stage", [(4096, 0), (1 << 20, 1 << 18), (3 * 4096 + 16, 4096)])
def test_staged_exchange_by_device_copies(S, stage):
    # the host-issued variant: same result, whole-expert staging, pieces, and a ragged last piece
    wl = I.WORKLOADS["qwen3"]
    E, R = wl.E, wl.R
    dev = torch.device("cuda")
    pi0 = I.random_placement(E, 7).tolist()
    counts = I.random_counts(E, 60000, 7, zipf_s=1.1).tolist()
    bud = O.Budget(max_swaps=6, global_ns=2**64 - 1, rank_ns=2**64 - 1, link_ns=2**64 - 1, tau_tokens=0,
                   gamma_num=1, gamma_den=100, alpha_ns=(0, 0), fs_per_byte=(0, 0), ranks_per_node=0, expert_bytes=0)
    swaps, pi_new, _, _ = O.plan_swaps(counts, pi0, R, bud)
    assert len(swaps) >= 2
    w = np.random.default_rng(2).integers(0, 256, size=(E, S), dtype=np.uint8)
    sw = np.zeros((8, 4), dtype=np.int32)
    sw[:len(swaps)] = swaps
    w_d = torch.from_numpy(w.copy()).to(dev)
    ctx = B.Context(128, wl.d, E, wl.k, R, wl.gate, wl.n_group, wl.topk_group)
    side = torch.cuda.Stream()
    ctx.fb_apply_swaps_staged(w_d, S, torch.tensor(pi0, dtype=torch.int32, device=dev), torch.from_numpy(sw).to(dev),
                              torch.tensor([len(swaps)], dtype=torch.int32, device=dev), 8, stage,
                              plan_stream=None, copy_stream=side)
    side.synchronize()
    ref, _ = O.apply_swaps(w, pi0, swaps)
    assert np.array_equal(w_d.cpu().numpy(), ref)
    ctx.close()


def test_calibration_predicts_the_exchange_time():
    dev = torch.device("cuda")
    small, large = 1 << 20, 44_040_192
    buf = torch.empty(2 * large, dtype=torch.uint8, device=dev)
    cal = B.fb_calibrate_exchange(buf, small, large, reps=5)
    assert cal["t_large_ns"] > cal["t_small_ns"] > 0
    assert (cal["alpha_ns"], cal["fs_per_byte"]) == O.fit_cost_model(cal["t_small_ns"], cal["t_large_ns"], small, large)
    gbps = 1e6 / cal["fs_per_byte"]                                  # bytes per ns = GB/s moved per direction
    assert 500 < gbps < 8000 and cal["alpha_ns"] < 50_000, cal
    # the fitted model, handed to the planner's cost function, reproduces an independent measurement
    bud = B.make_budget(max_swaps=4, alpha_ns=(cal["alpha_ns"],) * 2, fs_per_byte=(cal["fs_per_byte"],) * 2,
                        expert_bytes=16 << 20)
    predicted = B.fb_swap_cost_ns(bud, 0, 1)
    w = torch.empty(2 * (16 << 20), dtype=torch.uint8, device=dev)
    pi = torch.arange(2, dtype=torch.int32, device=dev)
    sw = torch.tensor([[0, 1, 0, 1]], dtype=torch.int32, device=dev)
    n = torch.tensor([1], dtype=torch.int32, device=dev)
    best = 1e9
    for _ in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); B.fb_apply_swaps(w, 16 << 20, 2, pi, sw, n, 1); b.record()
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b) * 1e6)
    assert 0.6 * best < predicted < 1.6 * best, (predicted, best, cal)
