"""ctypes binding of libfreebalance.so: argument marshalling only.

Every function below has the name and meaning of the C entry point declared in
``include/freebalance.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is
handed to the library, the stream is torch's current stream unless given.  There
is no fallback: if the shared library is missing or fails to load this raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

_U64_OFF = 2**64 - 1


class FbConfig(ctypes.Structure):
    _fields_ = [("T_max", ctypes.c_int32), ("d", ctypes.c_int32), ("E", ctypes.c_int32),
                ("k", ctypes.c_int32), ("R", ctypes.c_int32), ("gate", ctypes.c_int32),
                ("n_group", ctypes.c_int32), ("topk_group", ctypes.c_int32),
                ("renorm", ctypes.c_int32), ("route_scale", ctypes.c_float)]


class FbRouter(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("logit_bias", ctypes.c_void_p), ("select_bias", ctypes.c_void_p)]


class FbBudget(ctypes.Structure):
    _fields_ = [("max_swaps", ctypes.c_uint32), ("global_ns", ctypes.c_uint64),
                ("rank_ns", ctypes.c_uint64), ("link_ns", ctypes.c_uint64),
                ("tau_tokens", ctypes.c_uint32), ("gamma_num", ctypes.c_uint32),
                ("gamma_den", ctypes.c_uint32), ("alpha_ns", ctypes.c_uint64 * 2),
                ("fs_per_byte", ctypes.c_uint64 * 2), ("ranks_per_node", ctypes.c_int32),
                ("expert_bytes", ctypes.c_uint64), ("expert_bytes_table", ctypes.c_void_p),
                ("mode", ctypes.c_int32), ("frontier_width", ctypes.c_int32)]


FB_PLAN_LOOP, FB_PLAN_SWEEP, FB_PLAN_WIDE = 0, 1, 2


FB_OK = 0
FB_ERR_INVALID_ARG = 1
FB_ERR_UNSUPPORTED_SHAPE = 2
FB_ERR_CUDA = 3
FB_ERR_BAD_PLACEMENT = 4
FB_ERR_TIMEOUT = 5
FB_ERR_RANGE = 6
FB_ERR_INTERNAL = 7

EXPORTS = ["fb_create", "fb_destroy", "fb_budget_ns", "fb_swap_cost_ns", "fb_predict_load",
           "fb_plan_swaps", "fb_predict_and_plan", "fb_route_dispatch", "fb_layer_step_host",
           "fb_device_status", "fb_launch_count", "fb_status_string", "fb_predict_load_static", "fb_layer_step",
           "fb_set_pair_limit", "fb_set_stage_limit", "fb_max_pairs", "fb_persistent_launch_count",
           "fb_time_next_router_launch", "fb_router_floor", "fb_row_cosine_mean", "fb_topk_hits", "fb_apply_swaps",
           "fb_apply_swaps_staged", "fb_fit_cost_model", "fb_calibrate_exchange", "fb_selftest_wait_timeout",
           "fb_set_stamp_buffer", "fb_clock_probe", "fb_attention_begin", "fb_attention_end", "fb_layer_budget_ns",
           "fb_attention_set_time_ns", "fb_attention_reset", "fb_dispatch_slot_counts", "fb_dispatch_globalize",
           "fb_standin_attention", "fb_set_split"]

_lib = None


class FbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().fb_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{where}: {msg} (status {status})")


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the CUDA library."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if _build.is_stale():                    # (a variant selected with build.use_library is built by its caller)
        path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with paper_2608_14205_b200/build.py")
    L = ctypes.CDLL(path)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
    L.fb_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(FbConfig), ctypes.c_int]
    L.fb_destroy.argtypes = [vp]
    L.fb_budget_ns.argtypes = [u64, u64]
    L.fb_budget_ns.restype = u64
    L.fb_swap_cost_ns.argtypes = [ctypes.POINTER(FbBudget), i32, i32]
    L.fb_swap_cost_ns.restype = u64
    L.fb_predict_load.argtypes = [vp, ctypes.POINTER(FbRouter), vp, i32, vp, vp, vp, vp]
    L.fb_plan_swaps.argtypes = [vp, vp, vp, ctypes.POINTER(FbBudget), i32, vp, vp, vp, vp, vp, vp]
    L.fb_predict_and_plan.argtypes = [vp, ctypes.POINTER(FbRouter), vp, i32, vp, ctypes.POINTER(FbBudget), i32,
                                      vp, vp, vp, vp, vp, vp, vp]
    L.fb_route_dispatch.argtypes = [vp, ctypes.POINTER(FbRouter), vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.fb_layer_step.argtypes = [vp, ctypes.POINTER(FbRouter), vp, vp, i32, vp, ctypes.POINTER(FbBudget), i32] \
        + [vp] * 14
    L.fb_layer_step.restype = ctypes.c_int
    L.fb_layer_step_host.argtypes = [vp, ctypes.POINTER(FbRouter), vp, vp, i32, vp, ctypes.POINTER(FbBudget), i32] \
        + [vp] * 14
    L.fb_predict_load_static.argtypes = [ctypes.POINTER(FbConfig), ctypes.c_int, ctypes.POINTER(FbRouter), vp, i32,
                                         vp, vp, vp, vp]
    L.fb_predict_load_static.restype = ctypes.c_int
    L.fb_device_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    L.fb_set_stage_limit.argtypes = [vp, i32]
    L.fb_set_stage_limit.restype = ctypes.c_int
    L.fb_set_pair_limit.argtypes = [vp, i32]
    L.fb_set_pair_limit.restype = ctypes.c_int
    L.fb_max_pairs.argtypes = [vp]
    L.fb_max_pairs.restype = i32
    L.fb_dispatch_slot_counts.argtypes = [vp, vp, vp, vp]
    L.fb_dispatch_slot_counts.restype = ctypes.c_int
    L.fb_dispatch_globalize.argtypes = [vp, i32, i32, i32] + [vp] * 9
    L.fb_dispatch_globalize.restype = ctypes.c_int
    L.fb_attention_begin.argtypes = [vp, i32, i32, vp]
    L.fb_attention_end.argtypes = [vp, i32, i32, vp]
    L.fb_layer_budget_ns.argtypes = [vp, i32, u64, ctypes.POINTER(u64), ctypes.POINTER(i32)]
    L.fb_attention_set_time_ns.argtypes = [vp, i32, i32, u64]
    L.fb_attention_reset.argtypes = [vp]
    for name in ("fb_attention_begin", "fb_attention_end", "fb_layer_budget_ns", "fb_attention_set_time_ns",
                 "fb_attention_reset"):
        getattr(L, name).restype = ctypes.c_int
    L.fb_set_split.argtypes = [vp, i32, i32]
    L.fb_set_split.restype = ctypes.c_int
    L.fb_standin_attention.argtypes = [vp, i32, i32, vp]
    L.fb_standin_attention.restype = ctypes.c_int
    L.fb_clock_probe.argtypes = [vp, i32, ctypes.c_uint32, vp]
    L.fb_clock_probe.restype = ctypes.c_int
    L.fb_set_stamp_buffer.argtypes = [vp, vp]
    L.fb_set_stamp_buffer.restype = ctypes.c_int
    L.fb_selftest_wait_timeout.argtypes = [vp, u64, vp, vp]
    L.fb_selftest_wait_timeout.restype = ctypes.c_int
    L.fb_row_cosine_mean.argtypes = [vp, vp, ctypes.c_int64, i32, i32, vp, vp, vp]
    L.fb_row_cosine_mean.restype = ctypes.c_int
    L.fb_topk_hits.argtypes = [vp, vp, i32, i32, vp, vp]
    L.fb_apply_swaps.argtypes = [vp, u64, i32, vp, vp, vp, i32, vp, vp]
    L.fb_apply_swaps.restype = ctypes.c_int
    L.fb_apply_swaps_staged.argtypes = [vp, vp, u64, vp, vp, vp, i32, u64, vp, vp]
    L.fb_apply_swaps_staged.restype = ctypes.c_int
    L.fb_fit_cost_model.argtypes = [u64, u64, u64, u64, ctypes.POINTER(u64), ctypes.POINTER(u64)]
    L.fb_fit_cost_model.restype = ctypes.c_int
    L.fb_calibrate_exchange.argtypes = [vp, u64, u64, i32] + [ctypes.POINTER(u64)] * 4 + [vp]
    L.fb_calibrate_exchange.restype = ctypes.c_int
    L.fb_topk_hits.restype = ctypes.c_int
    L.fb_router_floor.argtypes = [vp, ctypes.POINTER(FbRouter), vp, i32, i32, vp]
    L.fb_router_floor.restype = ctypes.c_int
    L.fb_time_next_router_launch.argtypes = [vp, vp, vp]
    L.fb_time_next_router_launch.restype = ctypes.c_int
    L.fb_persistent_launch_count.argtypes = [vp]
    L.fb_persistent_launch_count.restype = u64
    L.fb_launch_count.argtypes = [vp]
    L.fb_launch_count.restype = u64
    L.fb_status_string.argtypes = [ctypes.c_int]
    L.fb_status_string.restype = ctypes.c_char_p
    for name in ("fb_create", "fb_destroy", "fb_predict_load", "fb_plan_swaps", "fb_predict_and_plan",
                 "fb_route_dispatch", "fb_layer_step_host", "fb_device_status"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors handed to the library must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return stream or None


def _check(status: int, where: str) -> None:
    if status != FB_OK:
        raise FbError(status, where)


def make_budget(max_swaps=0, global_ns=_U64_OFF, rank_ns=_U64_OFF, link_ns=_U64_OFF, tau_tokens=0,
                gamma_num=0, gamma_den=1, alpha_ns=(0, 0), fs_per_byte=(0, 0), ranks_per_node=0,
                expert_bytes=0, expert_bytes_table: Optional[torch.Tensor] = None, mode=FB_PLAN_LOOP,
                frontier_width=1) -> FbBudget:
    b = FbBudget()
    b.max_swaps, b.global_ns, b.rank_ns, b.link_ns = max_swaps, global_ns, rank_ns, link_ns
    b.tau_tokens, b.gamma_num, b.gamma_den = tau_tokens, gamma_num, gamma_den
    b.alpha_ns = (ctypes.c_uint64 * 2)(*alpha_ns)
    b.fs_per_byte = (ctypes.c_uint64 * 2)(*fs_per_byte)
    b.ranks_per_node, b.expert_bytes = ranks_per_node, expert_bytes
    b.expert_bytes_table = _ptr(expert_bytes_table)
    b.mode, b.frontier_width = mode, frontier_width
    b._keepalive = expert_bytes_table
    return b


def make_router(W: torch.Tensor, logit_bias: Optional[torch.Tensor] = None,
                select_bias: Optional[torch.Tensor] = None) -> FbRouter:
    assert W.dtype == torch.bfloat16
    r = FbRouter(_ptr(W), _ptr(logit_bias), _ptr(select_bias))
    r._keepalive = (W, logit_bias, select_bias)
    return r


def fb_budget_ns(t_attn_ns: int, delta_ns: int) -> int:
    return int(lib().fb_budget_ns(t_attn_ns, delta_ns))


def fb_swap_cost_ns(budget: FbBudget, rank_a: int, rank_b: int) -> int:
    return int(lib().fb_swap_cost_ns(ctypes.byref(budget), rank_a, rank_b))


FB_DTYPE_BF16, FB_DTYPE_F32 = 0, 1


def fb_row_cosine_mean(a: torch.Tensor, b: torch.Tensor, row_scratch: torch.Tensor, mean_out: torch.Tensor,
                       stream=None) -> None:
    """a, b: [rows, n] bf16 or f32 device tensors; row_scratch: float64 [rows]; mean_out: float64 [1]."""
    assert a.shape == b.shape and a.dtype == b.dtype and a.dim() == 2
    assert row_scratch.dtype == torch.float64 and mean_out.dtype == torch.float64
    dtype = {torch.bfloat16: FB_DTYPE_BF16, torch.float32: FB_DTYPE_F32}[a.dtype]
    _check(lib().fb_row_cosine_mean(_ptr(a), _ptr(b), a.shape[0], a.shape[1], dtype, _ptr(row_scratch),
                                    _ptr(mean_out), _stream(stream)), "fb_row_cosine_mean")


def fb_fit_cost_model(t_small_ns: int, t_large_ns: int, bytes_small: int, bytes_large: int) -> tuple[int, int]:
    """(alpha_ns, fs_per_byte) of Eq. 9 from two timed exchanges; host arithmetic only."""
    a, f = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _check(lib().fb_fit_cost_model(t_small_ns, t_large_ns, bytes_small, bytes_large, ctypes.byref(a),
                                   ctypes.byref(f)), "fb_fit_cost_model")
    return int(a.value), int(f.value)


def fb_calibrate_exchange(slot_weights: torch.Tensor, bytes_small: int, bytes_large: int, reps: int = 5,
                          stream=None) -> dict:
    """Time two exchanges on the device and fit Eq. 9; returns alpha_ns, fs_per_byte and the timings."""
    vals = [ctypes.c_uint64(0) for _ in range(4)]
    _check(lib().fb_calibrate_exchange(_ptr(slot_weights), bytes_small, bytes_large, reps,
                                       *[ctypes.byref(v) for v in vals], _stream(stream)), "fb_calibrate_exchange")
    return dict(alpha_ns=int(vals[0].value), fs_per_byte=int(vals[1].value), t_small_ns=int(vals[2].value),
                t_large_ns=int(vals[3].value))


def fb_apply_swaps(slot_weights: torch.Tensor, expert_bytes: int, E: int, expert_to_slot: torch.Tensor,
                   swaps: torch.Tensor, n_swaps: torch.Tensor, max_swaps: int, status_word=None, stream=None) -> None:
    """Exchange the slot images of every accepted swap in place (stage 3 on one device)."""
    _check(lib().fb_apply_swaps(_ptr(slot_weights), expert_bytes, E, _ptr(expert_to_slot), _ptr(swaps),
                                _ptr(n_swaps), max_swaps, _ptr(status_word), _stream(stream)), "fb_apply_swaps")


def fb_topk_hits(ids_a: torch.Tensor, ids_b: torch.Tensor, T: int, k: int, hits_out: torch.Tensor,
                 stream=None) -> None:
    _check(lib().fb_topk_hits(_ptr(ids_a), _ptr(ids_b), T, k, _ptr(hits_out), _stream(stream)), "fb_topk_hits")


def fb_predict_load_static(cfg: FbConfig, device: int, router: FbRouter, x, T: int, counts, topk_ids=None,
                           status_word=None, stream=None) -> None:
    """Context-free prediction pass that allocates nothing (scratch lives in the library image)."""
    _check(lib().fb_predict_load_static(ctypes.byref(cfg), device, ctypes.byref(router), _ptr(x), T, _ptr(counts),
                                        _ptr(topk_ids), _ptr(status_word), _stream(stream)),
           "fb_predict_load_static")


def fb_standin_attention(out, blocks: int, iters: int, stream=None) -> None:
    """Compute-bound stand-in for attention on exactly `blocks` SMs (out: float32 [blocks * 1024])."""
    _check(lib().fb_standin_attention(_ptr(out), blocks, iters, _stream(stream)), "fb_standin_attention")


def fb_clock_probe(samples, n: int, period_ns: int, stream=None) -> None:
    """(global timer ns, SM cycle counter) pairs into `samples` (int64 [2 n]) from a one-thread kernel."""
    _check(lib().fb_clock_probe(_ptr(samples), n, period_ns, _stream(stream)), "fb_clock_probe")


class Context:
    """Owns an fb_ctx; methods mirror the C entry points one to one."""

    def __init__(self, T_max, d, E, k, R, gate=0, n_group=1, topk_group=1, renorm=1, route_scale=1.0,
                 device: int = 0):
        self.cfg = FbConfig(T_max, d, E, k, R, gate, n_group, topk_group, renorm, route_scale)
        self._h = ctypes.c_void_p()
        _check(lib().fb_create(ctypes.byref(self._h), ctypes.byref(self.cfg), device), "fb_create")
        self.device = device

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().fb_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def fb_predict_load(self, router, x, T, counts, topk_ids=None, logits=None, stream=None):
        _check(lib().fb_predict_load(self._h, ctypes.byref(router), _ptr(x), T, _ptr(counts), _ptr(topk_ids),
                                     _ptr(logits), _stream(stream)), "fb_predict_load")

    def fb_plan_swaps(self, counts, expert_to_slot, budget, layer_id, expert_to_slot_out, swaps, n_swaps,
                      load_before, load_after, stream=None):
        _check(lib().fb_plan_swaps(self._h, _ptr(counts), _ptr(expert_to_slot), ctypes.byref(budget), layer_id,
                                   _ptr(expert_to_slot_out), _ptr(swaps), _ptr(n_swaps), _ptr(load_before),
                                   _ptr(load_after), _stream(stream)), "fb_plan_swaps")

    def fb_predict_and_plan(self, router, x, T, expert_to_slot, budget, layer_id, counts, expert_to_slot_out,
                            swaps, n_swaps, load_before, load_after, stream=None):
        _check(lib().fb_predict_and_plan(self._h, ctypes.byref(router), _ptr(x), T, _ptr(expert_to_slot),
                                         ctypes.byref(budget), layer_id, _ptr(counts), _ptr(expert_to_slot_out),
                                         _ptr(swaps), _ptr(n_swaps), _ptr(load_before), _ptr(load_after),
                                         _stream(stream)), "fb_predict_and_plan")

    def fb_route_dispatch(self, router, x, T, expert_to_slot, topk_ids, topk_w, slot_offsets, rank_offsets,
                          perm, inv_perm, rank_load, logits=None, stream=None):
        _check(lib().fb_route_dispatch(self._h, ctypes.byref(router), _ptr(x), T, _ptr(expert_to_slot),
                                       _ptr(topk_ids), _ptr(topk_w), _ptr(slot_offsets), _ptr(rank_offsets),
                                       _ptr(perm), _ptr(inv_perm), _ptr(rank_load), _ptr(logits),
                                       _stream(stream)), "fb_route_dispatch")

    def fb_layer_step(self, router, h_prev, H, T, expert_to_slot, budget, layer_id, counts, expert_to_slot_out,
                      swaps, n_swaps, load_before, load_after, topk_ids, topk_w, slot_offsets, rank_offsets, perm,
                      inv_perm, rank_load, stream=None):
        outs = [counts, expert_to_slot_out, swaps, n_swaps, load_before, load_after, topk_ids, topk_w,
                slot_offsets, rank_offsets, perm, inv_perm, rank_load]
        _check(lib().fb_layer_step(self._h, ctypes.byref(router), _ptr(h_prev), _ptr(H), T, _ptr(expert_to_slot),
                                   ctypes.byref(budget), layer_id, *[_ptr(o) for o in outs], _stream(stream)),
               "fb_layer_step")

    def fb_layer_step_host(self, router, h_prev_host, H_host, T, expert_to_slot_host, budget, layer_id,
                           counts=None, expert_to_slot_out=None, swaps=None, n_swaps=None, load_before=None,
                           load_after=None, topk_ids=None, topk_w=None, slot_offsets=None, rank_offsets=None,
                           perm=None, inv_perm=None, rank_load=None, stream=None):
        outs = [counts, expert_to_slot_out, swaps, n_swaps, load_before, load_after, topk_ids, topk_w,
                slot_offsets, rank_offsets, perm, inv_perm, rank_load]
        _check(lib().fb_layer_step_host(self._h, ctypes.byref(router), _ptr(h_prev_host), _ptr(H_host), T,
                                        _ptr(expert_to_slot_host), ctypes.byref(budget), layer_id,
                                        *[_ptr(o) for o in outs], _stream(stream)), "fb_layer_step_host")

    def fb_device_status(self, stream=None) -> int:
        word = ctypes.c_int32(0)
        _check(lib().fb_device_status(self._h, ctypes.byref(word), _stream(stream)), "fb_device_status")
        return int(word.value)

    def fb_apply_swaps_staged(self, slot_weights, expert_bytes, expert_to_slot, swaps, n_swaps, max_swaps,
                              staging_bytes=0, plan_stream=None, copy_stream=None) -> None:
        _check(lib().fb_apply_swaps_staged(self._h, _ptr(slot_weights), expert_bytes, _ptr(expert_to_slot),
                                           _ptr(swaps), _ptr(n_swaps), max_swaps, staging_bytes,
                                           _stream(plan_stream), _stream(copy_stream)), "fb_apply_swaps_staged")

    def fb_set_pair_limit(self, pairs: int) -> None:
        _check(lib().fb_set_pair_limit(self._h, pairs), "fb_set_pair_limit")

    def fb_set_stage_limit(self, stages: int) -> None:
        _check(lib().fb_set_stage_limit(self._h, stages), "fb_set_stage_limit")

    def fb_set_split(self, mode: int, owner_bias_kblocks: int = -1) -> None:
        _check(lib().fb_set_split(self._h, mode, owner_bias_kblocks), "fb_set_split")

    def fb_max_pairs(self) -> int:
        return int(lib().fb_max_pairs(self._h))

    def fb_dispatch_slot_counts(self, slot_offsets, slot_counts, stream=None) -> None:
        _check(lib().fb_dispatch_slot_counts(self._h, _ptr(slot_offsets), _ptr(slot_counts), _stream(stream)),
               "fb_dispatch_slot_counts")

    def fb_dispatch_globalize(self, T_local, world, rank, slot_counts_all, slot_offsets_local, topk_ids,
                              expert_to_slot, inv_perm, slot_offsets, rank_offsets, rank_load, stream=None) -> None:
        _check(lib().fb_dispatch_globalize(self._h, T_local, world, rank, _ptr(slot_counts_all),
                                           _ptr(slot_offsets_local), _ptr(topk_ids), _ptr(expert_to_slot),
                                           _ptr(inv_perm), _ptr(slot_offsets), _ptr(rank_offsets), _ptr(rank_load),
                                           _stream(stream)), "fb_dispatch_globalize")

    def fb_attention_begin(self, layer_id: int, attn_type: int = 0, stream=None) -> None:
        _check(lib().fb_attention_begin(self._h, layer_id, attn_type, _stream(stream)), "fb_attention_begin")

    def fb_attention_end(self, layer_id: int, attn_type: int = 0, stream=None) -> None:
        _check(lib().fb_attention_end(self._h, layer_id, attn_type, _stream(stream)), "fb_attention_end")

    def fb_layer_budget_ns(self, attn_type: int, delta_ns: int):
        """(B_l of Eq. 10 for a layer of this attention type, the layer r(l) it was measured on)."""
        budget, layer = ctypes.c_uint64(0), ctypes.c_int32(-1)
        _check(lib().fb_layer_budget_ns(self._h, attn_type, delta_ns, ctypes.byref(budget), ctypes.byref(layer)),
               "fb_layer_budget_ns")
        return int(budget.value), int(layer.value)

    def fb_attention_set_time_ns(self, attn_type: int, layer_id: int, t_attn_ns: int) -> None:
        _check(lib().fb_attention_set_time_ns(self._h, attn_type, layer_id, t_attn_ns), "fb_attention_set_time_ns")

    def fb_attention_reset(self) -> None:
        _check(lib().fb_attention_reset(self._h), "fb_attention_reset")

    def fb_set_stamp_buffer(self, stamps) -> None:
        """Only libraries built with -DFB_TIMING accept this (see phase_timing.py)."""
        _check(lib().fb_set_stamp_buffer(self._h, _ptr(stamps)), "fb_set_stamp_buffer")

    def fb_selftest_wait_timeout(self, limit_ns: int, waited_ns=None, stream=None) -> None:
        _check(lib().fb_selftest_wait_timeout(self._h, limit_ns, _ptr(waited_ns), _stream(stream)),
               "fb_selftest_wait_timeout")

    def fb_router_floor(self, router, x, T: int, what: int, stream=None) -> None:
        _check(lib().fb_router_floor(self._h, ctypes.byref(router), _ptr(x), T, what, _stream(stream)),
               "fb_router_floor")

    def fb_time_next_router_launch(self, event_before, event_after) -> None:
        """torch.cuda.Event objects (created with enable_timing=True); either may be None."""
        def handle(ev):
            if ev is None:
                return None
            if not ev.cuda_event:          # torch creates the CUDA event lazily, on the first record
                ev.record()
            return ctypes.c_void_p(ev.cuda_event)
        _check(lib().fb_time_next_router_launch(self._h, handle(event_before), handle(event_after)),
               "fb_time_next_router_launch")

    def fb_persistent_launch_count(self) -> int:
        return int(lib().fb_persistent_launch_count(self._h))

    def fb_launch_count(self) -> int:
        return int(lib().fb_launch_count(self._h))
