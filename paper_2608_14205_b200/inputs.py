"""Seeded synthetic prefill workloads shaped like the paper's evaluation batches.

This module only draws random tensors. It contains none of the method's
arithmetic (no router product, no gating, no top-k, no planner, no dispatch),
so both the CUDA path and the CPU oracle may be fed from it without sharing
any code of the method itself.

The paper evaluates on long-context prefill batches (batch 16, up to 8K tokens
per sequence) of two MoE models (Evaluation, "Models" / "Configurations").
Those batches and model weights are not available here; the generators below
stand in for them:

* router weights ``W[e, :] = bf16(c_e * 0.02 * N(0, 1))`` where the column scale
  ``c_e`` injects per-layer expert popularity skew (a fixed x1.5 boost of two
  experts, or a Zipf law over a per-layer seeded permutation of the experts);
* residual hidden states ``h_prev[i, :] = bf16(mu_{c(i)} + N(0, 1))`` where, for
  the multi-task shapes, each of 16 contiguous sequences belongs to one of three
  task clusters whose mean ``mu_c`` pushes that cluster's own Zipf-popular
  experts (the workload-dependent shift of the paper's Figure 2);
* the normal router input ``H = bf16(h_prev + delta)`` with a per-token drift of
  exact relative norm ``rho`` (the small residual update of Eq. 1).

Everything is produced by ``torch`` CPU generators so the bits are identical on
every machine.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

GATE_SOFTMAX_TOPK = 0
GATE_SIGMOID_GROUP_TOPK = 1


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and recipe of one synthetic configuration."""
    name: str
    T: int                       # tokens in the prefill batch (paper: N)
    d: int                       # hidden size
    E: int                       # routed experts
    k: int                       # experts per token
    R: int                       # logical expert-parallel ranks
    layers: int
    gate: int = GATE_SOFTMAX_TOPK
    n_group: int = 1
    topk_group: int = 1
    renorm: int = 1
    route_scale: float = 1.0
    rho: float = 0.1             # ||delta|| / ||h|| per token
    skew: str = "boost2"         # "boost2" | "zipf" | "clusters"
    zipf_s: float = 1.0
    kappa: float = 0.5
    n_clusters: int = 0
    n_sequences: int = 16
    # planner budget (see the C header for the meaning of each field)
    max_swaps: int = 0
    global_ns: int = 2**64 - 1
    rank_ns: int = 2**64 - 1
    link_ns: int = 2**64 - 1
    alpha_ns: int = 0
    fs_per_byte: int = 0
    expert_bytes: int = 0
    ranks_per_node: int = 0      # 0 -> all ranks in one node

    @property
    def m(self) -> int:
        return self.E // self.R


WORKLOADS = {
    "tiny": Workload("tiny", T=512, d=1024, E=8, k=2, R=4, layers=2, rho=0.1,
                     skew="boost2", max_swaps=2),
    "mixtral": Workload("mixtral", T=4096, d=4096, E=8, k=2, R=8, layers=32, rho=0.1,
                        skew="zipf", zipf_s=1.2, max_swaps=1),
    "qwen3": Workload("qwen3", T=8192, d=2048, E=128, k=8, R=8, layers=48, rho=0.15,
                      skew="zipf", zipf_s=1.0, max_swaps=6, expert_bytes=9 * 2**20),
    # The same model at the batch the paper evaluates it on: 16 sequences of 8K tokens.
    "qwen3_b16": Workload("qwen3_b16", T=131072, d=2048, E=128, k=8, R=8, layers=48, rho=0.15,
                          skew="zipf", zipf_s=1.0, max_swaps=6, expert_bytes=9 * 2**20),
    # Budget from the cost model: a 0.5 ms window, 44 MB per expert, 900 GB/s
    # (1111 fs per byte) and 2 us of fixed overhead give 99 858 ns per swap, so
    # exactly five swaps fit.
    "dsv3": Workload("dsv3", T=16384, d=7168, E=256, k=8, R=32, layers=58, rho=0.1,
                     gate=GATE_SIGMOID_GROUP_TOPK, n_group=8, topk_group=4,
                     skew="clusters", zipf_s=1.1, n_clusters=3, max_swaps=128,
                     global_ns=500_000, rank_ns=500_000, link_ns=500_000,
                     alpha_ns=2000, fs_per_byte=1111, expert_bytes=44_040_192),
    "sweep32k": Workload("sweep32k", T=32768, d=7168, E=256, k=8, R=64, layers=58, rho=0.2,
                         gate=GATE_SIGMOID_GROUP_TOPK, n_group=8, topk_group=4,
                         skew="clusters", zipf_s=1.1, n_clusters=3, max_swaps=5),
    "sweep64k": Workload("sweep64k", T=65536, d=7168, E=256, k=8, R=64, layers=58, rho=0.2,
                         gate=GATE_SIGMOID_GROUP_TOPK, n_group=8, topk_group=4,
                         skew="clusters", zipf_s=1.1, n_clusters=3, max_swaps=5),
}


def _gen(seed: int, layer: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((seed * 1_000_003 + layer) * 101 + stream)
    return g


def _zipf_log_weights(E: int, s: float, g: torch.Generator) -> torch.Tensor:
    """ln w_e - mean(ln w) for w_e = rank_e^-s over a seeded permutation."""
    order = torch.randperm(E, generator=g)
    rank = torch.empty(E, dtype=torch.float64)
    rank[order] = torch.arange(1, E + 1, dtype=torch.float64)
    lw = -s * torch.log(rank)
    return lw - lw.mean()


@dataclasses.dataclass
class LayerInputs:
    """One layer's tensors; bf16 tensors are the exact bits both sides consume."""
    h_prev: torch.Tensor          # bf16 [T, d]   residual state entering the layer
    H: torch.Tensor               # bf16 [T, d]   normal router input
    W: torch.Tensor               # bf16 [E, d]   router weight, one row per expert
    select_bias: Optional[torch.Tensor]   # fp32 [E] or None
    logit_bias: Optional[torch.Tensor]    # fp32 [E] or None
    expert_to_slot: torch.Tensor  # int32 [E]     initial placement (contiguous)


def make_router(wl: Workload, layer: int, seed: int = 0) -> torch.Tensor:
    g = _gen(seed, layer, 1)
    W = torch.randn(wl.E, wl.d, generator=g, dtype=torch.float32) * 0.02
    if wl.skew == "boost2":
        order = torch.randperm(wl.E, generator=_gen(seed, layer, 2))
        c = torch.ones(wl.E)
        c[order[:2]] = 1.5
    elif wl.skew == "zipf":
        lw = _zipf_log_weights(wl.E, wl.zipf_s, _gen(seed, layer, 2))
        c = torch.exp(wl.kappa * lw).float()
    else:
        c = torch.ones(wl.E)
    return (W * c[:, None]).to(torch.bfloat16)


def make_layer(wl: Workload, layer: int = 0, seed: int = 0, T: Optional[int] = None,
               rho: Optional[float] = None, with_logit_bias: bool = False) -> LayerInputs:
    """Draw one layer of the workload. ``T`` and ``rho`` override the recipe's values."""
    T = wl.T if T is None else T
    rho = wl.rho if rho is None else rho
    W = make_router(wl, layer, seed)

    g = _gen(seed, layer, 3)
    h = torch.randn(T, wl.d, generator=g, dtype=torch.float32)
    if wl.skew == "clusters" and T > 0:
        # Each task cluster favours its own Zipf-ordered experts: its mean is the
        # combination of router rows that shifts expert e's logit by o[c, e].
        Wf = W.float()
        row_norm2 = (Wf * Wf).sum(dim=1).clamp_min(1e-12)
        gc = _gen(seed, layer, 4)
        mus = []
        for _ in range(wl.n_clusters):
            o = wl.kappa * _zipf_log_weights(wl.E, wl.zipf_s, gc).float()
            mus.append(((o / row_norm2)[:, None] * Wf).sum(dim=0))
        mus = torch.stack(mus)                                   # [C, d]
        n_seq = min(wl.n_sequences, T)
        seq_cluster = torch.randint(0, wl.n_clusters, (n_seq,), generator=gc)
        seq_of_token = (torch.arange(T) * n_seq) // T
        h += mus[seq_cluster[seq_of_token]]
    h_prev = h.to(torch.bfloat16)

    g = _gen(seed, layer, 5)
    u = torch.randn(T, wl.d, generator=g, dtype=torch.float32)
    hf = h_prev.float()
    scale = rho * hf.norm(dim=1, keepdim=True) / u.norm(dim=1, keepdim=True).clamp_min(1e-20)
    H = (hf + u * scale).to(torch.bfloat16)

    select_bias = None
    if wl.gate == GATE_SIGMOID_GROUP_TOPK:
        select_bias = 0.02 * torch.randn(wl.E, generator=_gen(seed, layer, 6), dtype=torch.float32)
    logit_bias = None
    if with_logit_bias:
        logit_bias = 0.05 * torch.randn(wl.E, generator=_gen(seed, layer, 7), dtype=torch.float32)
    return LayerInputs(h_prev=h_prev, H=H, W=W, select_bias=select_bias, logit_bias=logit_bias,
                       expert_to_slot=torch.arange(wl.E, dtype=torch.int32))


def make_step_layer(wl: Workload, layer: int, step: int, seed: int = 0, T: Optional[int] = None,
                    rho: Optional[float] = None, sys_drift: float = 0.0) -> LayerInputs:
    """One layer of one prefill step of a changing-task serving sequence.

    Stands in for the paper's "Mixed Tasks" workload, where every prefill step draws all of
    its requests from one task and the task changes from step to step: the router weights
    of a layer are those of ``make_layer`` (fixed across steps), every token of step
    ``step`` belongs to the single task cluster ``c(step)`` (a seeded sequence over the
    workload's clusters; shapes without clusters just get fresh noise per step), and the
    normal router input adds, on top of the per-token drift of relative norm ``rho``, the
    same systematic vector to every token: the combination of router rows that moves the
    logit of expert e by about ``sys_drift * o_e``, where ``o`` is a seeded, zero-mean Zipf
    log-weight vector of the layer (logits have a standard deviation of about
    ``0.02 * sqrt(d)``).  The early pass then mispredicts the aggregate counts and not only
    single tokens.
    """
    T = wl.T if T is None else T
    rho = wl.rho if rho is None else rho
    W = make_router(wl, layer, seed)
    Wf = W.float()
    row_norm2 = (Wf * Wf).sum(dim=1).clamp_min(1e-12)

    g = _gen(seed, layer, 1000 + 10 * step + 3)
    h = torch.randn(T, wl.d, generator=g, dtype=torch.float32)
    if wl.skew == "clusters" and T > 0:
        gc = _gen(seed, layer, 4)                     # the same cluster means as make_layer
        mus = []
        for _ in range(wl.n_clusters):
            o = wl.kappa * _zipf_log_weights(wl.E, wl.zipf_s, gc).float()
            mus.append(((o / row_norm2)[:, None] * Wf).sum(dim=0))
        task = int(torch.randint(0, wl.n_clusters, (1,), generator=_gen(seed, 0, 2000 + step)).item())
        h += mus[task]
    h_prev = h.to(torch.bfloat16)

    g = _gen(seed, layer, 1000 + 10 * step + 5)
    u = torch.randn(T, wl.d, generator=g, dtype=torch.float32)
    hf = h_prev.float()
    hn = hf.norm(dim=1, keepdim=True)
    Hf = hf + u * (rho * hn / u.norm(dim=1, keepdim=True).clamp_min(1e-20))
    if sys_drift != 0.0 and T > 0:
        o = _zipf_log_weights(wl.E, max(wl.zipf_s, 1.0), _gen(seed, layer, 9)).float()
        direction = ((o / row_norm2)[:, None] * Wf).sum(dim=0)
        Hf = Hf + sys_drift * direction[None, :]
    H = Hf.to(torch.bfloat16)

    select_bias = None
    if wl.gate == GATE_SIGMOID_GROUP_TOPK:
        select_bias = 0.02 * torch.randn(wl.E, generator=_gen(seed, layer, 6), dtype=torch.float32)
    return LayerInputs(h_prev=h_prev, H=H, W=W, select_bias=select_bias, logit_bias=None,
                       expert_to_slot=torch.arange(wl.E, dtype=torch.int32))


def random_counts(E: int, total: int, seed: int, zipf_s: float = 1.0) -> torch.Tensor:
    """A skewed expert count vector with a given sum, for planner-only tests."""
    g = _gen(seed, 0, 8)
    lw = _zipf_log_weights(E, zipf_s, g)
    p = torch.softmax(lw, dim=0)
    if total == 0:
        return torch.zeros(E, dtype=torch.int64)
    draws = torch.multinomial(p, total, replacement=True, generator=g)
    return torch.bincount(draws, minlength=E)


def random_placement(E: int, seed: int) -> torch.Tensor:
    """A seeded non-contiguous expert -> slot bijection."""
    return torch.randperm(E, generator=_gen(seed, 0, 9)).to(torch.int32)


def default_gamma(T: int, k: int, R: int) -> tuple[int, int]:
    """Rational weight of the variance term of the load objective: 1 / (2 * ceil(T k / R))."""
    return 1, max(1, 2 * math.ceil(T * k / R))
