// Budgeted greedy expert-swap planner (Algorithm 1 lines 2-8, Eqs. 6-9) for one
// group of kPlanThreads threads: either a stand-alone one-block kernel or the tail of
// the router kernel, run by the block that finished last.  Integer arithmetic only, so
// every rank that replays it on the same count vector gets the same plan.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/freebalance.h"
#include "fb_ptx.cuh"

namespace fb {

constexpr int kPlanThreads = 128;
constexpr uint32_t kPlanBarrierId = 1;

struct PlanParams {
  int32_t E, R;
  uint32_t max_swaps;
  uint64_t global_ns, rank_ns, link_ns;
  uint32_t tau_tokens;
  uint32_t gamma_num, gamma_den;
  uint64_t alpha_ns[2];
  uint64_t fs_per_byte[2];
  uint64_t uniform_cost_ns[2];          // Eq. 9 evaluated on the host for the uniform expert size
  int32_t ranks_per_node;
  const uint64_t* expert_bytes_table;   // device [E] or nullptr
  const int32_t* expert_to_slot;        // device [E]
  int32_t* expert_to_slot_out;          // device [E]
  fb_swap* swaps;                       // device [max_swaps]
  int32_t* n_swaps;                     // device [1]
  uint32_t* load_before;                // device [R]
  uint32_t* load_after;                 // device [R]
};

struct PlanCandidate {
  long long benefit;                    // gamma_den * (Phi(L) - Phi(L')), > 0 when valid
  unsigned long long cost;              // C(s) in ns, >= 1
  int32_t ea, eb;                       // ea < 0: no candidate
};

struct PlanShared {
  uint32_t cnt[FB_MAX_EXPERTS];
  int32_t slot_of[FB_MAX_EXPERTS];       // expert -> slot (current placement)
  int32_t expert_at[FB_MAX_EXPERTS];     // slot -> expert
  uint8_t moved[FB_MAX_EXPERTS];
  uint32_t load[FB_MAX_RANKS];
  unsigned long long rank_spent[FB_MAX_RANKS];
  uint32_t link_key[FB_MAX_EXPERTS / 2]; // one entry per accepted swap
  unsigned long long link_cost[FB_MAX_EXPERTS / 2];
  PlanCandidate warp_best[kPlanThreads / 32];
  int32_t bad;
};

// true if x is a better choice than y: larger benefit / cost, compared exactly as
// cross products in 128 bits; equal ratios -> smaller (ea, eb).
__device__ __forceinline__ bool plan_better(const PlanCandidate& x, const PlanCandidate& y) {
  if (x.ea < 0) return false;
  if (y.ea < 0) return true;
  const unsigned __int128 l = static_cast<unsigned __int128>(static_cast<unsigned long long>(x.benefit)) * y.cost;
  const unsigned __int128 r = static_cast<unsigned __int128>(static_cast<unsigned long long>(y.benefit)) * x.cost;
  if (l != r) return l > r;
  if (x.ea != y.ea) return x.ea < y.ea;
  return x.eb < y.eb;
}

__device__ __forceinline__ unsigned long long plan_cost_ns(const PlanParams& p, int cls, int ea, int eb) {
  if (p.expert_bytes_table == nullptr) return p.uniform_cost_ns[cls];
  const unsigned __int128 bytes = static_cast<unsigned __int128>(p.expert_bytes_table[ea]) + p.expert_bytes_table[eb];
  const unsigned __int128 fs = bytes * p.fs_per_byte[cls];
  unsigned __int128 ns = (fs + 999999u) / 1000000u + p.alpha_ns[cls];
  if (ns > 0xFFFFFFFFFFFFFFFFull) ns = 0xFFFFFFFFFFFFFFFFull;
  const unsigned long long c = static_cast<unsigned long long>(ns);
  return c < 1 ? 1 : c;
}

// Called by exactly kPlanThreads threads with t = 0..kPlanThreads-1; sh.cnt must hold
// the count vector.  Synchronises with the named barrier kPlanBarrierId.
__device__ __noinline__ void plan_swaps_block(const PlanParams& p, PlanShared& sh, int t, int* status) {
  const int E = p.E, R = p.R, m = E / R;
  // ---- placement: load, invert, check that it is a bijection
  if (t == 0) sh.bad = 0;
  for (int e = t; e < E; e += kPlanThreads) { sh.expert_at[e] = -1; sh.moved[e] = 0; }
  for (int r = t; r < R; r += kPlanThreads) sh.rank_spent[r] = 0;
  named_bar_sync(kPlanBarrierId, kPlanThreads);
  for (int e = t; e < E; e += kPlanThreads) {
    const int s = p.expert_to_slot[e];
    sh.slot_of[e] = s;
    if (s < 0 || s >= E) sh.bad = 1;
    else if (atomicExch(&sh.expert_at[s], e) != -1) sh.bad = 1;
  }
  named_bar_sync(kPlanBarrierId, kPlanThreads);
  unsigned long long total = 0;
  if (t == 0) {
    for (int e = 0; e < E; ++e) total += sh.cnt[e];
    if (total > FB_MAX_COUNT_SUM) sh.bad = 2;
  }
  named_bar_sync(kPlanBarrierId, kPlanThreads);
  if (sh.bad) {
    // Unusable input: report it, keep the placement as given, empty plan.
    if (t == 0) {
      atomicCAS(status, 0, sh.bad == 1 ? FB_ERR_BAD_PLACEMENT : FB_ERR_RANGE);
      *p.n_swaps = 0;
    }
    for (int e = t; e < E; e += kPlanThreads) p.expert_to_slot_out[e] = p.expert_to_slot[e];
    for (int r = t; r < R; r += kPlanThreads) { p.load_before[r] = 0; p.load_after[r] = 0; }
    return;
  }
  // ---- rank loads (Algorithm 1 line 2)
  for (int r = t; r < R; r += kPlanThreads) {
    uint32_t s = 0;
    for (int j = 0; j < m; ++j) s += sh.cnt[sh.expert_at[r * m + j]];
    sh.load[r] = s;
    p.load_before[r] = s;
  }
  named_bar_sync(kPlanBarrierId, kPlanThreads);

  const long long gnum = p.gamma_den ? p.gamma_num : 0;
  const long long gden = p.gamma_den ? p.gamma_den : 1;
  unsigned long long global_spent = 0;
  uint32_t n = 0;
  while (n < p.max_swaps) {
    // frontier: most and least loaded rank, lowest index on ties (every thread computes it)
    int a = 0, b = 0;
    for (int r = 1; r < R; ++r) {
      if (sh.load[r] > sh.load[a]) a = r;
      if (sh.load[r] < sh.load[b]) b = r;
    }
    const long long La = sh.load[a], Lb = sh.load[b];
    if (La - Lb <= static_cast<long long>(p.tau_tokens)) break;
    long long M2 = 0;
    for (int r = 0; r < R; ++r)
      if (r != a && r != b && static_cast<long long>(sh.load[r]) > M2) M2 = sh.load[r];
    const int rpn = p.ranks_per_node;
    const int cls = (rpn <= 0 || a / rpn == b / rpn) ? 0 : 1;
    const int lo = a < b ? a : b, hi = a < b ? b : a;
    const uint32_t lkey = cls == 0 ? (static_cast<uint32_t>(lo) << 8 | static_cast<uint32_t>(hi))
                                   : (0x10000u | static_cast<uint32_t>(lo / rpn) << 8 | static_cast<uint32_t>(hi / rpn));
    unsigned long long link_spent = 0;
    for (uint32_t i = 0; i < n; ++i)
      if (sh.link_key[i] == lkey) link_spent += sh.link_cost[i];
    const unsigned long long rank_spent = sh.rank_spent[a] > sh.rank_spent[b] ? sh.rank_spent[a] : sh.rank_spent[b];

    PlanCandidate best;
    best.benefit = 0; best.cost = 1; best.ea = -1; best.eb = -1;
    for (int c = t; c < m * m; c += kPlanThreads) {
      const int ea = sh.expert_at[a * m + c / m];
      const int eb = sh.expert_at[b * m + c % m];
      if (sh.moved[ea] || sh.moved[eb]) continue;
      const long long dlt = static_cast<long long>(sh.cnt[ea]) - static_cast<long long>(sh.cnt[eb]);
      long long Mn = La - dlt;                                  // Eq. 6
      if (Lb + dlt > Mn) Mn = Lb + dlt;                         // Eq. 7
      if (M2 > Mn) Mn = M2;
      // gamma_den * (Phi(L) - Phi(L')): the mean is unchanged by a swap, so the
      // variance term reduces to 2 dlt (La - Lb - dlt).
      const long long benefit = gden * (La - Mn) + gnum * 2 * dlt * (La - Lb - dlt);
      if (benefit <= 0) continue;
      PlanCandidate cand;
      cand.benefit = benefit;
      cand.cost = plan_cost_ns(p, cls, ea, eb);                 // Eq. 9
      cand.ea = ea; cand.eb = eb;
      if (p.global_ns != FB_BUDGET_OFF && (cand.cost > p.global_ns || global_spent > p.global_ns - cand.cost)) continue;
      if (p.rank_ns != FB_BUDGET_OFF && (cand.cost > p.rank_ns || rank_spent > p.rank_ns - cand.cost)) continue;
      if (p.link_ns != FB_BUDGET_OFF && (cand.cost > p.link_ns || link_spent > p.link_ns - cand.cost)) continue;
      if (plan_better(cand, best)) best = cand;
    }
    // block arg-max
    for (int off = 16; off > 0; off >>= 1) {
      PlanCandidate o;
      o.benefit = __shfl_xor_sync(0xffffffffu, best.benefit, off);
      o.cost = __shfl_xor_sync(0xffffffffu, best.cost, off);
      o.ea = __shfl_xor_sync(0xffffffffu, best.ea, off);
      o.eb = __shfl_xor_sync(0xffffffffu, best.eb, off);
      if (plan_better(o, best)) best = o;
    }
    if ((t & 31) == 0) sh.warp_best[t >> 5] = best;
    named_bar_sync(kPlanBarrierId, kPlanThreads);
    best = sh.warp_best[0];
    for (int w = 1; w < kPlanThreads / 32; ++w)
      if (plan_better(sh.warp_best[w], best)) best = sh.warp_best[w];
    if (best.ea < 0) break;                                     // Algorithm 1 lines 6-7
    named_bar_sync(kPlanBarrierId, kPlanThreads);               // everyone has read warp_best / load
    if (t == 0) {
      const long long dlt = static_cast<long long>(sh.cnt[best.ea]) - static_cast<long long>(sh.cnt[best.eb]);
      sh.load[a] = static_cast<uint32_t>(La - dlt);
      sh.load[b] = static_cast<uint32_t>(Lb + dlt);
      const int sa = sh.slot_of[best.ea], sb = sh.slot_of[best.eb];
      sh.slot_of[best.ea] = sb; sh.slot_of[best.eb] = sa;
      sh.expert_at[sa] = best.eb; sh.expert_at[sb] = best.ea;
      sh.moved[best.ea] = 1; sh.moved[best.eb] = 1;
      sh.rank_spent[a] += best.cost; sh.rank_spent[b] += best.cost;
      sh.link_key[n] = lkey; sh.link_cost[n] = best.cost;
      fb_swap s; s.src_rank = a; s.dst_rank = b; s.expert_src = best.ea; s.expert_dst = best.eb;
      p.swaps[n] = s;
    }
    global_spent += best.cost;
    ++n;
    named_bar_sync(kPlanBarrierId, kPlanThreads);
  }
  if (t == 0) *p.n_swaps = static_cast<int32_t>(n);
  for (int e = t; e < E; e += kPlanThreads) p.expert_to_slot_out[e] = sh.slot_of[e];
  for (int r = t; r < R; r += kPlanThreads) p.load_after[r] = sh.load[r];
}

}  // namespace fb
