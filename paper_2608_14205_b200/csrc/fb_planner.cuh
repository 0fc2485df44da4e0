// Budgeted greedy expert-swap planner (Algorithm 1 lines 2-8, Eqs. 6-9), run by one
// warp: either a stand-alone one-warp kernel or the tail of the router kernel, in the
// block that finished last.  Integer arithmetic only, so every rank that replays it on
// the same count vector gets the same plan.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/freebalance.h"
#include "fb_ptx.cuh"

namespace fb {

constexpr int kPlanThreads = 32;          // the stand-alone planner kernel is one warp
constexpr uint32_t kPlanBarrierId = 1;    // named barrier of the router kernel's epilogue warps

struct PlanParams {
  int32_t E, R;
  uint32_t max_swaps;
  uint64_t global_ns, rank_ns, link_ns;
  uint32_t tau_tokens;
  uint32_t gamma_num, gamma_den;
  uint64_t alpha_ns[2];
  uint64_t fs_per_byte[2];
  uint64_t uniform_cost_ns[2];          // Eq. 9 evaluated on the host for the uniform expert size
  uint64_t uniform_link_cap[2];         // link_ns / uniform_cost_ns: swaps one link can carry (host)
  int32_t ranks_per_node;
  int32_t mode;                         // fb_plan_mode
  int32_t frontier_width;               // FB_PLAN_WIDE: ranks taken from each end of the load order (1..4)
  const uint64_t* expert_bytes_table;   // device [E] or nullptr
  const int32_t* expert_to_slot;        // device [E]
  int32_t* expert_to_slot_out;          // device [E]
  fb_swap* swaps;                       // device [max_swaps]
  int32_t* n_swaps;                     // device [1]
  uint32_t* load_before;                // device [R]
  uint32_t* load_after;                 // device [R]
  unsigned long long* stamps;           // this block's 64 phase-stamp words (FB_TIMING builds) or nullptr
};

// Phase stamps of the planner (FB_TIMING builds only): 18 planner entered, 19 rank loads formed,
// 20 greedy loop left.
#ifdef FB_TIMING
#define FB_PLAN_STAMP(i)                                                                    \
  do {                                                                                      \
    if (p.stamps != nullptr && lane == 0) {                                                 \
      unsigned long long t_;                                                                \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                \
      p.stamps[i] = t_;                                                                     \
      p.stamps[32 + (i)] = static_cast<unsigned long long>(clock64());                      \
    }                                                                                       \
  } while (0)
#else
#define FB_PLAN_STAMP(i) do { } while (0)
#endif

struct PlanCandidate {
  long long benefit;                    // gamma_den * (Phi(L) - Phi(L')), > 0 when valid
  unsigned long long cost;              // C(s) in ns, >= 1
  int32_t a, b;                         // source and destination rank
  int32_t ea, eb;                       // ea < 0: no candidate
};

constexpr int kMaxFrontierWidth = 4;

struct PlanShared {
  uint32_t cnt[FB_MAX_EXPERTS];
  int32_t slot_of[FB_MAX_EXPERTS];       // expert -> slot (current placement)
  int32_t expert_at[FB_MAX_EXPERTS];     // slot -> expert
  uint8_t moved[FB_MAX_EXPERTS];
  // fast loop: one word per slot - bits 0..21 the count of the expert placed there, bits 22..29
  // that expert's id, bit 31 set once the expert has moved
  uint32_t slot_cnt[FB_MAX_EXPERTS];
  uint8_t cand_a[FB_MAX_EXPERTS];        // fast loop: candidate c pairs slot c / m of the heavy rank ...
  uint8_t cand_b[FB_MAX_EXPERTS];        // ... with slot c % m of the light rank
  uint8_t rank_of[FB_MAX_EXPERTS];       // expert -> rank under the placement as given
  uint8_t node_of[FB_MAX_RANKS];         // rank -> node (all 0 when every rank is in one node)
  uint32_t load[FB_MAX_RANKS];           // rank loads under the placement as given
  unsigned long long rank_spent[FB_MAX_RANKS];
  uint32_t link_key[FB_MAX_EXPERTS / 2]; // one entry per accepted swap
  unsigned long long link_cost[FB_MAX_EXPERTS / 2];
  int32_t bad;                           // the placement is not a bijection
  int32_t bad_range;                     // a count beyond the planner's range
  int32_t fast;                          // the fast loop ran: the placement is in slot_cnt, not in expert_at
};

constexpr uint32_t kSlotCountMask = (1u << 22) - 1;
constexpr uint32_t kSlotMoved = 1u << 31;
static_assert(FB_MAX_COUNT_SUM <= kSlotCountMask && FB_MAX_EXPERTS <= 256, "slot word layout");

// true if x is a better choice than y: larger benefit / cost, compared exactly as
// cross products in 128 bits; equal ratios -> smaller (a, b, ea, eb).
__device__ __forceinline__ bool plan_better(const PlanCandidate& x, const PlanCandidate& y) {
  if (x.ea < 0) return false;
  if (y.ea < 0) return true;
  const unsigned __int128 l = static_cast<unsigned __int128>(static_cast<unsigned long long>(x.benefit)) * y.cost;
  const unsigned __int128 r = static_cast<unsigned __int128>(static_cast<unsigned long long>(y.benefit)) * x.cost;
  if (l != r) return l > r;
  if (x.a != y.a) return x.a < y.a;
  if (x.b != y.b) return x.b < y.b;
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

// Load the placement into shared memory, invert it and check that it is a bijection.
// Called by `nthreads` threads (t = 0..nthreads-1); the caller synchronises afterwards.
// sh.bad must have been cleared and sh.expert_at filled with -1 beforehand.
__device__ __forceinline__ void plan_load_placement(const PlanParams& p, PlanShared& sh, int t, int nthreads) {
  for (int e = t; e < p.E; e += nthreads) {
    const int s = p.expert_to_slot[e];
    sh.slot_of[e] = s;
    sh.moved[e] = 0;
    if (s < 0 || s >= p.E) sh.bad = 1;
    else if (atomicExch(&sh.expert_at[s], e) != -1) sh.bad = 1;
  }
  const int m = p.E / p.R;
  for (int e = t; e < p.E; e += nthreads) {
    const int s = sh.slot_of[e];
    sh.rank_of[e] = static_cast<uint8_t>((s >= 0 && s < p.E) ? s / m : 0);
  }
  for (int r = t; r < p.R; r += nthreads)
    sh.node_of[r] = static_cast<uint8_t>(p.ranks_per_node > 0 ? r / p.ranks_per_node : 0);
  for (int c = t; c < FB_MAX_EXPERTS; c += nthreads) {
    sh.cand_a[c] = static_cast<uint8_t>(c / m);
    sh.cand_b[c] = static_cast<uint8_t>(c % m);
  }
}
__device__ __forceinline__ void plan_clear(PlanShared& sh, int t, int nthreads) {
  if (t == 0) { sh.bad = 0; sh.bad_range = 0; sh.fast = 0; }
  for (int e = t; e < FB_MAX_EXPERTS; e += nthreads) sh.expert_at[e] = -1;
  for (int r = t; r < FB_MAX_RANKS; r += nthreads) sh.load[r] = 0;
}

// The count of expert e arrives (any thread, once per expert, after plan_load_placement and a
// barrier; another barrier follows before the planner warp runs): it goes into the slot word
// of the expert's slot and into its rank's load (Algorithm 1 line 2).
__device__ __forceinline__ void plan_put_count(PlanShared& sh, int e, uint32_t c) {
  sh.cnt[e] = c;
  if (c > FB_MAX_COUNT_SUM) { sh.bad_range = 1; return; }
  if (sh.bad) return;
  sh.slot_cnt[sh.slot_of[e]] = c | static_cast<uint32_t>(e) << 22;
  atomicAdd(&sh.load[sh.rank_of[e]], c);
}

// The new placement (called by all those threads after the planner warp is done and a
// barrier): slot s holds the expert its slot word names (fast loop) or expert_at[s].  An
// unusable input keeps the placement as given.
__device__ __forceinline__ void plan_write_placement(const PlanParams& p, PlanShared& sh, int t, int nthreads) {
  if (sh.bad || sh.bad_range) {
    for (int e = t; e < p.E; e += nthreads) p.expert_to_slot_out[e] = p.expert_to_slot[e];
  } else if (sh.fast) {
    for (int sl = t; sl < p.E; sl += nthreads) p.expert_to_slot_out[(sh.slot_cnt[sl] >> 22) & 0xffu] = sl;
  } else {
    for (int sl = t; sl < p.E; sl += nthreads) p.expert_to_slot_out[sh.expert_at[sl]] = sl;
  }
}

// Greedy loop specialised for the common case: one cost per link class (no per-expert
// size table) and at most 256 candidate pairs per iteration (m <= 16), kPerLane fixed (slot,
// slot) pairs per lane.  One warp runs alone here, so what counts is the length of the
// dependent instruction chain of an iteration, not the instruction count: every load of an
// iteration is issued before the first result is needed, nothing branches on a loaded value
// until the candidates are evaluated, and the accepted pair's slots and counts come from the
// winning lane's registers by shuffle instead of a second trip through shared memory.  Same
// decisions as the general loop below; 32-bit arithmetic where the ranges allow (loads < 2^22).
// L0 / L1: this lane's rank loads (ranks lane and lane + 32, -1 if absent).
// k32: every benefit of the call is known to stay below 2^32 (the caller checks the bound
// gamma_den * Lmax + 2 gamma_num * Lmax^2 / 4 for the largest rank load Lmax, which no swap
// raises), so benefits are formed and compared in 32 bits and the winner needs two warp
// reductions instead of three plus a ballot.
// kSide: the per-rank or the per-link budget can bind.  With a uniform cost per link class
// a rank or a link is never charged more than the whole plan, so a side budget that starts at
// or above the global one (the usual case: all three start at the same B) can never stop a
// swap the global budget admits; the instance without them keeps no per-rank or per-link
// books at all.
template <int kPerLane, bool k32, bool kSide>
__device__ __forceinline__ uint32_t plan_loop_uniform(const PlanParams& p, PlanShared& sh, int lane,
                                                      int& L0, int& L1) {
  const int R = p.R, m = p.E / R, mm = m * m;
  const uint32_t full = 0xffffffffu;
  int cand_sa[kPerLane], cand_sb[kPerLane];                     // slot offsets inside the two ranks
  bool cand_ok[kPerLane];
#pragma unroll
  for (int t = 0; t < kPerLane; ++t) {
    cand_ok[t] = lane + 32 * t < mm;
    cand_sa[t] = cand_ok[t] ? sh.cand_a[lane + 32 * t] : 0;
    cand_sb[t] = cand_ok[t] ? sh.cand_b[lane + 32 * t] : 0;
  }
  const uint32_t gden = p.gamma_den ? p.gamma_den : 1u;
  const uint32_t gnum2 = p.gamma_den ? 2u * p.gamma_num : 0u;   // <= 2^21
  // loop invariants in registers (no access to the parameter block inside the loop)
  const unsigned long long cost0 = p.uniform_cost_ns[0], cost1 = p.uniform_cost_ns[1];
  const unsigned long long global_ns = p.global_ns, rank_ns = p.rank_ns;
  const bool global_on = global_ns != FB_BUDGET_OFF;
  const bool rank_on = kSide && rank_ns != FB_BUDGET_OFF, link_on = kSide && p.link_ns != FB_BUDGET_OFF;
  // A link is only ever charged one cost (its class's), so its budget is a swap count.
  const unsigned long long link_cap0 = p.uniform_link_cap[0], link_cap1 = p.uniform_link_cap[1];
  const uint32_t max_swaps = p.max_swaps, tau = p.tau_tokens;
  uint32_t my_links[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};   // lane i keeps the links of swaps i, i+32, ...
  unsigned long long global_spent = 0;
  uint32_t n = 0;
  __syncwarp();
  while (n < max_swaps) {
    // frontier (lowest index on ties): max of load<<6 | (63 - rank), min of load<<6 | rank
    const uint32_t h0 = L0 >= 0 ? (static_cast<uint32_t>(L0) << 6 | static_cast<uint32_t>(63 - lane)) : 0u;
    const uint32_t h1 = L1 >= 0 ? (static_cast<uint32_t>(L1) << 6 | static_cast<uint32_t>(31 - lane)) : 0u;
    const uint32_t l0 = L0 >= 0 ? (static_cast<uint32_t>(L0) << 6 | static_cast<uint32_t>(lane)) : 0xffffffffu;
    const uint32_t l1 = L1 >= 0 ? (static_cast<uint32_t>(L1) << 6 | static_cast<uint32_t>(lane + 32)) : 0xffffffffu;
    const uint32_t hi_key = __reduce_max_sync(full, h0 > h1 ? h0 : h1);
    const uint32_t lo_key = __reduce_min_sync(full, l0 < l1 ? l0 : l1);
    const int a = 63 - static_cast<int>(hi_key & 63u), b = static_cast<int>(lo_key & 63u);
    const int La = static_cast<int>(hi_key >> 6), Lb = static_cast<int>(lo_key >> 6);
    const int D = La - Lb;
    // ---- every load of the iteration, before anything depends on one
    const int base_a = a * m, base_b = b * m;
    uint32_t wa[kPerLane], wb[kPerLane];                           // slot words: count, expert, moved
#pragma unroll
    for (int t = 0; t < kPerLane; ++t) {
      wa[t] = sh.slot_cnt[base_a + cand_sa[t]];
      wb[t] = sh.slot_cnt[base_b + cand_sb[t]];
    }
    unsigned long long rs_a = 0, rs_b = 0;
    if (kSide) { rs_a = sh.rank_spent[a]; rs_b = sh.rank_spent[b]; }
    const int node_a = sh.node_of[a], node_b = sh.node_of[b];
    int m2l = 0;
    if (lane != a && lane != b && L0 > m2l) m2l = L0;
    if (lane + 32 != a && lane + 32 != b && L1 > m2l) m2l = L1;
    const int M2 = static_cast<int>(__reduce_max_sync(full, static_cast<uint32_t>(m2l)));
    // ---- budgets: the cost is the same for every pair of this iteration
    const int cls = node_a == node_b ? 0 : 1;
    const unsigned long long c_ns = cls ? cost1 : cost0;
    // link: the unordered rank pair inside a node, the unordered node pair across nodes
    const int ka = cls ? node_a : a, kb = cls ? node_b : b;
    const uint32_t lkey = static_cast<uint32_t>(cls) << 16 | static_cast<uint32_t>(ka < kb ? ka : kb) << 8 |
                          static_cast<uint32_t>(ka < kb ? kb : ka);
    bool stop = static_cast<uint32_t>(D) <= tau;
    stop = stop || (global_on && (c_ns > global_ns || global_spent > global_ns - c_ns));
    const unsigned long long rs = rs_a > rs_b ? rs_a : rs_b;
    stop = stop || (rank_on && (c_ns > rank_ns || rs > rank_ns - c_ns));
    if (link_on) {
      uint32_t used = 0;                                         // swaps already charged to this link
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (n > 32u * q) used += __popc(__ballot_sync(full, my_links[q] == lkey));    // n is the same in all lanes
      stop = stop || used >= (cls ? link_cap1 : link_cap0);
    }
    // ---- candidates of this lane: largest benefit, ties -> smallest (expert on a, expert on b)
    int src, ea, eb, sa, sb;
    uint32_t wwa, wwb;                                            // slot words of the accepted pair
    if (k32) {
      // One 64-bit key per candidate: benefit, then the complement of the pair (so that the
      // larger key is the better candidate), then the candidate's index in this lane.  The
      // candidates of a lane are independent of each other; only the maximum chains them.
      // Written stage by stage over all candidates (differences, bounds, benefits, keys) and reduced
      // by a tree, so that nothing but the data flow orders the instructions of different candidates.
      int dl[kPerLane];
      uint32_t ben[kPerLane];
      unsigned long long key[kPerLane];
#pragma unroll
      for (int t = 0; t < kPerLane; ++t)
        dl[t] = static_cast<int>(wa[t] & kSlotCountMask) - static_cast<int>(wb[t] & kSlotCountMask);   // tokens moved a -> b
#pragma unroll
      for (int t = 0; t < kPerLane; ++t) {
        int Mn = La - dl[t];                                      // Eq. 6
        if (Lb + dl[t] > Mn) Mn = Lb + dl[t];                     // Eq. 7
        if (M2 > Mn) Mn = M2;
        // gamma_den * (Phi(L) - Phi(L')), variance term 2 dlt (La - Lb - dlt).  It is positive only
        // for 0 < dlt < D, and inside that range both terms are non-negative.
        const bool usable = cand_ok[t] && ((wa[t] | wb[t]) >> 31) == 0 && dl[t] > 0 && dl[t] < D;   // neither expert moved yet
        const uint32_t b32 = gden * static_cast<uint32_t>(La - Mn) +
                             gnum2 * (static_cast<uint32_t>(dl[t]) * static_cast<uint32_t>(D - dl[t]));
        ben[t] = usable ? b32 : 0u;
      }
#pragma unroll
      for (int t = 0; t < kPerLane; ++t) {
        const uint32_t pair = ((wa[t] >> 22) & 0xffu) << 8 | ((wb[t] >> 22) & 0xffu);
        key[t] = static_cast<unsigned long long>(ben[t]) << 32 |
                 static_cast<unsigned long long>(0xffffu - pair) << 8 | static_cast<unsigned>(t);
      }
#pragma unroll
      for (int w = kPerLane / 2; w >= 1; w >>= 1)
#pragma unroll
        for (int t = 0; t < w; ++t) key[t] = key[t] > key[t + w] ? key[t] : key[t + w];
      const unsigned long long best_key = key[0];
      const uint32_t mine = static_cast<uint32_t>(best_key >> 32);
      const uint32_t top = __reduce_max_sync(full, mine);
      if (stop || top == 0) break;                                // Algorithm 1 lines 6-7
      // among the lanes that hold the top benefit: smallest pair, i.e. largest complement; the lane rides along
      const uint32_t low = static_cast<uint32_t>(best_key);      // complement of the pair << 8 | index
      const uint32_t win = __reduce_max_sync(full, mine == top ? ((low >> 8) << 5 | static_cast<uint32_t>(31 - lane)) : 0u);
      src = 31 - static_cast<int>(win & 31u);
      const uint32_t pair = 0xffffu - (win >> 5);
      ea = static_cast<int>(pair >> 8);
      eb = static_cast<int>(pair & 0xffu);
      // the winning lane's candidate index gives the slots; their words come from shared memory
      const int t_win = __shfl_sync(full, static_cast<int>(low & 0xffu), src);
      sa = base_a + sh.cand_a[src + 32 * t_win];
      sb = base_b + sh.cand_b[src + 32 * t_win];
      wwa = sh.slot_cnt[sa];
      wwb = sh.slot_cnt[sb];
    } else {
      unsigned long long best_ben = 0;
      uint32_t best_pair = 0xffffffffu, best_slots = 0, best_wa = 0, best_wb = 0;
#pragma unroll
      for (int t = 0; t < kPerLane; ++t) {
        const int dlt = static_cast<int>(wa[t] & kSlotCountMask) - static_cast<int>(wb[t] & kSlotCountMask);
        int Mn = La - dlt;
        if (Lb + dlt > Mn) Mn = Lb + dlt;
        if (M2 > Mn) Mn = M2;
        const bool usable = cand_ok[t] && ((wa[t] | wb[t]) >> 31) == 0 && dlt > 0 && dlt < D;
        const long long ben = static_cast<long long>(gden) * (La - Mn) +
                              static_cast<long long>(gnum2) * (static_cast<long long>(dlt) * (D - dlt));
        const unsigned long long ub = usable ? static_cast<unsigned long long>(ben) : 0ull;
        const uint32_t pair = ((wa[t] >> 22) & 0xffu) << 16 | ((wb[t] >> 22) & 0xffu);
        if (ub > best_ben || (ub == best_ben && ub > 0 && pair < best_pair)) {
          best_ben = ub; best_pair = pair; best_wa = wa[t]; best_wb = wb[t];
          best_slots = static_cast<uint32_t>(base_a + cand_sa[t]) << 16 | static_cast<uint32_t>(base_b + cand_sb[t]);
        }
      }
      const uint32_t top_hi = __reduce_max_sync(full, static_cast<uint32_t>(best_ben >> 32));
      const uint32_t top_lo = __reduce_max_sync(full, static_cast<uint32_t>(best_ben >> 32) == top_hi ? static_cast<uint32_t>(best_ben) : 0u);
      const unsigned long long top_ben = static_cast<unsigned long long>(top_hi) << 32 | top_lo;
      if (stop || top_ben == 0) break;                            // Algorithm 1 lines 6-7
      const uint32_t win = __reduce_min_sync(full, best_ben == top_ben ? best_pair : 0xffffffffu);
      src = __ffs(__ballot_sync(full, best_ben == top_ben && best_pair == win)) - 1;
      ea = static_cast<int>(win >> 16);
      eb = static_cast<int>(win & 0xffffu);
      // the lane that holds the accepted pair hands out its slots and slot words
      const uint32_t slots = __shfl_sync(full, best_slots, src);
      wwa = __shfl_sync(full, best_wa, src);
      wwb = __shfl_sync(full, best_wb, src);
      sa = static_cast<int>(slots >> 16);
      sb = static_cast<int>(slots & 0xffffu);
    }
    const int dlt = static_cast<int>(wwa & kSlotCountMask) - static_cast<int>(wwb & kSlotCountMask);
    if (lane == 0) {
      sh.slot_cnt[sa] = wwb | kSlotMoved; sh.slot_cnt[sb] = wwa | kSlotMoved;   // the two experts trade slots
      if (kSide) { sh.rank_spent[a] = rs_a + c_ns; sh.rank_spent[b] = rs_b + c_ns; }
      // The accepted swap stays in shared memory until the loop is over (ranks and expert ids
      // are below 256: one word; link_key is otherwise unused on this path): a global store
      // here would be waited for at the warp barrier below, once per iteration.
      sh.link_key[n] = static_cast<uint32_t>(a) << 24 | static_cast<uint32_t>(b) << 16 |
                       static_cast<uint32_t>(ea) << 8 | static_cast<uint32_t>(eb);
    }
    if (lane == a) L0 -= dlt;
    if (lane + 32 == a) L1 -= dlt;
    if (lane == b) L0 += dlt;
    if (lane + 32 == b) L1 += dlt;
    if (kSide && static_cast<int>(n & 31u) == lane) {
#pragma unroll
      for (int q = 0; q < 4; ++q) if (static_cast<int>(n >> 5) == q) my_links[q] = lkey;
    }
    global_spent += c_ns;
    ++n;
    __syncwarp();                                                 // the next iteration reads what lane 0 wrote
  }
  for (uint32_t i = lane; i < n; i += 32) {                       // the plan, in order of acceptance
    const uint32_t w = sh.link_key[i];
    fb_swap sw;
    sw.src_rank = static_cast<int32_t>(w >> 24); sw.dst_rank = static_cast<int32_t>((w >> 16) & 0xffu);
    sw.expert_src = static_cast<int32_t>((w >> 8) & 0xffu); sw.expert_dst = static_cast<int32_t>(w & 0xffu);
    p.swaps[i] = sw;
  }
  return n;
}

// Which plans the fast loop cannot serve (host and device agree on this test).
__host__ __device__ inline bool plan_needs_general_loop(const PlanParams& p) {
  return p.expert_bytes_table != nullptr || p.E / p.R > 16 || p.mode != FB_PLAN_LOOP;
}

// The general greedy loop: per-expert sizes, more than 16 experts per rank, or a planner
// variant (the one-pass sweep of the ordering paragraph, a widened frontier).  Plain and slow;
// a function of its own so that its registers and spills stay out of the common path.
// L0 / L1: this lane's rank loads (ranks lane and lane + 32, -1 if absent).
__device__ __noinline__ void plan_loop_general(const PlanParams& p, PlanShared& sh, int lane, long long L0,
                                               long long L1) {
  const int E = p.E, R = p.R, m = E / R;
  const uint32_t full = 0xffffffffu;
  const long long gnum = p.gamma_den ? p.gamma_num : 0;
  const long long gden = p.gamma_den ? p.gamma_den : 1;
  const int rpn = p.ranks_per_node;
  const bool uniform = p.expert_bytes_table == nullptr;     // one cost per link class
  const bool sweep = p.mode == FB_PLAN_SWEEP;
  int W = p.mode == FB_PLAN_WIDE ? p.frontier_width : 1;
  W = W < 1 ? 1 : (W > kMaxFrontierWidth ? kMaxFrontierWidth : W);
  if (W > R) W = R;
  const int mm = m * m;
  unsigned long long global_spent = 0;
  uint32_t n = 0;
  // the sweep scores every pair once, against the frontier and the loads of the placement as given
  int top[kMaxFrontierWidth], bot[kMaxFrontierWidth];
  long long Ltop[kMaxFrontierWidth], Lbot[kMaxFrontierWidth], other_max[kMaxFrontierWidth * kMaxFrontierWidth];
  while (n < p.max_swaps) {
    if (!sweep || n == 0) {
      // The W most and the W least loaded ranks, lowest index on ties, by repeated extraction.
      // Loads are below 2^22, so (load, rank) packs into 32 bits: max of load<<6 | (63 - rank),
      // min of load<<6 | rank.
      unsigned long long taken_hi = 0, taken_lo = 0;
#pragma unroll
      for (int w = 0; w < kMaxFrontierWidth; ++w) {
        if (w < W) {
          const bool f0 = L0 >= 0 && !((taken_hi >> lane) & 1ull), f1 = L1 >= 0 && !((taken_hi >> (lane + 32)) & 1ull);
          const uint32_t h0 = f0 ? (static_cast<uint32_t>(L0) << 6 | static_cast<uint32_t>(63 - lane)) : 0u;
          const uint32_t h1 = f1 ? (static_cast<uint32_t>(L1) << 6 | static_cast<uint32_t>(31 - lane)) : 0u;
          const uint32_t hi_key = __reduce_max_sync(full, h0 > h1 ? h0 : h1);
          top[w] = 63 - static_cast<int>(hi_key & 63u);
          Ltop[w] = hi_key >> 6;
          taken_hi |= 1ull << top[w];
          const bool g0 = L0 >= 0 && !((taken_lo >> lane) & 1ull), g1 = L1 >= 0 && !((taken_lo >> (lane + 32)) & 1ull);
          const uint32_t l0 = g0 ? (static_cast<uint32_t>(L0) << 6 | static_cast<uint32_t>(lane)) : 0xffffffffu;
          const uint32_t l1 = g1 ? (static_cast<uint32_t>(L1) << 6 | static_cast<uint32_t>(lane + 32)) : 0xffffffffu;
          const uint32_t lo_key = __reduce_min_sync(full, l0 < l1 ? l0 : l1);
          bot[w] = static_cast<int>(lo_key & 63u);
          Lbot[w] = lo_key >> 6;
          taken_lo |= 1ull << bot[w];
        }
      }
      // largest load among the ranks other than the two of a pair
#pragma unroll
      for (int wa = 0; wa < kMaxFrontierWidth; ++wa)
#pragma unroll
        for (int wb = 0; wb < kMaxFrontierWidth; ++wb)
          if (wa < W && wb < W) {
            const int a = top[wa], b = bot[wb];
            uint32_t o = 0;
            if (lane != a && lane != b && L0 > 0) o = static_cast<uint32_t>(L0);
            if (lane + 32 != a && lane + 32 != b && L1 > static_cast<long long>(o)) o = static_cast<uint32_t>(L1);
            other_max[wa * kMaxFrontierWidth + wb] = __reduce_max_sync(full, o);
          }
    }
    if (Ltop[0] - Lbot[0] <= static_cast<long long>(p.tau_tokens)) break;
    const long long M = Ltop[0];                                  // the maximum rank load
    PlanCandidate best;
    best.benefit = 0; best.cost = 1; best.a = -1; best.b = -1; best.ea = -1; best.eb = -1;
#pragma unroll
    for (int wa = 0; wa < kMaxFrontierWidth; ++wa) {
#pragma unroll
      for (int wb = 0; wb < kMaxFrontierWidth; ++wb) {
        if (wa >= W || wb >= W) continue;
        const int a = top[wa], b = bot[wb];
        const long long La = Ltop[wa], Lb = Lbot[wb];
        if (a == b || La <= Lb) continue;                         // a source carries strictly more than its destination
        const long long O = other_max[wa * kMaxFrontierWidth + wb];
        const int cls = (rpn <= 0 || a / rpn == b / rpn) ? 0 : 1;
        const int lo = a < b ? a : b, hi = a < b ? b : a;
        const uint32_t lkey = cls == 0 ? (static_cast<uint32_t>(lo) << 8 | static_cast<uint32_t>(hi))
                                       : (0x10000u | static_cast<uint32_t>(lo / rpn) << 8 | static_cast<uint32_t>(hi / rpn));
        unsigned long long link_spent = 0;
        if (p.link_ns != FB_BUDGET_OFF)
          for (uint32_t i = 0; i < n; ++i)
            if (sh.link_key[i] == lkey) link_spent += sh.link_cost[i];
        const unsigned long long rs_a = sh.rank_spent[a], rs_b = sh.rank_spent[b];
        const unsigned long long rank_spent = rs_a > rs_b ? rs_a : rs_b;
        const long long D = La - Lb;
        for (int c = lane; c < mm; c += 32) {
          const int ea = sh.expert_at[a * m + c / m];
          const int eb = sh.expert_at[b * m + c % m];
          if (sh.moved[ea] || sh.moved[eb]) continue;
          const long long dlt = static_cast<long long>(sh.cnt[ea]) - static_cast<long long>(sh.cnt[eb]);   // tokens moved a -> b
          long long Mn = La - dlt;                                // Eq. 6
          if (Lb + dlt > Mn) Mn = Lb + dlt;                       // Eq. 7
          if (O > Mn) Mn = O;
          // gamma_den * (Phi(L) - Phi(L')): the mean is unchanged by a swap, so the
          // variance term reduces to 2 dlt (La - Lb - dlt).
          const long long benefit = gden * (M - Mn) + 2 * gnum * (dlt * (D - dlt));
          if (benefit <= 0) continue;
          PlanCandidate cand;
          cand.benefit = benefit;
          cand.a = a; cand.b = b; cand.ea = ea; cand.eb = eb;
          cand.cost = uniform ? p.uniform_cost_ns[cls] : plan_cost_ns(p, cls, ea, eb);   // Eq. 9
          if (p.global_ns != FB_BUDGET_OFF && (cand.cost > p.global_ns || global_spent > p.global_ns - cand.cost)) continue;
          if (p.rank_ns != FB_BUDGET_OFF && (cand.cost > p.rank_ns || rank_spent > p.rank_ns - cand.cost)) continue;
          if (p.link_ns != FB_BUDGET_OFF && (cand.cost > p.link_ns || link_spent > p.link_ns - cand.cost)) continue;
          if (plan_better(cand, best)) best = cand;
        }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      PlanCandidate o;
      o.benefit = __shfl_xor_sync(full, best.benefit, off);
      o.cost = __shfl_xor_sync(full, best.cost, off);
      o.a = __shfl_xor_sync(full, best.a, off);
      o.b = __shfl_xor_sync(full, best.b, off);
      o.ea = __shfl_xor_sync(full, best.ea, off);
      o.eb = __shfl_xor_sync(full, best.eb, off);
      if (plan_better(o, best)) best = o;
    }
    if (best.ea < 0) break;                                     // Algorithm 1 lines 6-7
    const int a = best.a, b = best.b;
    const long long dlt = static_cast<long long>(sh.cnt[best.ea]) - static_cast<long long>(sh.cnt[best.eb]);
    const int cls = (rpn <= 0 || a / rpn == b / rpn) ? 0 : 1;
    const int lo = a < b ? a : b, hi = a < b ? b : a;
    const uint32_t lkey = cls == 0 ? (static_cast<uint32_t>(lo) << 8 | static_cast<uint32_t>(hi))
                                   : (0x10000u | static_cast<uint32_t>(lo / rpn) << 8 | static_cast<uint32_t>(hi / rpn));
    __syncwarp();                                               // all lanes are done reading the tables
    if (lane == 0) {
      const int sa = sh.slot_of[best.ea], sb = sh.slot_of[best.eb];
      sh.slot_of[best.ea] = sb; sh.slot_of[best.eb] = sa;
      sh.expert_at[sa] = best.eb; sh.expert_at[sb] = best.ea;
      sh.moved[best.ea] = 1; sh.moved[best.eb] = 1;
      sh.rank_spent[a] += best.cost; sh.rank_spent[b] += best.cost;
      sh.link_key[n] = lkey; sh.link_cost[n] = best.cost;
      fb_swap sw; sw.src_rank = a; sw.dst_rank = b; sw.expert_src = best.ea; sw.expert_dst = best.eb;
      p.swaps[n] = sw;
    }
    if (lane == a) L0 -= dlt;
    if (lane + 32 == a) L1 -= dlt;
    if (lane == b) L0 += dlt;
    if (lane + 32 == b) L1 += dlt;
    global_spent += best.cost;
    ++n;
    __syncwarp();
  }
  if (lane == 0) *p.n_swaps = static_cast<int32_t>(n);
  if (lane < R) p.load_after[lane] = static_cast<uint32_t>(L0);
  if (lane + 32 < R) p.load_after[lane + 32] = static_cast<uint32_t>(L1);
}

// The planner, run by ONE warp (all 32 lanes) once plan_load_placement has filled the
// placement arrays, sh.cnt holds the count vector and plan_scatter_counts has turned it into
// counts per slot.  A single warp keeps the rank loads in registers (lane r holds ranks r and
// r + 32) and needs no block barrier.  Writes the swaps, their number and the rank loads
// before and after; the new placement is written afterwards by plan_write_placement.
// kGeneral: the instance carries the general loop as well.  The router kernels' fused tail uses
// the instance without it (the host launches the stand-alone planner kernel behind the router
// kernel when a plan needs the general loop - see plan_needs_general_loop): the general loop's
// registers and code would otherwise weigh on every router kernel.
template <bool kGeneral>
__device__ __noinline__ void plan_swaps_warp(const PlanParams& p, PlanShared& sh, int lane, int* status) {
  const int E = p.E, R = p.R, m = E / R;
  const uint32_t full = 0xffffffffu;
  __syncwarp();
  FB_PLAN_STAMP(18);
  // ---- rank loads (Algorithm 1 line 2), formed by plan_put_count: lane holds L[lane] and
  // L[lane + 32]; their sum is checked against the planner's range
  const unsigned long long s0 = lane < R ? sh.load[lane] : 0u, s1 = lane + 32 < R ? sh.load[lane + 32] : 0u;
  const uint32_t total = __reduce_add_sync(full, static_cast<uint32_t>(s0 + s1));   // at most 256 counts of <= 2^21 each
  int bad = sh.bad ? 1 : ((sh.bad_range || total > FB_MAX_COUNT_SUM) ? 2 : 0);
  if (bad) {
    // Unusable input: report it, keep the placement as given, empty plan.
    if (lane == 0) {
      atomicCAS(status, 0, bad == 1 ? FB_ERR_BAD_PLACEMENT : FB_ERR_RANGE);
      *p.n_swaps = 0;
      sh.bad_range = 1;                          // plan_write_placement copies the input placement
    }
    for (int r = lane; r < R; r += 32) { p.load_before[r] = 0; p.load_after[r] = 0; }
    return;
  }
  long long L0 = -1, L1 = -1;                  // -1 marks "no such rank"
  if (lane < R) {
    L0 = static_cast<long long>(s0);
    p.load_before[lane] = static_cast<uint32_t>(s0);
    sh.rank_spent[lane] = 0;
  }
  if (lane + 32 < R) {
    L1 = static_cast<long long>(s1);
    p.load_before[lane + 32] = static_cast<uint32_t>(s1);
    sh.rank_spent[lane + 32] = 0;
  }
  __syncwarp();
  FB_PLAN_STAMP(19);

  if (!plan_needs_general_loop(p)) {
    int l0 = static_cast<int>(L0), l1 = static_cast<int>(L1);
    const int mm = m * m;
    // largest benefit any swap of this call can have (rank loads never exceed the initial maximum)
    const unsigned long long lmax = __reduce_max_sync(full, static_cast<uint32_t>(s0 > s1 ? s0 : s1));
    const unsigned long long bound = static_cast<unsigned long long>(p.gamma_den ? p.gamma_den : 1u) * lmax +
                                     (p.gamma_den ? 2ull * p.gamma_num : 0ull) * ((lmax * lmax) >> 2);
    const bool narrow = bound < (1ull << 32);
    // can the per-rank or the per-link budget stop a swap that the global budget admits?
    const bool side = (p.rank_ns != FB_BUDGET_OFF && !(p.global_ns != FB_BUDGET_OFF && p.rank_ns >= p.global_ns)) ||
                      (p.link_ns != FB_BUDGET_OFF && !(p.global_ns != FB_BUDGET_OFF && p.link_ns >= p.global_ns));
    uint32_t n_fast;
    if (lane == 0) sh.fast = 1;
    if (narrow && !side)
      n_fast = mm <= 32 ? plan_loop_uniform<1, true, false>(p, sh, lane, l0, l1)
               : mm <= 64 ? plan_loop_uniform<2, true, false>(p, sh, lane, l0, l1)
               : mm <= 128 ? plan_loop_uniform<4, true, false>(p, sh, lane, l0, l1)
                           : plan_loop_uniform<8, true, false>(p, sh, lane, l0, l1);
    else if (narrow)
      n_fast = mm <= 64 ? plan_loop_uniform<2, true, true>(p, sh, lane, l0, l1)
                        : plan_loop_uniform<8, true, true>(p, sh, lane, l0, l1);
    else
      n_fast = mm <= 64 ? plan_loop_uniform<2, false, true>(p, sh, lane, l0, l1)
                        : plan_loop_uniform<8, false, true>(p, sh, lane, l0, l1);
    FB_PLAN_STAMP(20);
    if (lane == 0) *p.n_swaps = static_cast<int32_t>(n_fast);
    if (lane < R) p.load_after[lane] = static_cast<uint32_t>(l0);
    if (lane + 32 < R) p.load_after[lane + 32] = static_cast<uint32_t>(l1);
    return;
  }
  if constexpr (kGeneral) {
    plan_loop_general(p, sh, lane, L0, L1);
  } else {
    // not reachable when the host follows plan_needs_general_loop; an empty plan otherwise
    if (lane == 0) *p.n_swaps = 0;
    if (lane < R) p.load_after[lane] = static_cast<uint32_t>(L0);
    if (lane + 32 < R) p.load_after[lane + 32] = static_cast<uint32_t>(L1);
  }
}


}  // namespace fb
