// Fused router kernel: logits = x W^T (+ b) on tcgen05 tensor cores with fp32
// accumulators in tensor memory, fed by TMA; then, straight out of tensor memory, the
// model's gating rule, top-k, and a per-expert histogram (Eqs. 2-5).  The block that
// finishes last publishes the count vector and, when asked, runs the swap planner.
//
// One block owns 128 token rows and all N = pad16(E) expert columns.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer for the even k-blocks (owns the
// TMEM allocation), warp 18 = MMA issuer for the odd k-blocks, warps 2..17 = epilogue.
// A thread that issues tcgen05.mma gets the next one accepted only ~175 cycles later,
// whatever the MMA's shape, which is slower than the tensor pipe and than the x stream
// from HBM; two issuing threads, each accumulating its own k-blocks into its own TMEM
// accumulator (columns [0, N) and [N, 2N)), remove that limit and keep the summation
// order fixed.  The epilogue adds the two accumulators.
// Epilogue warps:  A warp may only read the 32 TMEM lanes (token rows) selected
// by warp_id % 4, so the 16 epilogue warps form 4 "row quarters" x 4 "subs"; the subs of
// a quarter split the expert columns between them in 32-column chunks, one thread per
// token row, and sub 0 merges the partial results.
//
// Epilogue outline (after the accumulator is complete the pipeline's shared memory is
// idle and is reused as scratch):
//   pass 1  TMEM -> registers, 32 independent columns at a time: logit (+bias), selection
//           key (logit, or sigmoid + bias); keys are parked in shared memory; the sigmoid
//           gate also records each group's score (sum of its two largest keys).
//   choose  every thread picks its row's best groups and a lower bound for the k-th key.
//   pass 2  keys are re-read from shared memory; per chunk the few that can still enter
//           the top-k are compacted, then inserted (one insertion routine, rolled loops:
//           the code stays small enough for the instruction cache).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fb_planner.cuh"
#include "fb_ptx.cuh"

// Phase time stamps (builds with -DFB_TIMING only; see fb_set_stamp_buffer): one designated
// thread per role writes %globaltimer (slot i) and clock64 (slot 32 + i) of its block at the
// phase boundaries below.  Without the flag the macro is empty and the kernels carry none of it.
//   0 block start          1 set-up done            2 accumulators complete  3 keys computed
//   4 barrier              5 groups chosen          7 candidates collected   8 candidates ranked
//   9 top-k read back     10 outputs written       11 counts published      12 planner done
//  13 block exit          14 first load issued     15 last load issued      16 first operands landed
//  17 last MMA issued     18 planner entered       19 rank loads formed    20 greedy loop left
#ifdef FB_TIMING
#define FB_STAMP(i, who)                                                                    \
  do {                                                                                      \
    if (p.stamps != nullptr && threadIdx.x == (who)) {                                      \
      unsigned long long* st_ = p.stamps + static_cast<size_t>(blockIdx.x) * 64;           \
      st_[i] = global_timer_ns();                                                           \
      st_[32 + (i)] = static_cast<unsigned long long>(clock64());                           \
    }                                                                                       \
  } while (0)
#else
#define FB_STAMP(i, who) do { } while (0)
#endif

namespace fb {

constexpr int kTileM = 128;            // token rows per block
constexpr int kBlockK = 64;            // bf16 elements per k-block = one 128-byte swizzled row
constexpr int kUmmaK = 16;             // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxStages = 8;
constexpr int kEpiSubs = 4;            // epilogue warps per row quarter
constexpr int kEpilogueThreads = 128 * kEpiSubs;
constexpr int kRouterThreads = 64 + kEpilogueThreads + 32;
constexpr int kSecondIssuerWarp = kRouterThreads / 32 - 1;
constexpr int kATileBytes = kTileM * kBlockK * 2;
constexpr uint32_t kAccumBarrierId = 2;      // named barrier: accumulator finished (MMA warp -> epilogue warps)
constexpr uint32_t kRowBarrierBase = 3;      // named barriers 3..6: the kEpiSubs warps that share one quarter of the rows

enum RouterMode : int {
  kModePredict = 0,        // histogram -> counts
  kModePredictPlan = 1,    // histogram -> counts -> planner in the last block
  kModeDispatch = 2,       // ids, weights, per-tile histogram for the dispatch index
  kModeLayer = 3           // one launch for a whole layer: blocks [0, tiles_first) run the early pass
                           // (mode 1) on the first input, the others the normal pass (mode 2) on
                           // the second; the second wave of blocks fills the SMs the first frees
};

struct RouterParams {
  int32_t T, d, E, N, k;
  int32_t gate, n_group, topk_group, renorm;
  float route_scale;
  int32_t num_kb;                    // ceil(d / 64)
  int32_t stages;
  int32_t tmem_cols;                 // power of two >= max(32, 2 N): two accumulators
  int32_t mode;
  int32_t tiles_first;               // kModeLayer: blocks below this index (even) belong to the early pass
  int32_t ticket_target;             // number of blocks that take a ticket (those that publish counts)
  int32_t fuse_planner;              // prediction modes: the block that finishes last runs the planner
  const float* logit_bias;           // [E] or nullptr
  const float* select_bias;          // [E] or nullptr
  uint32_t* counts_scratch;          // [E] zero on entry, zero again on exit
  uint32_t* ticket;                  // zero on entry, zero again on exit
  int32_t* status;
  uint32_t* counts_out;              // [E]           (predict modes)
  int32_t* topk_ids;                 // [T][k] or nullptr
  float* topk_w;                     // [T][k] or nullptr
  float* logits;                     // [T][E] or nullptr
  uint32_t* tile_counts;             // [tiles][E]    (dispatch mode)
  unsigned long long* stamps;        // [blocks][64] phase time stamps (FB_TIMING builds) or nullptr
  int32_t probe;                     // measurement aid: 1 = operands are loaded but no MMA is issued and nothing
                                     // follows the main loop; 2 = with the MMAs, still nothing after them
  // k-range split (kSplit instances): the first 2 * split_helpers blocks are helper pairs, the
  // tiles' owners follow.  An owner accumulates k-blocks [0, split_ko) of its tile; the rest,
  // [split_ko, num_kb), is cut into split_j pieces, each summed by one helper pair (helper
  // t * split_j + j for piece j of tile pair t) into a partial tile in global memory that the
  // owner adds before its epilogue.
  int32_t split_helpers;             // helper pairs in the grid (0: no split)
  int32_t split_ko;                  // k-blocks an owner keeps
  int32_t split_j;                   // pieces per tile = helper pairs per tile pair
  uint32_t split_epoch;              // value a partial's flag takes when it is complete; the owner that has added
                                     // the partial puts the flag back to 0, so a launch starts from clean flags
                                     // whatever ran before it (a replayed graph included)
  float* split_partial;              // [slot][2 blocks][N columns][128 rows]
  uint32_t* split_flags;             // [slot][2 blocks]
  PlanParams plan;
};

struct TopK {
  float v[FB_MAX_TOPK];
  int32_t i[FB_MAX_TOPK];
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) { v[j] = -INFINITY; i[j] = 0; }
  }
  // Candidates arrive in ascending id order, so a strict comparison keeps the lower
  // id ahead of an equal key.
  __device__ __forceinline__ void insert(float x, int32_t id) {
    if (x > v[FB_MAX_TOPK - 1]) {
#pragma unroll
      for (int j = FB_MAX_TOPK - 1; j > 0; --j) {
        const bool above_prev = x > v[j - 1];
        const bool above_cur = x > v[j];
        v[j] = above_prev ? v[j - 1] : (above_cur ? x : v[j]);
        i[j] = above_prev ? i[j - 1] : (above_cur ? id : i[j]);
      }
      if (x > v[0]) { v[0] = x; i[0] = id; }
    }
  }
  // Same list, candidates in any order: equal keys are ordered by ascending id.
  __device__ __forceinline__ void insert_any_order(float x, int32_t id) {
    const bool enters = x > v[FB_MAX_TOPK - 1] || (x == v[FB_MAX_TOPK - 1] && id < i[FB_MAX_TOPK - 1]);
    if (enters) {
#pragma unroll
      for (int j = FB_MAX_TOPK - 1; j > 0; --j) {
        const bool above_prev = x > v[j - 1] || (x == v[j - 1] && id < i[j - 1]);
        const bool above_cur = x > v[j] || (x == v[j] && id < i[j]);
        v[j] = above_prev ? v[j - 1] : (above_cur ? x : v[j]);
        i[j] = above_prev ? i[j - 1] : (above_cur ? id : i[j]);
      }
      if (x > v[0] || (x == v[0] && id < i[0])) { v[0] = x; i[0] = id; }
    }
  }
};

// 1 / (1 + 2^(-z log2 e)) with the two hardware approximations (relative error ~1e-7).
// 2^x overflows to +inf for z < -88 and the reciprocal of +inf is 0, as it should be.
__device__ __forceinline__ float fb_sigmoid(float z) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(z * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return r;
}

// Shared-memory scratch of the epilogue (it reuses the pipeline stages): keys [N][128],
// group scores and group lower bounds [32][128] each, partial top-k lists of subs 1..,
// partial softmax sums.
constexpr int kCandCap = 32;           // candidates per row the fast selection path can hold
constexpr int kBoundRows = 8;          // chunks per row on that path, at most (rows of the bound tables)
__host__ __device__ constexpr size_t epilogue_scratch_bytes(int N) {
  return (static_cast<size_t>(N) * kTileM + 2 * FB_MAX_GROUPS * kTileM + 2 * kCandCap * kTileM) * 4;
}

static_assert(2 * kCandCap >= 2 * (kEpiSubs - 1) * FB_MAX_TOPK + kEpiSubs * 2, "merge area must fit in the candidate area");

// Which selection code a launch needs.  The ranking selection applies to DeepSeek-V3-like
// sigmoid gates (groups of exactly one 32-column chunk, at most 8 groups, at most kEpiSubs
// kept, two known keys per kept group >= k) and to softmax gates over whole chunks (every
// chunk counts as a kept group; not when the softmax denominator is needed, i.e. weights
// without renormalisation).  Everything else takes the general insertion code.
enum SelectKind : int { kSelectGeneral = 0, kSelectSigmoidRank = 1, kSelectSoftmaxRank = 2 };
__host__ __device__ inline int select_kind(int E, int N, int k, int gate, int n_group, int topk_group, bool want_sum) {
  if (gate != FB_GATE_SOFTMAX_TOPK)
    return (E / n_group == 32 && E % n_group == 0 && n_group <= 8 && topk_group <= kEpiSubs && topk_group * 2 >= k)
               ? kSelectSigmoidRank : kSelectGeneral;
  const int n_chunks = (N + 31) >> 5;
  return (E % 32 == 0 && n_chunks <= 8 && n_chunks * 2 >= k && !want_sum) ? kSelectSoftmaxRank : kSelectGeneral;
}

struct RouterShared {
  uint64_t full_bar[kMaxStages];
  uint64_t empty_bar[kMaxStages];
  uint64_t accum_bar;
  uint32_t tmem_base;
  int32_t abort_flag;
  int32_t is_last;
  int32_t accum_ok;
  int32_t issuer_progress[2];                // rings with an odd number of stages: see issuer_turn_wait
  float logit_bias[FB_MAX_EXPERTS + 32];     // + 32: a partial last chunk is read in full
  alignas(16) float select_bias[FB_MAX_EXPERTS + 32];
  uint32_t hist[FB_MAX_EXPERTS];
  uint32_t cand_count[kTileM];               // fast selection path: candidates claimed per row
  PlanShared plan;
};

// Order-preserving map of a float onto unsigned integers, and back.
__device__ __forceinline__ uint32_t ordered_bits(float x) {
  const uint32_t b = __float_as_uint(x);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t u) {
  return __uint_as_float(u ^ ((u >> 31) ? 0x80000000u : 0xffffffffu));
}

// The k-th largest of the known keys of a row: tab holds three tables of kBoundRows rows
// (each chunk's best, second and third key), of which the first n_chunks rows are valid
// (3 n_chunks >= k).  Counting instead of sorting: value v is the answer if at least k values
// are >= v and it is the largest such value; all comparisons are independent of each other.
template <int kRows>
__device__ __forceinline__ float kth_largest_of_tables(const float* tab, int n_chunks, int k, int row_in_tile) {
  float v[3 * kRows];
#pragma unroll
  for (int t = 0; t < 3; ++t)
#pragma unroll
    for (int c = 0; c < kRows; ++c)
      v[t * kRows + c] = c < n_chunks ? tab[(t * kBoundRows + c) * kTileM + row_in_tile] : -INFINITY;
  float best = -INFINITY;
#pragma unroll
  for (int i = 0; i < 3 * kRows; ++i) {
    int at_least = 0;
#pragma unroll
    for (int j = 0; j < 3 * kRows; ++j) at_least += v[j] >= v[i] ? 1 : 0;
    if (at_least >= k) best = fmaxf(best, v[i]);
  }
  return best;
}
__device__ __forceinline__ float kth_largest_known(const float* tab, int n_chunks, int k, int row_in_tile) {
  return n_chunks <= 4 ? kth_largest_of_tables<4>(tab, n_chunks, k, row_in_tile)
                       : kth_largest_of_tables<kBoundRows>(tab, n_chunks, k, row_in_tile);
}

// Ranking selection, shared by both router kernels.  cand[c * 128 + row] holds candidate c of
// the row as one 64-bit word: ordered key bits in the high half, ~expert id in the low half,
// so that "larger word" means "larger key, then lower id".  The kEpiSubs threads of a row
// share the candidates (candidate c belongs to thread c % kEpiSubs); a candidate with fewer
// than FB_MAX_TOPK larger ones is written to out_hi/out_lo[rank][row].  Returns true when
// the row had more candidates than the list holds (nothing is written for it then).
__device__ __forceinline__ bool rank_candidates(const unsigned long long* cand, uint32_t n_all, int sub,
                                                int row_in_tile, uint32_t* out_hi, uint32_t* out_lo) {
  const bool overflow = n_all > kCandCap;
  const uint32_t n = overflow ? 0u : n_all;
  const uint32_t n_most = __reduce_max_sync(0xffffffffu, n);
#pragma unroll 1
  for (uint32_t tier = 0; tier * 4 * kEpiSubs < n_most; ++tier) {
    unsigned long long mykey[4];
    uint32_t rank[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const uint32_t c = (tier * 4 + t) * kEpiSubs + sub;
      mykey[t] = cand[(c < n ? c : 0) * kTileM + row_in_tile];
      rank[t] = 0;
    }
#pragma unroll 2
    for (uint32_t d = 0; d < n_most; ++d) {
      const unsigned long long other = d < n ? cand[d * kTileM + row_in_tile] : 0ull;
#pragma unroll
      for (int t = 0; t < 4; ++t) rank[t] += other > mykey[t] ? 1u : 0u;
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const uint32_t c = (tier * 4 + t) * kEpiSubs + sub;
      if (c < n && rank[t] < static_cast<uint32_t>(FB_MAX_TOPK)) {
        out_hi[rank[t] * kTileM + row_in_tile] = static_cast<uint32_t>(mykey[t] >> 32);
        out_lo[rank[t] * kTileM + row_in_tile] = static_cast<uint32_t>(mykey[t]);
      }
    }
  }
  return overflow;
}

// The row's top-k list as rank_candidates left it.
__device__ __forceinline__ void read_ranked(TopK& top, int k, const uint32_t* out_hi, const uint32_t* out_lo,
                                            int row_in_tile) {
#pragma unroll
  for (int j = 0; j < FB_MAX_TOPK; ++j) {
    if (j < k) {
      top.v[j] = from_ordered_bits(out_hi[j * kTileM + row_in_tile]);
      top.i[j] = static_cast<int32_t>(~out_lo[j * kTileM + row_in_tile]);
    }
  }
}

// Expert ids and routing weights of one token (Eq. 3's top-k with the model's weight rule).
// select_bias_s: the selection bias in shared memory; sm_max / sm_sum: the row's softmax
// denominator in the form sum * exp(max), used only by softmax gates without renormalisation.
__device__ __forceinline__ void write_row_outputs(const TopK& top, const RouterParams& p, long long row,
                                                  int32_t* out_ids, float* out_w, const float* select_bias_s,
                                                  float sm_max, float sm_sum) {
  const int k = p.k;
  const bool sigmoid_gate = p.gate != FB_GATE_SOFTMAX_TOPK;
#ifdef FB_DEBUG
  // what the sanitizer would catch: a chosen expert outside [0, E), a repeated expert, a row outside [0, T)
  {
    bool bad = row < 0 || row >= p.T;
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) {
      if (j < k) {
        bad = bad || top.i[j] < 0 || top.i[j] >= p.E;
#pragma unroll
        for (int h = 0; h < FB_MAX_TOPK; ++h) bad = bad || (h < j && top.i[h] == top.i[j]);
      }
    }
    if (bad) atomicCAS(p.status, 0, FB_ERR_INTERNAL);
  }
#endif
  if (out_ids != nullptr) {
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j)
      if (j < k) out_ids[row * k + j] = top.i[j];
  }
  if (out_w != nullptr) {
    float w[FB_MAX_TOPK];
    float wsum = 0.0f;
    const float ref = top.v[0];                         // row maximum of the keys
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) {
      if (!sigmoid_gate) w[j] = (j < k) ? __expf(top.v[j] - ref) : 0.0f;
      else w[j] = (j < k) ? top.v[j] - select_bias_s[top.i[j]] : 0.0f;   // unbiased sigmoid score
      wsum += w[j];
    }
    float scale;
    if (!sigmoid_gate) scale = p.renorm ? 1.0f / wsum : 1.0f / (sm_sum * __expf(sm_max - ref));
    else scale = p.renorm ? p.route_scale / wsum : p.route_scale;
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j)
      if (j < k) out_w[row * k + j] = w[j] * scale;
  }
}

// End of a tile in the prediction modes: add the tile's histogram (shared memory, cleared
// here) to the cross-block counts, take a ticket, and in the block that takes the last one
// publish the count vector (Eq. 5), re-arm the scratch for the next call and run the planner
// (Algorithm 1) when asked.  Called by all epilogue threads; et = thread index among them.
template <class Shared>
__device__ __forceinline__ void publish_counts(Shared& sh, const RouterParams& p, int et, int warp, int lane,
                                               bool run_planner) {
  for (int e = et; e < p.E; e += kEpilogueThreads) {
    const uint32_t c = sh.hist[e];
    if (c) atomicAdd(&p.counts_scratch[e], c);
    sh.hist[e] = 0;
  }
  named_bar_sync(kPlanBarrierId, kEpilogueThreads);
  if (et == 0) {
    // The barrier orders every thread's histogram atomics before this fence, and the
    // fence (cumulative) publishes them device-wide before the ticket is taken.
    __threadfence();
    const uint32_t prev = atomicAdd(p.ticket, 1u);
    const bool last = prev == static_cast<uint32_t>(p.ticket_target) - 1;
    // Acquire side of the same hand-shake: the other blocks' counts are visible to this thread
    // after the fence and, through the barrier below, to the whole block.
    if (last) __threadfence();
    sh.is_last = last ? 1 : 0;
  }
  named_bar_sync(kPlanBarrierId, kEpilogueThreads);
  FB_STAMP(11, 64);
  if (sh.is_last) {
    // Every other tile has published its counts: this block finishes the pass.
    for (int e = et; e < p.E; e += kEpilogueThreads) {
      const uint32_t c = __ldcg(&p.counts_scratch[e]);
      p.counts_out[e] = c;
      if (run_planner) plan_put_count(sh.plan, e, c);
      p.counts_scratch[e] = 0;           // ready for the next call
    }
    if (et == 0) *p.ticket = 0;
    if (sh.abort_flag) { if (et == 0) atomicCAS(p.status, 0, FB_ERR_TIMEOUT); }
    if (run_planner) {
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      if (warp == 2) {
#ifdef FB_TIMING
        PlanParams pt = p.plan;
        pt.stamps = p.stamps != nullptr ? p.stamps + static_cast<size_t>(blockIdx.x) * 64 : nullptr;
        plan_swaps_warp<false>(pt, sh.plan, lane, p.status);
#else
        plan_swaps_warp<false>(p.plan, sh.plan, lane, p.status);
#endif
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      plan_write_placement(p.plan, sh.plan, et, kEpilogueThreads);
    }
  }
}

// Load columns [c0, c0 + 32) (or 16 when fewer remain) of this warp's 32 rows.
__device__ __forceinline__ void load_chunk(uint32_t taddr, int c0, int N, uint32_t (&r)[32]) {
  if (N - c0 >= 32) tmem_ld_32x32b_x32(taddr + c0, r);
  else tmem_ld_32x32b_x16(taddr + c0, r);
  tmem_ld_wait();
}

// Wait until a partial's flag holds the "complete" value (bounded like every other wait).
__device__ __forceinline__ bool flag_wait(const uint32_t* flag, uint32_t epoch, volatile int* abort_flag) {
  uint32_t polls = 0;
  uint64_t t0 = 0;
  for (;;) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v == epoch) return true;
    if ((++polls & 0x3Fu) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

// Two MMA issuers share one ring of stages.  With an even number of stages a stage always serves
// the same issuer, which therefore sees every phase of the stage's "full" barrier.  With an odd
// number a stage alternates between them, and a parity wait alone cannot tell "the other issuer's
// use of this stage is still being filled" (a wait for my parity passes on the phase before it)
// from "my use is complete".  So each issuer publishes the ring position of the last k-block whose
// operands it has seen arrive, and before it waits for position g on a stage whose previous use
// (position g - stages) was the other issuer's, it waits until the other one has got that far.
__device__ __forceinline__ bool issuer_turn_wait(const volatile int32_t* other_progress, int32_t need,
                                                 volatile int* abort_flag) {
  uint32_t polls = 0;
  uint64_t t0 = 0;
  while (*other_progress < need) {
    if ((++polls & 0x3Fu) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
  return true;
}

// Offset (in floats) of column `col`, row 0 of the partial tile that block `cta` of a pair owns in `slot`.
__device__ __forceinline__ size_t partial_offset(int slot, uint32_t cta, int N, int col) {
  return ((static_cast<size_t>(slot) * 2 + cta) * static_cast<size_t>(N) + static_cast<size_t>(col)) * kTileM;
}

// kCtas == 1: every block computes its 128 x N tile alone.
// kCtas == 2: launched in clusters of two; the pair shares one 256 x N MMA
// (tcgen05 cta_group::2).  Each block still loads its own 128 rows of x, but only half
// of the W tile, which halves the W traffic out of L2 and leaves room for more pipeline
// stages.  The even block of the pair issues the MMAs and owns the "full" barriers;
// both blocks get their stage-free and accumulator-ready signals from its commits.
// kSel (SelectKind): one instance per selection code, so that each carries only the code and
// the registers its gate needs; the host picks it with select_kind().
// kLogitBias: whether a logit bias (Eq. 2's "+ b") is given; without it the key computation
// shrinks to one variant.
// kSplit (pairs only): the grid has more block pairs than the call has tile pairs, and the spare
// pairs take the tail of every tile's k-range (see RouterParams).  A tile that fills one SM
// pair for the whole main loop leaves the spare SMs' tensor cores idle otherwise (128 tiles on
// 148 SMs; 64 tiles on 148 SMs for the smaller shapes).  The split is a function of the shape
// and of the number of pairs only, so a call's result is reproducible; its logits differ from
// the unsplit kernel's in the order of the fp32 additions.
template <int kCtas, int kSel, bool kLogitBias, bool kSplit = false>
__global__ void __launch_bounds__(kRouterThreads, 1)
fb_router_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_x2,
                 const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ RouterParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ RouterShared sh;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // kModeLayer: which pass this block belongs to, its tile there and its input
  const bool is_helper = kSplit && static_cast<int>(blockIdx.x) < 2 * p.split_helpers;
  const int owner_block = kSplit ? static_cast<int>(blockIdx.x) - 2 * p.split_helpers : static_cast<int>(blockIdx.x);
  const bool second_pass = p.mode == kModeLayer && !is_helper && owner_block >= p.tiles_first;
  const int mode = p.mode == kModeLayer ? (second_pass ? kModeDispatch : kModePredictPlan) : p.mode;
  const int tile = second_pass ? owner_block - p.tiles_first : owner_block;
  const int kb_end = kSplit ? p.split_ko : p.num_kb;        // k-blocks this block accumulates for its own tile
  const CUtensorMap* xmap = second_pass ? &tmap_x2 : &tmap_x;
  // outputs of the normal pass are not written by blocks of the early pass
  int32_t* const out_ids = (p.mode == kModeLayer && !second_pass) ? nullptr : p.topk_ids;
  float* const out_w = (p.mode == kModeLayer && !second_pass) ? nullptr : p.topk_w;
  const uint32_t cta_rank = kCtas == 2 ? cluster_ctarank() : 0u;
  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.N / kCtas) * kBlockK * 2;
  const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle atoms need 1024-byte alignment
  volatile int* abort_flag = &sh.abort_flag;
  FB_STAMP(0, 64);

  if (threadIdx.x == 0) {
    sh.abort_flag = 0;
    sh.is_last = 0;
    sh.issuer_progress[0] = -1;
    sh.issuer_progress[1] = -1;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&sh.full_bar[s]), 1);
      mbar_init(smem_u32(&sh.empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&sh.accum_bar), 2);                 // one commit per MMA issuer
    fence_mbar_init();
    prefetch_tensormap(xmap);
    prefetch_tensormap(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc<kCtas>(smem_u32(&sh.tmem_base), static_cast<uint32_t>(p.tmem_cols));
    tmem_relinquish<kCtas>();
  }
  if (warp >= 2) {
    const int et = threadIdx.x - 64;
    for (int e = et; e < FB_MAX_EXPERTS + 32; e += kEpilogueThreads) {
      if (e < FB_MAX_EXPERTS) sh.hist[e] = 0;
      if (e < kTileM) sh.cand_count[e] = 0;
    }
    if (mode == kModePredictPlan) plan_clear(sh.plan, et, kEpilogueThreads);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (kCtas == 2) { cluster_arrive(); cluster_wait(); }   // the partner's barriers and TMEM are ready too
  tcgen05_fence_after();
  // Everything above touched only this block's own state and the call's parameters; from here on
  // the kernel reads memory that earlier work of the stream may have written.
  pdl_wait();
  // From here on the next kernel of the stream may be scheduled (if it was launched with
  // programmatic stream serialization - the library's own router launches are): its blocks
  // take the SMs as this grid's blocks leave them and do their set-up while the last blocks
  // of this grid finish; they read nothing before their own griddepcontrol.wait, which returns
  // only when this grid has completed.  Issued after this block's wait, so a dependent never
  // starts before everything this grid itself depended on is complete.
  pdl_launch_dependents();
  const uint32_t tmem_base = sh.tmem_base;
  FB_STAMP(1, 64);

  if (is_helper) {
    // ============================================================ helper pair (kSplit instances)
    // Helper pair hp sums piece j = hp % split_j of the remaining k-blocks [split_ko, num_kb) of
    // tile pair t = hp / split_j into the partial tile of slot hp.  Even / odd k-blocks of the
    // piece go to the two issuers' accumulators as in an owner.
    const int hp = static_cast<int>(blockIdx.x) >> 1;
    const int rest = p.num_kb - p.split_ko;
    const int tp = hp / p.split_j, piece = hp % p.split_j;
    const int kb0 = p.split_ko + rest * piece / p.split_j, kb1 = p.split_ko + rest * (piece + 1) / p.split_j;
    // (tile pairs are numbered over both passes of a layer launch; a pair never straddles them)
    const int pair_tile = 2 * tp + static_cast<int>(cta_rank);
    const bool helps_second = p.mode == kModeLayer && pair_tile >= p.tiles_first;
    const int my_tile = helps_second ? pair_tile - p.tiles_first : pair_tile;
    const CUtensorMap* hmap = helps_second ? &tmap_x2 : &tmap_x;
    if (warp == 0) {
      // ---------------------------------------------------------- TMA producer
      if (lane == 0) {
        const uint64_t pol_x = l2_policy_evict_first();
        const uint64_t pol_w = l2_policy_evict_last();
        for (int kb = kb0; kb < kb1; ++kb) {
          const int s = (kb - kb0) % p.stages;
          const uint32_t phase = static_cast<uint32_t>((kb - kb0) / p.stages) & 1u;
          if (!mbar_wait<true>(smem_u32(&sh.empty_bar[s]), phase ^ 1u, abort_flag)) break;
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
          const uint32_t full = map_to_cta(smem_u32(&sh.full_bar[s]), 0u);
          if (cta_rank == 0) mbar_arrive_expect_tx(smem_u32(&sh.full_bar[s]), 2u * stage_bytes);
          tma_load_2d_pair(a_dst, hmap, full, kb * kBlockK, my_tile * kTileM, pol_x);
          tma_load_2d_pair(a_dst + kATileBytes, &tmap_w, full, kb * kBlockK,
                           static_cast<int32_t>(cta_rank) * (p.N / 2), pol_w);
        }
      }
      __syncwarp();
      cluster_arrive();
    } else if (warp == 1 || warp == kSecondIssuerWarp) {
      // ---------------------------------------------------------- MMA issuers (even block only)
      if (lane == 0 && cta_rank == 0) {
        const int first_kb = kb0 + (warp == 1 ? 0 : 1);
        const uint32_t acc = tmem_base + (warp == 1 ? 0u : static_cast<uint32_t>(p.N));
        const uint32_t idesc = umma_idesc_bf16_f32(kTileM * 2, static_cast<uint32_t>(p.N));
        bool ok = true;
        const bool odd_ring = (p.stages & 1) != 0;
        volatile int32_t* my_progress = &sh.issuer_progress[warp == 1 ? 0 : 1];
        const volatile int32_t* other_progress = &sh.issuer_progress[warp == 1 ? 1 : 0];
        for (int kb = first_kb; kb < kb1 && ok; kb += 2) {
          const int s = (kb - kb0) % p.stages;
          const uint32_t phase = static_cast<uint32_t>((kb - kb0) / p.stages) & 1u;
          if (odd_ring && kb - kb0 >= p.stages) ok = issuer_turn_wait(other_progress, kb - kb0 - p.stages, abort_flag);
          ok = ok && mbar_wait<true>(smem_u32(&sh.full_bar[s]), phase, abort_flag);
          if (!ok) break;
          if (odd_ring) *my_progress = kb - kb0;
          tcgen05_fence_after();
          const uint32_t a_addr = smem_base + static_cast<uint32_t>(s) * stage_bytes;
          const uint64_t adesc = umma_smem_desc_sw128(a_addr);
          const uint64_t bdesc = umma_smem_desc_sw128(a_addr + kATileBytes);
#pragma unroll
          for (int kk = 0; kk < kBlockK / kUmmaK; ++kk)
            umma_bf16<2>(acc, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb != first_kb || kk != 0) ? 1u : 0u);
          umma_commit_pair(smem_u32(&sh.empty_bar[s]), cta_rank);
        }
        umma_commit_pair(smem_u32(&sh.accum_bar), cta_rank);      // this issuer's share of the piece is complete
      }
      __syncwarp();
      cluster_arrive();
    } else {
      // ---------------------------------------------------------- copy-out warps
      const int et = threadIdx.x - 64;
      const int quarter = warp & 3;
      const int sub = (warp - 2) >> 2;
      const int row_in_tile = quarter * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      const int N = p.N;
      const int n_chunks = (N + 31) >> 5;
      if (et == 0) sh.accum_ok = mbar_wait<true>(smem_u32(&sh.accum_bar), 0u, abort_flag) ? 1 : 0;
      named_bar_sync(kAccumBarrierId, kEpilogueThreads);
      if (sh.accum_ok != 0) {
        tcgen05_fence_after();
        // every piece has at least two k-blocks (the host sees to it): both accumulators are live
        float* part = p.split_partial + partial_offset(hp, cta_rank, N, 0) + row_in_tile;
        for (int c = sub; c < n_chunks; c += kEpiSubs) {
          const int c0 = c * 32;
          uint32_t r[32], r2[32];
          load_chunk(taddr, c0, N, r);
          load_chunk(taddr + N, c0, N, r2);
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c0 + j < N) __stcg(part + static_cast<size_t>(c0 + j) * kTileM, __uint_as_float(r[j]) + __uint_as_float(r2[j]));
        }
        tcgen05_fence_before();
        // publish the partial: every thread's stores, then one release of the flag
        named_bar_sync(kPlanBarrierId, kEpilogueThreads);
        if (et == 0) {
          __threadfence();
          uint32_t* flag = p.split_flags + static_cast<size_t>(hp) * 2 + cta_rank;
          asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(p.split_epoch) : "memory");
        }
      }
      __syncwarp();
      cluster_arrive();
    }
  } else {
    if (warp == 0) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0) {
        const uint64_t pol_x = l2_policy_evict_first();   // x is streamed once
        const uint64_t pol_w = l2_policy_evict_last();    // W is re-read by every block
        for (int kb = 0; kb < kb_end; ++kb) {
          const int s = kb % p.stages;
          const uint32_t phase = static_cast<uint32_t>(kb / p.stages) & 1u;
          if (!mbar_wait<kCtas == 2>(smem_u32(&sh.empty_bar[s]), phase ^ 1u, abort_flag)) break;
          if (kb == 0) FB_STAMP(14, 0);
          if (kb == kb_end - 1) FB_STAMP(15, 0);
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
          if (kCtas == 1) {
            const uint32_t full = smem_u32(&sh.full_bar[s]);
            mbar_arrive_expect_tx(full, stage_bytes);
            tma_load_2d(a_dst, xmap, full, kb * kBlockK, tile * kTileM, pol_x);
            tma_load_2d(a_dst + kATileBytes, &tmap_w, full, kb * kBlockK, 0, pol_w);
          } else {
            // both blocks report their bytes to the even block's barrier, which expects
            // the bytes of the whole pair
            const uint32_t full = map_to_cta(smem_u32(&sh.full_bar[s]), 0u);
            if (cta_rank == 0) mbar_arrive_expect_tx(smem_u32(&sh.full_bar[s]), 2u * stage_bytes);
            tma_load_2d_pair(a_dst, xmap, full, kb * kBlockK, tile * kTileM, pol_x);
            tma_load_2d_pair(a_dst + kATileBytes, &tmap_w, full, kb * kBlockK,
                             static_cast<int32_t>(cta_rank) * (p.N / 2), pol_w);
          }
        }
      }
      __syncwarp();
      if (kCtas == 2) cluster_arrive();          // this warp is done with the pair's shared state (see the teardown)
    } else if (warp == 1 || warp == kSecondIssuerWarp) {
      // ------------------------------------------------------------ MMA issuers
      // warp 1: k-blocks 0, 2, 4, ... into accumulator 0; the last warp: 1, 3, 5, ... into
      // accumulator 1 (N columns further).  In a pair only the even block issues.
      if (lane == 0 && cta_rank == 0) {
        const int first_kb = warp == 1 ? 0 : 1;
        const uint32_t acc = tmem_base + (warp == 1 ? 0u : static_cast<uint32_t>(p.N));
        const uint32_t idesc = umma_idesc_bf16_f32(kTileM * kCtas, static_cast<uint32_t>(p.N));
        bool ok = true;
        const bool odd_ring = (p.stages & 1) != 0;
        volatile int32_t* my_progress = &sh.issuer_progress[warp == 1 ? 0 : 1];
        const volatile int32_t* other_progress = &sh.issuer_progress[warp == 1 ? 1 : 0];
        for (int kb = first_kb; kb < kb_end && ok; kb += 2) {
          const int s = kb % p.stages;
          const uint32_t phase = static_cast<uint32_t>(kb / p.stages) & 1u;
          // an odd ring: the stage's previous use (k-block kb - stages) was the other issuer's
          if (odd_ring && kb >= p.stages) ok = issuer_turn_wait(other_progress, kb - p.stages, abort_flag);
          ok = ok && mbar_wait<kCtas == 2>(smem_u32(&sh.full_bar[s]), phase, abort_flag);
          if (!ok) break;
          if (odd_ring) *my_progress = kb;
          tcgen05_fence_after();
          if (kb == 0) FB_STAMP(16, 32);
          const uint32_t a_addr = smem_base + static_cast<uint32_t>(s) * stage_bytes;
          const uint64_t adesc = umma_smem_desc_sw128(a_addr);
          const uint64_t bdesc = umma_smem_desc_sw128(a_addr + kATileBytes);
          if (p.probe != 1) {
  #pragma unroll
            for (int kk = 0; kk < kBlockK / kUmmaK; ++kk) {
              // advance 16 elements = 32 bytes inside the swizzled row: +2 in the address field
              umma_bf16<kCtas>(acc, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb != first_kb || kk != 0) ? 1u : 0u);
            }
          }
          // frees the stage (in both blocks of a pair) when these MMAs retire
          if (kCtas == 1) umma_commit_1cta(smem_u32(&sh.empty_bar[s]));
          else umma_commit_pair(smem_u32(&sh.empty_bar[s]), cta_rank);
        }
        if (warp == 1) FB_STAMP(17, 32);
        // this issuer's accumulator is complete
        if (kCtas == 1) umma_commit_1cta(smem_u32(&sh.accum_bar));
        else umma_commit_pair(smem_u32(&sh.accum_bar), cta_rank);
      }
      if (warp == 1) {
      // One thread polls for the finished accumulator on behalf of the 16 epilogue warps,
      // which sleep at a hardware barrier meanwhile (no issue slots, no power).
      if (lane == 0) {
        bool ok = mbar_wait<kCtas == 2>(smem_u32(&sh.accum_bar), 0u, abort_flag);
        if (kSplit) {
          // ... and for the helpers' partial sums of this tile's remaining k-blocks
          const int tp = owner_block >> 1;
          for (int j = 0; j < p.split_j && ok; ++j)
            ok = flag_wait(p.split_flags + (static_cast<size_t>(tp) * p.split_j + j) * 2 + cta_rank, p.split_epoch, abort_flag);
        }
        sh.accum_ok = ok ? 1 : 0;
      }
      __syncwarp();
      named_bar_arrive(kAccumBarrierId, kEpilogueThreads + 32);
      }
      __syncwarp();
      if (kCtas == 2) cluster_arrive();
    } else {
      // ------------------------------------------------------------ epilogue
      const int et = threadIdx.x - 64;                       // 0 .. kEpilogueThreads-1
      const int quarter = warp & 3;                          // TMEM lanes this warp may touch
      const int sub = (warp - 2) >> 2;                       // which share of the columns
      const int row_in_tile = quarter * 32 + lane;
      const long long row = static_cast<long long>(tile) * kTileM + row_in_tile;
      const bool valid = row < p.T;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      const int E = p.E, N = p.N, k = p.k;
      const bool sigmoid_gate = kSel == kSelectSigmoidRank ? true
                                : kSel == kSelectSoftmaxRank ? false : p.gate != FB_GATE_SOFTMAX_TOPK;
      const int gs = kSel == kSelectSigmoidRank ? 32 : (sigmoid_gate ? E / p.n_group : E);   // experts per group
      // Which sub owns chunk c: whole groups must stay with one sub.
      const int n_chunks = (N + 31) >> 5;
      const int chunks_per_group = (sigmoid_gate && gs % 32 == 0) ? gs / 32 : 1;
      const bool splittable = !sigmoid_gate || gs % 32 == 0 || 32 % gs == 0;
      const bool want_sum = kSel == kSelectGeneral && out_w != nullptr && !p.renorm && !sigmoid_gate;
      // Selection by ranking a short candidate list instead of insertion (see select_kind).
      constexpr bool fast_select = kSel != kSelectGeneral;
      // Softmax gate over at most 32 experts (one chunk): the thread of sub 0 holds its whole row in
      // registers after pass 1 and selects there; nothing is parked in shared memory, nothing is
      // merged, and the warps that share the rows need not meet.
      const bool small_gate = kSel == kSelectGeneral && !sigmoid_gate && n_chunks == 1;

      // Chunk bookkeeping, worked out while the main loop runs (integer divisions by run-time
      // values are slow and would otherwise sit between the chunks of the epilogue):
      // which chunks this warp owns, which of them end a group, and each chunk's group.
      uint32_t owned_chunks = 0, group_end_chunks = 0, chunk_group = 0;     // bit c / nibble c
      for (int c = 0; c < n_chunks; ++c) {
        const int owner = splittable ? (c / chunks_per_group) % kEpiSubs : 0;
        if (owner == sub) owned_chunks |= 1u << c;
        if (sigmoid_gate && gs % 32 == 0) {
          if ((c * 32 + 32) % gs == 0) group_end_chunks |= 1u << c;
          chunk_group |= static_cast<uint32_t>((c * 32) / gs) << (4 * c);   // at most 8 groups here
        }
      }
      // While the main loop runs, stage the biases (read by these warps only, after the barrier
      // below) and the placement for the planner (any block may turn out to be the last one).
      for (int e = et; e < FB_MAX_EXPERTS + 32; e += kEpilogueThreads) {
        sh.logit_bias[e] = (p.logit_bias != nullptr && e < p.E) ? p.logit_bias[e] : 0.0f;
        sh.select_bias[e] = (p.select_bias != nullptr && e < p.E) ? p.select_bias[e] : 0.0f;
      }
      if (mode == kModePredictPlan) plan_load_placement(p.plan, sh.plan, et, kEpilogueThreads);
      named_bar_sync(kAccumBarrierId, kEpilogueThreads + 32);
      const bool got = sh.accum_ok != 0 && p.probe == 0;     // a measurement launch ends with its main loop
      tcgen05_fence_after();
      FB_STAMP(2, 64);

      // scratch carved out of the (now idle) pipeline stages
      float* key_s = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));   // [N][128]
      float* gscore_s = key_s + static_cast<size_t>(N) * kTileM;                               // [32][128]
      float* glow_s = gscore_s + FB_MAX_GROUPS * kTileM;                                       // [32][128]
      float* merge_v = glow_s + FB_MAX_GROUPS * kTileM;                                        // [subs-1][8][128]
      int32_t* merge_i = reinterpret_cast<int32_t*>(merge_v + (kEpiSubs - 1) * FB_MAX_TOPK * kTileM);
      float* part_s = reinterpret_cast<float*>(merge_i + (kEpiSubs - 1) * FB_MAX_TOPK * kTileM);   // [subs][2][128]

      // Between pass 1 and the histogram, data passes only between the kEpiSubs warps that share
      // this warp's rows: they meet at a barrier of their own and do not wait for the other rows' warps.
      auto row_sync = [&]() { if (!small_gate) named_bar_sync(kRowBarrierBase + static_cast<uint32_t>(quarter), kEpiSubs * 32); };

      TopK top;
      top.init();
      float sm_max = -INFINITY, sm_sum = 0.0f;               // softmax denominator (weights without renorm)
      constexpr bool has_lb = kLogitBias;
      if (got) {
        // ---------------- pass 1
        // On the ranking paths E is a multiple of 32 (N == E: every chunk is full) and sub s owns
        // chunks s, s + kEpiSubs, ...; with the DeepSeek-V3-like gate a chunk is exactly one group.
        constexpr bool kFullChunks = kSel != kSelectGeneral;
        constexpr bool kChunkIsGroup = kSel == kSelectSigmoidRank;
        float m1 = -INFINITY, m2 = -INFINITY;
#pragma unroll 1
        for (int c = kFullChunks ? sub : 0; c < n_chunks; c += kFullChunks ? kEpiSubs : 1) {
          if (!kFullChunks && ((owned_chunks >> c) & 1u) == 0) continue;
          const int c0 = c * 32;
          uint32_t r[32];
          float q[32];
          if (kFullChunks) {
            // both accumulators' loads in flight at once, one wait
            uint32_t r2[32];
            tmem_ld_32x32b_x32(taddr + c0, r);
            if (kb_end > 1) tmem_ld_32x32b_x32(taddr + N + c0, r2);
            tmem_ld_wait();
            if (kb_end > 1) {
  #pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
            }
          } else {
          load_chunk(taddr, c0, N, r);
          if (kb_end > 1) {                                    // add the odd k-blocks' accumulator
            const int halves = (N - c0 >= 32) ? 2 : 1;         // 16 columns at a time keeps registers low
            for (int h = 0; h < halves; ++h) {
              uint32_t r2[32];
              tmem_ld_32x32b_x16(taddr + N + c0 + 16 * h, r2);
              tmem_ld_wait();
              if (h == 0) {
  #pragma unroll
                for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
              } else {
  #pragma unroll
                for (int j = 0; j < 16; ++j) r[16 + j] = __float_as_uint(__uint_as_float(r[16 + j]) + __uint_as_float(r2[j]));
              }
            }
          }
          }
          if (kSplit) {
            // add the helpers' partial sums of the remaining k-blocks, piece by piece in a fixed order;
            // a partial tile is stored column by column, so the warp's 32 rows read 128 contiguous bytes
            const int tp = owner_block >> 1;
            for (int pj = 0; pj < p.split_j; ++pj) {
              const float* part = p.split_partial + partial_offset(tp * p.split_j + pj, cta_rank, N, c0) + row_in_tile;
  #pragma unroll
              for (int h = 0; h < 2; ++h) {
                float pv[16];
  #pragma unroll
                for (int j = 0; j < 16; ++j) pv[j] = (c0 + 16 * h + j < N) ? __ldcg(part + (16 * h + j) * kTileM) : 0.0f;
  #pragma unroll
                for (int j = 0; j < 16; ++j) r[16 * h + j] = __float_as_uint(__uint_as_float(r[16 * h + j]) + pv[j]);
              }
            }
          }
          if (p.logits != nullptr && valid) {
  #pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c0 + j < E)
                p.logits[row * E + c0 + j] = __uint_as_float(r[j]) + (has_lb ? sh.logit_bias[c0 + j] : 0.0f);
          }
          if (sigmoid_gate && (kFullChunks || c0 + 32 <= E) && !has_lb) {
            // whole chunk valid, no logit bias (the common case).  Every key goes through the
            // same two hardware approximations, so equal logits give equal keys in every column
            // (an FMA-pipe reciprocal on alternate columns was no faster and broke exact ties).
            const float4* sb4 = reinterpret_cast<const float4*>(&sh.select_bias[c0]);
  #pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const float4 b = sb4[j4];
              q[4 * j4 + 0] = fb_sigmoid(__uint_as_float(r[4 * j4 + 0])) + b.x;
              q[4 * j4 + 1] = fb_sigmoid(__uint_as_float(r[4 * j4 + 1])) + b.y;
              q[4 * j4 + 2] = fb_sigmoid(__uint_as_float(r[4 * j4 + 2])) + b.z;
              q[4 * j4 + 3] = fb_sigmoid(__uint_as_float(r[4 * j4 + 3])) + b.w;
            }
          } else if (sigmoid_gate) {
  #pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float z = __uint_as_float(r[j]) + (has_lb ? sh.logit_bias[c0 + j] : 0.0f);
              q[j] = (c0 + j < E) ? fb_sigmoid(z) + sh.select_bias[c0 + j] : -INFINITY;
            }
          } else {
  #pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float z = __uint_as_float(r[j]) + (has_lb ? sh.logit_bias[c0 + j] : 0.0f);
              q[j] = (c0 + j < E) ? z : -INFINITY;
            }
          }
          if (!small_gate) {
            float* kcol = key_s + c0 * kTileM + row_in_tile;
  #pragma unroll
            for (int j = 0; j < 32; ++j)
              if (kFullChunks || c0 + j < N) kcol[j * kTileM] = q[j];
          }
          if (want_sum) {
            float cmax = q[0];
  #pragma unroll
            for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, q[j]);
            const float nmax = fmaxf(sm_max, cmax);
            float part = 0.0f;
  #pragma unroll
            for (int j = 0; j < 32; ++j) part += __expf(q[j] - nmax);     // exp(-inf) = 0 for padding
            sm_sum = sm_sum * __expf(sm_max - nmax) + part;
            sm_max = nmax;
          }
          if (small_gate) {
            // k rounds of "largest remaining key"; the scan runs in ascending column order with a
            // strict comparison, so the lower expert id wins a tie.  Padding columns hold -inf.
  #pragma unroll 1
            for (int rnd = 0; rnd < k; ++rnd) {
              float best = q[0];
              int bi = 0;
  #pragma unroll
              for (int j = 1; j < 32; ++j)
                if (q[j] > best) { best = q[j]; bi = j; }
              top.insert_any_order(best, bi);
  #pragma unroll
              for (int j = 0; j < 32; ++j) q[j] = (j == bi) ? -INFINITY : q[j];
            }
            continue;
          }
          if (sigmoid_gate && gs % 32 == 0) {
            // the chunk lies inside one group: branch-free top-2 of its 32 keys by a merge tree
            float a1[16], a2[16];
  #pragma unroll
            for (int j = 0; j < 16; ++j) { a1[j] = fmaxf(q[2 * j], q[2 * j + 1]); a2[j] = fminf(q[2 * j], q[2 * j + 1]); }
  #pragma unroll
            for (int w = 8; w >= 1; w >>= 1) {
  #pragma unroll
              for (int j = 0; j < w; ++j) {
                const float hi = fmaxf(a1[j], a1[j + w]);
                a2[j] = fmaxf(fminf(a1[j], a1[j + w]), fmaxf(a2[j], a2[j + w]));
                a1[j] = hi;
              }
            }
            if (kChunkIsGroup) {
              gscore_s[c * kTileM + row_in_tile] = a1[0] + a2[0];
              glow_s[c * kTileM + row_in_tile] = a2[0];
              continue;
            }
            m2 = fmaxf(fminf(m1, a1[0]), fmaxf(m2, a2[0]));
            m1 = fmaxf(m1, a1[0]);
            if ((group_end_chunks >> c) & 1u) {                 // last chunk of the group
              const int g = static_cast<int>((chunk_group >> (4 * c)) & 15u);
              gscore_s[g * kTileM + row_in_tile] = m1 + m2;
              glow_s[g * kTileM + row_in_tile] = m2;
              m1 = -INFINITY; m2 = -INFINITY;
            }
          } else if (!sigmoid_gate && fast_select) {
            // softmax gate, fast selection: the chunk's three best keys (sorted) feed the bound
            float a1[16], a2[16], a3[16];
  #pragma unroll
            for (int j = 0; j < 16; ++j) {
              a1[j] = fmaxf(q[2 * j], q[2 * j + 1]); a2[j] = fminf(q[2 * j], q[2 * j + 1]); a3[j] = -INFINITY;
            }
  #pragma unroll
            for (int w = 8; w >= 1; w >>= 1) {
  #pragma unroll
              for (int j = 0; j < w; ++j) {
                // best three of two sorted triples
                const float lo1 = fminf(a1[j], a1[j + w]), hi2 = fmaxf(a2[j], a2[j + w]);
                a1[j] = fmaxf(a1[j], a1[j + w]);
                a2[j] = fmaxf(lo1, hi2);
                a3[j] = fmaxf(fminf(lo1, hi2), fmaxf(a3[j], a3[j + w]));
              }
            }
            gscore_s[c * kTileM + row_in_tile] = a1[0];
            gscore_s[(kBoundRows + c) * kTileM + row_in_tile] = a2[0];
            gscore_s[(2 * kBoundRows + c) * kTileM + row_in_tile] = a3[0];
          } else if (sigmoid_gate) {
            int g = c0 / gs, pos = c0 % gs;
  #pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < E) {
                m2 = fmaxf(m2, fminf(m1, q[j]));
                m1 = fmaxf(m1, q[j]);
                if (++pos == gs) {                              // group complete (uniform branch)
                  gscore_s[g * kTileM + row_in_tile] = gs >= 2 ? m1 + m2 : m1;
                  glow_s[g * kTileM + row_in_tile] = gs >= 2 ? m2 : m1;
                  ++g; pos = 0; m1 = -INFINITY; m2 = -INFINITY;
                }
              }
            }
          }
        }
      }
      FB_STAMP(3, 64);
      tcgen05_fence_before();
      // This warp has read its part of tensor memory: its share of the pair's closing barrier
      // is delivered now, so that nobody waits for it at the end (see the teardown).
      if (kCtas == 2) cluster_arrive();
      row_sync();
      FB_STAMP(4, 64);
      if (got && fast_select) {
        // ---------------- choose: rank the (at most 8) group scores of this row
        unsigned long long* cand = reinterpret_cast<unsigned long long*>(merge_v);   // [kCandCap][128], see rank_candidates
        int my_groups[2] = {-1, -1};                        // the 32-column groups this sub scans
        float floor_key = INFINITY;
        if (sigmoid_gate) {
          float sc[8];
  #pragma unroll
          for (int g = 0; g < 8; ++g) sc[g] = g < p.n_group ? gscore_s[g * kTileM + row_in_tile] : -INFINITY;
  #pragma unroll
          for (int g = 0; g < 8; ++g) {
            int rank = 0;
  #pragma unroll
            for (int h = 0; h < 8; ++h)          // a lower-numbered group wins ties
              if (h != g) rank += (h < g ? sc[h] >= sc[g] : sc[h] > sc[g]) ? 1 : 0;
            if (g < p.n_group && rank < p.topk_group) {
              floor_key = fminf(floor_key, glow_s[g * kTileM + row_in_tile]);
              if (rank == sub) my_groups[0] = g;   // sub s scans the row's s-th best group
            }
          }
        } else {
          // bound for the k-th key: the k-th largest of the chunks' three best keys (3 n_chunks >= k of them)
          floor_key = kth_largest_known(gscore_s, n_chunks, k, row_in_tile);
          if (sub < n_chunks) my_groups[0] = sub;
          if (sub + kEpiSubs < n_chunks) my_groups[1] = sub + kEpiSubs;
        }
        FB_STAMP(5, 64);
        // ---------------- collect the keys >= floor (at least k keys qualify: the bound is one of k known keys)
  #pragma unroll 1
        for (int gi = 0; gi < 2; ++gi) {
          if (my_groups[gi] < 0) continue;                  // no such group: true for the whole warp at once
          const int base = my_groups[gi] * 32;              // (which group may differ from row to row)
          uint32_t mask = 0;
  #pragma unroll
          for (int j = 0; j < 32; ++j)
            mask |= (key_s[(base + j) * kTileM + row_in_tile] >= floor_key) ? (1u << j) : 0u;
          const uint32_t mine = __popc(mask);
          const uint32_t first = atomicAdd(&sh.cand_count[row_in_tile], mine);
          const uint32_t most = __reduce_max_sync(0xffffffffu, mine);
  #pragma unroll 1
          for (uint32_t i = 0; i < most; ++i) {
            if (mask != 0 && first + i < kCandCap) {
              const int j = __ffs(mask) - 1;
              mask &= mask - 1;
              cand[(first + i) * kTileM + row_in_tile] =
                  (static_cast<unsigned long long>(ordered_bits(key_s[(base + j) * kTileM + row_in_tile])) << 32) |
                  ~static_cast<uint32_t>(base + j);
            }
          }
        }
      }
      row_sync();
      FB_STAMP(7, 64);
      uint32_t* out_hi = reinterpret_cast<uint32_t*>(gscore_s);               // [8][128], group scores are dead now
      uint32_t* out_lo = out_hi + FB_MAX_TOPK * kTileM;
      bool overflow = false;
      if (got && fast_select) {
        overflow = rank_candidates(reinterpret_cast<const unsigned long long*>(merge_v), sh.cand_count[row_in_tile], sub,
                                   row_in_tile, out_hi, out_lo);
      }
      row_sync();
      FB_STAMP(8, 64);
      if (got && fast_select && sub == 0) {
        if (!overflow) read_ranked(top, k, out_hi, out_lo, row_in_tile);
        if (__any_sync(0xffffffffu, overflow)) {
          // More than kCandCap keys reached the floor (many equal keys): plain scan of the
          // kept groups for the rows concerned.
          if (overflow && !sigmoid_gate) {
            top.init();
            for (int e = 0; e < E; ++e) {
              const float x = key_s[e * kTileM + row_in_tile];
              if (x > top.v[FB_MAX_TOPK - 1]) top.insert(x, e);
            }
          } else if (overflow) {
            float sc[8];
  #pragma unroll
            for (int g = 0; g < 8; ++g) sc[g] = -INFINITY;
            // group scores were overwritten by the output area: recompute them from the keys
            for (int g = 0; g < p.n_group; ++g) {
              float a1 = -INFINITY, a2 = -INFINITY;
              for (int j = 0; j < 32; ++j) {
                const float x = key_s[(g * 32 + j) * kTileM + row_in_tile];
                a2 = fmaxf(a2, fminf(a1, x));
                a1 = fmaxf(a1, x);
              }
  #pragma unroll
              for (int h = 0; h < 8; ++h) if (h == g) sc[h] = a1 + a2;
            }
            top.init();
  #pragma unroll
            for (int g = 0; g < 8; ++g) {
              int rank = 0;
  #pragma unroll
              for (int h = 0; h < 8; ++h)
                if (h != g) rank += (h < g ? sc[h] >= sc[g] : sc[h] > sc[g]) ? 1 : 0;
              if (g < p.n_group && rank < p.topk_group) {
                for (int j = 0; j < 32; ++j) {
                  const float x = key_s[(g * 32 + j) * kTileM + row_in_tile];
                  if (x > top.v[FB_MAX_TOPK - 1] || x == top.v[FB_MAX_TOPK - 1]) top.insert_any_order(x, g * 32 + j);
                }
              }
            }
          }
        }
      }
      if (got && !fast_select && !small_gate) {
        // ---------------- choose the groups; lower bound for the k-th key
        uint32_t keep = 1u;
        float floor_key = -INFINITY;
        if (sigmoid_gate) {
          TopK gtop;                                          // FB_MAX_TOPK >= topk_group
          gtop.init();
          for (int g = 0; g < p.n_group; ++g) {
            const float sc = gscore_s[g * kTileM + row_in_tile];
            if (sc > gtop.v[FB_MAX_TOPK - 1]) gtop.insert(sc, g);
          }
          keep = 0;
          float low = INFINITY;
  #pragma unroll
          for (int j = 0; j < FB_MAX_TOPK; ++j) {
            if (j < p.topk_group) {
              keep |= 1u << gtop.i[j];
              low = fminf(low, glow_s[gtop.i[j] * kTileM + row_in_tile]);
            }
          }
          // The kept groups' best (two) keys are eligible; if there are at least k of
          // them, the smallest is a lower bound for the k-th largest eligible key.
          if (p.topk_group * (gs >= 2 ? 2 : 1) >= k) floor_key = low;
        }
        // ---------------- pass 2
        for (int c = 0; c < n_chunks; ++c) {
          if (((owned_chunks >> c) & 1u) == 0) continue;
          const int c0 = c * 32;
          int g = sigmoid_gate ? c0 / gs : 0, pos = sigmoid_gate ? c0 % gs : 0;
          const int g_start = g, pos_start = pos;
          uint32_t cnt = 0;
          unsigned long long packed = 0;                      // up to 8 column offsets, one byte each
  #pragma unroll 4
          for (int j = 0; j < 32; ++j) {
            const int e = c0 + j;
            if (e < E) {
              const float x = key_s[e * kTileM + row_in_tile];
              if (((keep >> g) & 1u) && x >= floor_key && x > top.v[FB_MAX_TOPK - 1]) {
                if (cnt < 8) packed |= static_cast<unsigned long long>(j) << (8 * cnt);
                ++cnt;
              }
              if (++pos == gs) { ++g; pos = 0; }
            }
          }
          const uint32_t most = __reduce_max_sync(0xffffffffu, cnt);
          if (most > 8) {
            // too many candidates for the packed list somewhere in the warp: plain scan
            g = g_start; pos = pos_start;
  #pragma unroll 1
            for (int j = 0; j < 32; ++j) {
              const int e = c0 + j;
              if (e < E) {
                const float x = key_s[e * kTileM + row_in_tile];
                if (((keep >> g) & 1u) && x > top.v[FB_MAX_TOPK - 1]) top.insert(x, e);
                if (++pos == gs) { ++g; pos = 0; }
              }
            }
          } else {
  #pragma unroll 1
            for (uint32_t i = 0; i < most; ++i) {
              if (i < cnt) {
                const int e = c0 + static_cast<int>((packed >> (8 * i)) & 0xffu);
                const float x = key_s[e * kTileM + row_in_tile];
                if (x > top.v[FB_MAX_TOPK - 1]) top.insert(x, e);
              }
            }
          }
        }
        // ---------------- hand the partial lists to sub 0
        if (sub != 0) {
  #pragma unroll
          for (int j = 0; j < FB_MAX_TOPK; ++j) {
            merge_v[((sub - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile] = top.v[j];
            merge_i[((sub - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile] = top.i[j];
          }
        }
        if (want_sum) {
          part_s[(sub * 2 + 0) * kTileM + row_in_tile] = sm_max;
          part_s[(sub * 2 + 1) * kTileM + row_in_tile] = sm_sum;
        }
      }
      row_sync();
      const bool writer = got && valid && sub == 0;
      if (got && sub == 0 && !fast_select && !small_gate) {
  #pragma unroll 1
        for (int s2 = 1; s2 < kEpiSubs; ++s2) {
  #pragma unroll 1
          for (int j = 0; j < FB_MAX_TOPK; ++j) {
            const float x = merge_v[((s2 - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile];
            if (x > -INFINITY) top.insert_any_order(x, merge_i[((s2 - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile]);
          }
        }
        if (want_sum) {
          float mx = -INFINITY;
          for (int s2 = 0; s2 < kEpiSubs; ++s2) mx = fmaxf(mx, part_s[(s2 * 2 + 0) * kTileM + row_in_tile]);
          float sum = 0.0f;
          for (int s2 = 0; s2 < kEpiSubs; ++s2)
            sum += part_s[(s2 * 2 + 1) * kTileM + row_in_tile] * __expf(part_s[(s2 * 2 + 0) * kTileM + row_in_tile] - mx);
          sm_max = mx; sm_sum = sum;
        }
      }

      FB_STAMP(9, 64);
      // ---- outputs per row
      if (writer) write_row_outputs(top, p, row, out_ids, out_w, sh.select_bias, sm_max, sm_sum);
      FB_STAMP(10, 64);
      // ---- histogram: one shared-memory atomic per distinct expert per warp (Eq. 5)
      if (sub == 0) {
        if (E > 32) {
          // many bins: lanes rarely collide, plain shared-memory atomics are cheapest
  #pragma unroll
          for (int j = 0; j < FB_MAX_TOPK; ++j)
            if (j < k && writer) atomicAdd(&sh.hist[top.i[j]], 1u);
        } else {
          // few bins: add once per distinct expert per warp
  #pragma unroll
          for (int j = 0; j < FB_MAX_TOPK; ++j) {
            if (j < k) {
              const int e = writer ? top.i[j] : -1;
              const uint32_t same = __match_any_sync(0xffffffffu, e);
              if (e >= 0 && lane == __ffs(same) - 1) atomicAdd(&sh.hist[e], __popc(same));
            }
          }
        }
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      if (kSplit && et < p.split_j) {
        // every thread of this block has added the helpers' partials (pass 1 lies before the
        // barrier above): their flags go back to "not ready" for whatever launch comes next
        p.split_flags[(static_cast<size_t>(owner_block >> 1) * p.split_j + et) * 2 + cta_rank] = 0u;
      }
      if (mode == kModeDispatch) {
        if (static_cast<long long>(tile) * kTileM < p.T)       // the padding block of an odd pair owns no tile
          for (int e = et; e < E; e += kEpilogueThreads)
            p.tile_counts[static_cast<size_t>(tile) * E + e] = sh.hist[e];
      } else if (p.probe == 0) {
        publish_counts(sh, p, et, warp, lane, mode == kModePredictPlan && p.fuse_planner != 0);
      }
      FB_STAMP(12, 64);
    }
  }

  // ---------------------------------------------------------------- teardown
  // Tensor memory may be released, and a block may leave, only when both blocks of the pair
  // are done with it: every warp has delivered its arrival for the pair's barrier as soon as
  // its own last access was over (producer and issuers after their loops, epilogue warps after
  // reading the accumulators), so this wait normally finds the barrier complete.
  tcgen05_fence_before();
  __syncthreads();
  if (kCtas == 2) cluster_wait();
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(p.status, 0, FB_ERR_TIMEOUT);
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc<kCtas>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
  FB_STAMP(13, 64);
}

// Self-test of the bounded wait every kernel of this library relies on: one thread waits, for
// at most limit_ns, on a barrier that nobody ever arrives at.  The wait gives up, the kernel
// records FB_ERR_TIMEOUT in the status word and returns normally - the same path a router
// kernel takes when a copy or an MMA it waits for never completes.
__global__ void __launch_bounds__(32, 1)
fb_wait_selftest_kernel(uint64_t limit_ns, int32_t* status, uint64_t* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int32_t abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
    const uint64_t t0 = global_timer_ns();
    const bool ok = mbar_wait<false>(smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (waited_ns != nullptr) *waited_ns = global_timer_ns() - t0;
    if (!ok) atomicCAS(status, 0, FB_ERR_TIMEOUT);
  }
}

// Stand-alone planner: one warp.
__global__ void __launch_bounds__(kPlanThreads, 1)
fb_plan_kernel(const __grid_constant__ PlanParams p, const uint32_t* __restrict__ counts, int32_t* status) {
  __shared__ PlanShared sh;
  const int t = threadIdx.x;
  plan_clear(sh, t, kPlanThreads);
  __syncwarp();
  plan_load_placement(p, sh, t, kPlanThreads);
  __syncwarp();
  for (int e = t; e < p.E; e += kPlanThreads) plan_put_count(sh, e, counts[e]);
  plan_swaps_warp<true>(p, sh, t, status);
  __syncwarp();
  plan_write_placement(p, sh, t, kPlanThreads);
}

}  // namespace fb
