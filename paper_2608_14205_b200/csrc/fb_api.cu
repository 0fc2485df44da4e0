// Host side of the C ABI declared in include/freebalance.h: argument checks, TMA
// descriptors, kernel launches.  No computation of the method happens on the host
// except the two pure helpers fb_budget_ns (Eq. 10) and fb_swap_cost_ns (Eq. 9).
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <new>

#include "../../include/freebalance.h"
#include "../../include/freebalance_aids.h"
#include "fb_dispatch.cuh"
#include "fb_migrate.cuh"
#include "fb_planner.cuh"
#include "fb_quality.cuh"
#include "fb_router.cuh"
#include "fb_router_persistent.cuh"

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapEntry {
  const void* ptr = nullptr;
  int64_t rows = -1;
  uint32_t box_rows = 0;
  CUtensorMap map;
};

constexpr int kMapCache = 8;

}  // namespace

struct fb_ctx {
  fb_config cfg;
  int device = 0;
  int N = 0;                      // experts padded to a multiple of 16 (UMMA N)
  int stages[2] = {0, 0};         // pipeline depth for the single-block and the pair kernel
  int tmem_cols = 0;
  size_t smem_bytes[2] = {0, 0};
  int max_tiles = 0;
  // persistent router kernel (several tiles per block pair): pipeline depth (0 = not usable
  // for this shape), dynamic shared memory, block pairs that fit on the GPU at once, and
  // the caller's limit on the pairs to use (0 = none)
  int persist_stages = 0;
  size_t persist_smem = 0;
  int max_pairs = 0;
  int pair_limit = 0;
  int stage_limit = 0;                 // diagnostic: pipeline stages at most (0 = as many as fit)
  int dispatch_blocks_max = 296;       // resident blocks of the dispatch-index kernel (2 per SM)
  // k-range split of the one-tile pair kernel: block pairs that fit on the GPU at once, the
  // partial tiles and their flags (one slot per helper item; set by the helper, put back by the
  // owner), and the caller's switch / tuning value
  int split_pairs = 0;
  float* split_partial = nullptr;
  uint32_t* split_flags = nullptr;
  int split_mode = 1;                  // 0 off, 1 on
  int split_bias = -1;                 // extra k-blocks an owner keeps (-1: the built-in choice)
  EncodeTiledFn encode = nullptr;
  // device scratch
  uint32_t* counts_scratch = nullptr;   // [256], zero between calls
  uint32_t* ticket = nullptr;           // [1],   zero between calls
  int32_t* status = nullptr;            // [1]
  uint32_t* tile_counts = nullptr;      // [max_tiles][E]
  uint32_t* super_counts = nullptr;     // [ceil(max_tiles / 32)][E]
  // descriptor cache
  MapEntry x_maps[kMapCache];
  MapEntry w_maps[kMapCache];
  int x_next = 0, w_next = 0;
  // staging for fb_layer_step_host (allocated on first use)
  bool staged = false;
  void* st_hprev = nullptr; void* st_H = nullptr;
  // staging for fb_apply_swaps_staged (allocated on first use): pinned host copy of a plan and of the
  // placement, and one device buffer of mig_stage_bytes
  void* mig_host = nullptr; void* mig_stage = nullptr; uint64_t mig_stage_bytes = 0;
  int32_t* st_pi = nullptr; int32_t* st_pi_out = nullptr;
  uint32_t* st_counts = nullptr; fb_swap* st_swaps = nullptr; int32_t* st_nswaps = nullptr;
  uint32_t* st_load_before = nullptr; uint32_t* st_load_after = nullptr;
  int32_t* st_ids = nullptr; float* st_w = nullptr;
  uint32_t* st_slot_offsets = nullptr; uint32_t* st_rank_offsets = nullptr;
  int32_t* st_perm = nullptr; int32_t* st_inv_perm = nullptr; uint32_t* st_rank_load = nullptr;
  uint64_t launches = 0;
  uint64_t persistent_launches = 0;
  cudaEvent_t ev_before = nullptr, ev_after = nullptr;   // one-shot: recorded around the next router launch
  unsigned long long* stamps = nullptr;                  // caller's phase-stamp buffer (FB_TIMING builds)
  // attention profile (Eq. 10): one measurement per attention type, taken on the first layer of the type
  struct AttnSlot {
    int32_t layer = -1;                // r(l): the layer whose attention is (being) measured; -1 = none yet
    bool open = false;                 // begin recorded, end not yet
    bool pending = false;              // both events recorded, time not read yet
    bool has_time = false;
    uint64_t t_ns = 0;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
  } attn[FB_MAX_ATTENTION_TYPES];
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int next_pow2_at_least_32(int n) {
  int c = 32;
  while (c < n) c <<= 1;
  return c;
}

fb_status check_config(const fb_config& c) {
  if (c.T_max < 0 || c.d <= 0 || c.E <= 0 || c.k <= 0 || c.R <= 0) return FB_ERR_INVALID_ARG;
  if (c.gate != FB_GATE_SOFTMAX_TOPK && c.gate != FB_GATE_SIGMOID_GROUP_TOPK) return FB_ERR_INVALID_ARG;
  if (c.E > FB_MAX_EXPERTS || c.k > FB_MAX_TOPK || c.k > c.E) return FB_ERR_UNSUPPORTED_SHAPE;
  if (c.R > FB_MAX_RANKS || c.E % c.R != 0) return FB_ERR_UNSUPPORTED_SHAPE;
  if (c.d < 8 || c.d % 8 != 0) return FB_ERR_UNSUPPORTED_SHAPE;
  const int64_t widest = c.E > c.k ? c.E : c.k;
  if (static_cast<int64_t>(c.T_max) * widest >= (int64_t{1} << 31)) return FB_ERR_UNSUPPORTED_SHAPE;
  if (c.gate == FB_GATE_SIGMOID_GROUP_TOPK) {
    if (c.n_group <= 0 || c.topk_group <= 0) return FB_ERR_INVALID_ARG;
    if (c.n_group > FB_MAX_GROUPS || c.E % c.n_group != 0) return FB_ERR_UNSUPPORTED_SHAPE;
    if (c.topk_group > c.n_group || c.topk_group > FB_MAX_TOPK) return FB_ERR_UNSUPPORTED_SHAPE;
    if (static_cast<int64_t>(c.topk_group) * (c.E / c.n_group) < c.k) return FB_ERR_UNSUPPORTED_SHAPE;
  }
  return FB_OK;
}

fb_status make_map(fb_ctx* ctx, MapEntry* cache, int* next, const void* ptr, int64_t rows, uint32_t box_rows,
                   const CUtensorMap** out) {
  for (int i = 0; i < kMapCache; ++i)
    if (cache[i].ptr == ptr && cache[i].rows == rows && cache[i].box_rows == box_rows) {
      *out = &cache[i].map;
      return FB_OK;
    }
  if ((reinterpret_cast<uintptr_t>(ptr) & 15u) != 0) return FB_ERR_INVALID_ARG;
  MapEntry& e = cache[*next];
  *next = (*next + 1) % kMapCache;
  const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(ctx->cfg.d), static_cast<cuuint64_t>(rows)};
  const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ctx->cfg.d) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(fb::kBlockK), box_rows};
  const cuuint32_t estride[2] = {1, 1};
  const CUresult r = ctx->encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride,
                                 box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { e.ptr = nullptr; e.rows = -1; return FB_ERR_CUDA; }
  e.ptr = ptr;
  e.rows = rows;
  e.box_rows = box_rows;
  *out = &e.map;
  return FB_OK;
}

uint64_t uniform_cost(const fb_budget& b, int cls) {
  const unsigned __int128 fs = static_cast<unsigned __int128>(b.expert_bytes) * 2u * b.fs_per_byte[cls];
  const unsigned __int128 ns = (fs + 999999u) / 1000000u + b.alpha_ns[cls];
  if (ns > UINT64_MAX) return 0;
  const uint64_t c = static_cast<uint64_t>(ns);
  return c < 1 ? 1 : c;
}

fb_status fill_plan(const fb_ctx* ctx, const fb_budget* b, const int32_t* pi, int32_t* pi_out, fb_swap* swaps,
                    int32_t* n_swaps, uint32_t* load_before, uint32_t* load_after, fb::PlanParams* pp) {
  if (!b || !pi || !pi_out || !n_swaps || !load_before || !load_after) return FB_ERR_INVALID_ARG;
  if (b->max_swaps > static_cast<uint32_t>(ctx->cfg.E / 2)) return FB_ERR_INVALID_ARG;
  if (b->max_swaps > 0 && !swaps) return FB_ERR_INVALID_ARG;
  if (b->gamma_num > FB_MAX_GAMMA_NUM) return FB_ERR_INVALID_ARG;
  pp->E = ctx->cfg.E;
  pp->R = ctx->cfg.R;
  pp->max_swaps = b->max_swaps;
  pp->global_ns = b->global_ns;
  pp->rank_ns = b->rank_ns;
  pp->link_ns = b->link_ns;
  pp->tau_tokens = b->tau_tokens;
  pp->gamma_num = b->gamma_num;
  pp->gamma_den = b->gamma_den;
  for (int c = 0; c < 2; ++c) {
    pp->alpha_ns[c] = b->alpha_ns[c];
    pp->fs_per_byte[c] = b->fs_per_byte[c];
    pp->uniform_cost_ns[c] = uniform_cost(*b, c);
    if (b->expert_bytes_table == nullptr && pp->uniform_cost_ns[c] == 0) return FB_ERR_INVALID_ARG;
    pp->uniform_link_cap[c] = pp->uniform_cost_ns[c] ? b->link_ns / pp->uniform_cost_ns[c] : 0;
  }
  if (b->mode != FB_PLAN_LOOP && b->mode != FB_PLAN_SWEEP && b->mode != FB_PLAN_WIDE) return FB_ERR_INVALID_ARG;
  pp->mode = b->mode;
  pp->frontier_width = b->frontier_width;
  pp->ranks_per_node = b->ranks_per_node;
  pp->expert_bytes_table = b->expert_bytes_table;
  pp->expert_to_slot = pi;
  pp->expert_to_slot_out = pi_out;
  pp->swaps = swaps;
  pp->n_swaps = n_swaps;
  pp->load_before = load_before;
  pp->load_after = load_after;
  return FB_OK;
}

// Kernel instances by (selection kind, logit bias present).
using RouterKernelFn = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, fb::RouterParams);
template <int kCtas>
static RouterKernelFn router_kernel_fn(int sel, bool lb) {
  switch (sel * 2 + (lb ? 1 : 0)) {
    case 0: return fb::fb_router_kernel<kCtas, fb::kSelectGeneral, false>;
    case 1: return fb::fb_router_kernel<kCtas, fb::kSelectGeneral, true>;
    case 2: return fb::fb_router_kernel<kCtas, fb::kSelectSigmoidRank, false>;
    case 3: return fb::fb_router_kernel<kCtas, fb::kSelectSigmoidRank, true>;
    case 4: return fb::fb_router_kernel<kCtas, fb::kSelectSoftmaxRank, false>;
    default: return fb::fb_router_kernel<kCtas, fb::kSelectSoftmaxRank, true>;
  }
}
static RouterKernelFn router_split_kernel_fn(int sel, bool lb) {
  switch (sel * 2 + (lb ? 1 : 0)) {
    case 0: return fb::fb_router_kernel<2, fb::kSelectGeneral, false, true>;
    case 1: return fb::fb_router_kernel<2, fb::kSelectGeneral, true, true>;
    case 2: return fb::fb_router_kernel<2, fb::kSelectSigmoidRank, false, true>;
    case 3: return fb::fb_router_kernel<2, fb::kSelectSigmoidRank, true, true>;
    case 4: return fb::fb_router_kernel<2, fb::kSelectSoftmaxRank, false, true>;
    default: return fb::fb_router_kernel<2, fb::kSelectSoftmaxRank, true, true>;
  }
}
static RouterKernelFn persistent_kernel_fn(bool sigmoid, bool lb) {
  if (sigmoid) return lb ? fb::fb_router_persistent_kernel<true, true> : fb::fb_router_persistent_kernel<true, false>;
  return lb ? fb::fb_router_persistent_kernel<false, true> : fb::fb_router_persistent_kernel<false, false>;
}

// Launch the router kernel in one of its three modes.
// x2 is the second input of kModeLayer (the normal router input), nullptr otherwise.
fb_status launch_router(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T, int mode,
                        uint32_t* counts_out, int32_t* topk_ids, float* topk_w, float* logits,
                        const fb::PlanParams* plan, cudaStream_t stream, const void* x2 = nullptr, int probe = 0) {
  const CUtensorMap *mx = nullptr, *mx2 = nullptr, *mw = nullptr;
  fb_status st = make_map(ctx, ctx->x_maps, &ctx->x_next, x, T, fb::kTileM, &mx);
  if (st != FB_OK) return st;
  const CUtensorMap map_x = *mx;     // by value: the second lookup may evict the cache slot mx points to
  mx = &map_x;
  mx2 = mx;
  if (mode == fb::kModeLayer) {
    st = make_map(ctx, ctx->x_maps, &ctx->x_next, x2, T, fb::kTileM, &mx2);
    if (st != FB_OK) return st;
  }
  const int tiles = (T + fb::kTileM - 1) / fb::kTileM;
  const int pair = (tiles > 1 && ctx->stages[1] >= 2) ? 1 : 0;   // a single tile gains nothing from a partner
  st = make_map(ctx, ctx->w_maps, &ctx->w_next, router->W, ctx->cfg.E,
                static_cast<uint32_t>(pair ? ctx->N / 2 : ctx->N), &mw);
  if (st != FB_OK) return st;
  fb::RouterParams p;
  memset(&p, 0, sizeof(p));
  const fb_config& c = ctx->cfg;
  p.T = T; p.d = c.d; p.E = c.E; p.N = ctx->N; p.k = c.k;
  p.gate = c.gate; p.n_group = c.gate == FB_GATE_SIGMOID_GROUP_TOPK ? c.n_group : 1;
  p.topk_group = c.gate == FB_GATE_SIGMOID_GROUP_TOPK ? c.topk_group : 1;
  p.renorm = c.renorm; p.route_scale = c.route_scale;
  p.num_kb = (c.d + fb::kBlockK - 1) / fb::kBlockK;
  p.stages = ctx->stages[pair];
  if (ctx->stage_limit >= 2 && ctx->stage_limit < p.stages) p.stages = ctx->stage_limit;
  p.tmem_cols = ctx->tmem_cols;
  p.mode = mode;
  p.logit_bias = router->logit_bias;
  p.select_bias = c.gate == FB_GATE_SIGMOID_GROUP_TOPK ? router->select_bias : nullptr;
  p.counts_scratch = ctx->counts_scratch;
  p.ticket = ctx->ticket;
  p.status = ctx->status;
  p.counts_out = counts_out;
  p.topk_ids = topk_ids;
  p.topk_w = topk_w;
  p.logits = logits;
  p.tile_counts = ctx->tile_counts;
  p.stamps = ctx->stamps;
  p.probe = probe;
  if (plan) p.plan = *plan;
  // The fused tail serves the common plans; a plan that needs the general loop (per-expert sizes,
  // more than 16 experts per rank, a planner variant) gets the stand-alone planner kernel behind
  // the router kernel instead.
  const bool plan_wanted = plan != nullptr && (mode == fb::kModePredictPlan || mode == fb::kModeLayer);
  p.fuse_planner = (plan_wanted && !fb::plan_needs_general_loop(*plan)) ? 1 : 0;
  const int tiles_pad = pair ? (tiles + 1) / 2 * 2 : tiles;       // a pair never straddles the two passes
  int blocks = mode == fb::kModeLayer ? 2 * tiles_pad : tiles_pad;
  p.tiles_first = tiles_pad;
  p.ticket_target = tiles_pad;
  // More tile pairs than block pairs fit on the GPU (or than the caller allows): the
  // persistent kernel walks several tiles per block pair and overlaps their epilogues.
  // selection code of this launch: the ranking selection only if it applies to every block
  // (in layer mode the normal pass writes weights, the early pass does not)
  const int sel = fb::select_kind(c.E, ctx->N, c.k, c.gate, p.n_group, p.topk_group,
                                  topk_w != nullptr && !c.renorm && c.gate == FB_GATE_SOFTMAX_TOPK);
  bool persistent = false;
  if (pair && ctx->persist_stages >= 2 && logits == nullptr && probe == 0) {
    const bool want_sum = topk_w != nullptr && !c.renorm && c.gate == FB_GATE_SOFTMAX_TOPK;
    const int pairs_avail = ctx->pair_limit > 0 && ctx->pair_limit < ctx->max_pairs ? ctx->pair_limit : ctx->max_pairs;
    if (fb::persistent_gate_ok(c.E, c.k, c.gate, p.n_group, p.topk_group, want_sum) && blocks / 2 > pairs_avail) {
      persistent = true;
      // no more block pairs than the number of rounds needs: 128 tile pairs run as 2 rounds on 64
      // block pairs just as fast as on 74 (measured), and the other SMs stay free for other streams
      const int rounds = (blocks / 2 + pairs_avail - 1) / pairs_avail;
      blocks = 2 * ((blocks / 2 + rounds - 1) / rounds);
      // every block publishes its counts once: as many tickets as blocks that own a tile of the
      // counted pass
      p.ticket_target = blocks < tiles_pad ? blocks : tiles_pad;
      // room for two accumulator sets (4 N columns) when the 512 tensor-memory columns allow it
      if (4 * ctx->N <= 512) p.tmem_cols = next_pow2_at_least_32(4 * ctx->N);
      p.stages = ctx->persist_stages;
      if (ctx->stage_limit >= 2 && ctx->stage_limit < p.stages) p.stages = ctx->stage_limit;
    }
  }
  // Fewer tile pairs than block pairs fit on the GPU: the spare pairs become helpers that sum
  // the tail of every tile's k-range (see RouterParams).  The schedule depends on the shape and
  // on the number of pairs only.
  bool split = false;
  if (pair && !persistent && ctx->split_partial != nullptr && ctx->split_mode != 0 && probe == 0) {
    const int tile_pairs = blocks / 2;                   // over both passes of a layer launch
    int pairs_avail = ctx->split_pairs;
    if (ctx->pair_limit > 0 && ctx->pair_limit < pairs_avail) pairs_avail = ctx->pair_limit;
    const int spare = pairs_avail - tile_pairs;
    // Worth it only where at least half of the pairs would idle: with 64 tile pairs on 74 block
    // pairs (the 16k-token DeepSeek-V3 shape) the chip is power bound while the main loop runs -
    // more busy SMs lower the clock, rows per microsecond rise by 5 % from 128 to 148 SMs - and
    // helpers add their copy-outs on top (measured: 60 -> 68 us).
    if (spare >= tile_pairs && p.num_kb >= 32) {
      int J = spare / tile_pairs;                      // helpers per tile: J pieces each
      if (J > 3) J = 3;
      const int helpers = tile_pairs * J;
      int ko = (p.num_kb + J) / (J + 1);
      // a helper pays for the copy-out of its partial, the owner for reading it: owners keep a
      // few k-blocks more than an even share
      ko += ctx->split_bias >= 0 ? ctx->split_bias : 4;
      if (ko > p.num_kb - 2 * J) ko = p.num_kb - 2 * J;     // every piece has at least two k-blocks
      if (ko >= 2) {
        split = true;
        p.split_helpers = helpers;
        p.split_ko = ko;
        p.split_j = J;
        p.split_epoch = 1;          // "complete"; the owner that consumed a partial puts the flag back to 0
        p.split_partial = ctx->split_partial;
        p.split_flags = ctx->split_flags;
        blocks += 2 * helpers;
      }
    }
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(fb::kRouterThreads, 1, 1);
  cfg.dynamicSmemBytes = ctx->smem_bytes[pair];
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  cudaError_t err;
  if (persistent) cfg.dynamicSmemBytes = ctx->persist_smem;
  if (ctx->ev_before) cudaEventRecord(ctx->ev_before, stream);
  // Programmatic dependent launch: when the previous kernel of the stream allows it (the
  // dispatch-index kernel does), this kernel's set-up overlaps that kernel's execution; the
  // kernel waits for its completion (griddepcontrol.wait) before it reads any global memory.
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (pair) {
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    const bool lb = router->logit_bias != nullptr;
    err = cudaLaunchKernelEx(&cfg, persistent ? persistent_kernel_fn(c.gate == FB_GATE_SIGMOID_GROUP_TOPK, lb)
                                   : split    ? router_split_kernel_fn(sel, lb)
                                              : router_kernel_fn<2>(sel, lb), *mx, *mx2, *mw, p);
  } else {
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
    err = cudaLaunchKernelEx(&cfg, router_kernel_fn<1>(sel, router->logit_bias != nullptr), *mx, *mx2, *mw, p);
  }
  if (ctx->ev_after) cudaEventRecord(ctx->ev_after, stream);
  ctx->ev_before = ctx->ev_after = nullptr;
  ++ctx->launches;
  if (persistent) ++ctx->persistent_launches;
  if (err != cudaSuccess) return FB_ERR_CUDA;
  if (plan_wanted && !p.fuse_planner) {
    fb::fb_plan_kernel<<<1, fb::kPlanThreads, 0, stream>>>(*plan, counts_out, ctx->status);
    ++ctx->launches;
    if (cudaGetLastError() != cudaSuccess) return FB_ERR_CUDA;
  }
  return FB_OK;
}

// Dispatch index from the router kernel's top-k ids and per-tile histograms.
fb_status launch_dispatch_index(fb_ctx* ctx, int32_t T, const int32_t* expert_to_slot, const int32_t* topk_ids,
                                uint32_t* slot_offsets, uint32_t* rank_offsets, int32_t* perm, int32_t* inv_perm,
                                uint32_t* rank_load, cudaStream_t stream) {
  const fb_config& c = ctx->cfg;
  fb::DispatchParams dp;
  dp.T = T; dp.k = c.k; dp.E = c.E; dp.R = c.R;
  dp.num_tiles = (T + fb::kDispatchTile - 1) / fb::kDispatchTile;
  dp.topk_ids = topk_ids;
  dp.tile_counts = ctx->tile_counts;
  dp.super_counts = nullptr;
  if (dp.num_tiles > 4 * fb::kSuperTiles) {                 // beyond 16k tokens the two-level sums pay off
    const int n_super = (dp.num_tiles + fb::kSuperTiles - 1) / fb::kSuperTiles;
    fb::fb_tile_sums_kernel<<<n_super, FB_MAX_EXPERTS, 0, stream>>>(ctx->tile_counts, ctx->super_counts,
                                                                     dp.num_tiles, c.E);
    ++ctx->launches;
    if (cudaGetLastError() != cudaSuccess) return FB_ERR_CUDA;
    dp.super_counts = ctx->super_counts;
  }
  dp.expert_to_slot = expert_to_slot;
  dp.slot_offsets = slot_offsets;
  dp.rank_offsets = rank_offsets;
  dp.perm = perm;
  dp.inv_perm = inv_perm;
  dp.rank_load = rank_load;
  dp.status = ctx->status;
  // at most two blocks per SM are resident (1024 threads each): more tiles than that are walked in runs
  const int dispatch_blocks = dp.num_tiles < ctx->dispatch_blocks_max ? dp.num_tiles : ctx->dispatch_blocks_max;
  fb::fb_dispatch_kernel<<<dispatch_blocks, fb::kDispatchThreads, 0, stream>>>(dp);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status launch_plan(fb_ctx* ctx, const fb::PlanParams& pp, const uint32_t* counts, cudaStream_t stream) {
  fb::fb_plan_kernel<<<1, fb::kPlanThreads, 0, stream>>>(pp, counts, ctx->status);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

// The device that owns a device pointer (-1 if it is not device memory).
int device_of(const void* p) {
  cudaPointerAttributes pa;
  if (cudaPointerGetAttributes(&pa, p) != cudaSuccess) { cudaGetLastError(); return -1; }
  return (pa.type == cudaMemoryTypeDevice || pa.type == cudaMemoryTypeManaged) ? pa.device : -1;
}

// A fixed one-swap plan over two slots for fb_calibrate_exchange: [placement: 2][swap: 4][n: 1].
// Constant data inside the library image, so the calibration allocates nothing.
__device__ const int32_t g_calibration_plan[8] = {0, 1, 0, 1, 0, 1, 1, 0};

template <typename Tp>
bool dev_alloc(Tp** p, size_t count) {
  return cudaMalloc(reinterpret_cast<void**>(p), (count ? count : 1) * sizeof(Tp)) == cudaSuccess;
}

}  // namespace

// Shape-dependent launch parameters of the one-tile router kernel (host arithmetic
// only): padded width, TMEM columns, pipeline depth and dynamic shared
// memory of the single-block and the pair variant.
static fb_status setup_router_shape(fb_ctx* ctx, const cudaDeviceProp& prop) {
  const fb_config& cfg = ctx->cfg;
  ctx->N = (cfg.E + 15) / 16 * 16;
  ctx->tmem_cols = next_pow2_at_least_32(2 * ctx->N)   /* two accumulators */;
  const size_t budget = static_cast<size_t>(prop.sharedMemPerBlockOptin) - sizeof(fb::RouterShared) - 2048;
  for (int pair = 0; pair < 2; ++pair) {
    const size_t stage_bytes = fb::kATileBytes + static_cast<size_t>(ctx->N / (pair + 1)) * fb::kBlockK * 2;
    int stages = static_cast<int>((budget - 1024) / stage_bytes);
    if (stages > fb::kMaxStages) stages = fb::kMaxStages;
    size_t dyn = stages * stage_bytes;
    if (dyn < fb::epilogue_scratch_bytes(ctx->N)) dyn = fb::epilogue_scratch_bytes(ctx->N);
    if (stages < 2 || dyn + 1024 > budget) {
      if (pair == 0) return FB_ERR_UNSUPPORTED_SHAPE;
      stages = 0;                                      // pair kernel not usable for this shape
    }
    ctx->stages[pair] = stages;
    ctx->smem_bytes[pair] = dyn + 1024;
  }
  ctx->max_tiles = (cfg.T_max + fb::kTileM - 1) / fb::kTileM;
  ctx->dispatch_blocks_max = 2 * prop.multiProcessorCount;
  return FB_OK;
}

// The ceiling on a kernel's dynamic shared memory belongs to the function on a device, not
// to a context: contexts of different shapes share the kernel instances.  It is therefore
// raised once per device, for every router kernel instance, to the most the device allows
// beside the kernel's static shared memory, and never lowered again.
static fb_status ensure_kernel_attributes(int device, const cudaDeviceProp& prop) {
  static bool done[64] = {};
  if (device >= 0 && device < 64 && done[device]) return FB_OK;
  bool ok = true;
  auto raise = [&](RouterKernelFn fn) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, reinterpret_cast<const void*>(fn)) != cudaSuccess) { ok = false; return; }
    const int most = static_cast<int>(prop.sharedMemPerBlockOptin) - static_cast<int>(fa.sharedSizeBytes);
    ok = ok && most > 0 &&
         cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, most) ==
             cudaSuccess;
  };
  for (int sel = 0; sel < 3; ++sel)
    for (int lb = 0; lb < 2; ++lb) {
      raise(router_kernel_fn<1>(sel, lb != 0));
      raise(router_kernel_fn<2>(sel, lb != 0));
      raise(router_split_kernel_fn(sel, lb != 0));
    }
  for (int sg = 0; sg < 2; ++sg)
    for (int lb = 0; lb < 2; ++lb) raise(persistent_kernel_fn(sg != 0, lb != 0));
  if (!ok) { cudaGetLastError(); return FB_ERR_CUDA; }
  if (device >= 0 && device < 64) done[device] = true;
  return FB_OK;
}

extern "C" {

const char* fb_status_string(fb_status s) {
  switch (s) {
    case FB_OK: return "ok";
    case FB_ERR_INVALID_ARG: return "invalid argument";
    case FB_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case FB_ERR_CUDA: return "CUDA call failed";
    case FB_ERR_BAD_PLACEMENT: return "expert_to_slot is not a bijection";
    case FB_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case FB_ERR_RANGE: return "sum of counts beyond the planner's range";
    case FB_ERR_INTERNAL: return "debug build: an output index was out of range";
  }
  return "unknown status";
}

uint64_t fb_budget_ns(uint64_t t_attn_ns, uint64_t delta_ns) {
  return t_attn_ns > delta_ns ? t_attn_ns - delta_ns : 0;
}

uint64_t fb_swap_cost_ns(const fb_budget* b, int32_t rank_a, int32_t rank_b) {
  if (!b) return 0;
  const int rpn = b->ranks_per_node;
  const int cls = (rpn <= 0 || rank_a / rpn == rank_b / rpn) ? 0 : 1;
  return uniform_cost(*b, cls);
}

fb_status fb_create(fb_ctx** out, const fb_config* cfg, int device) {
  if (!out || !cfg) return FB_ERR_INVALID_ARG;
  *out = nullptr;
  const fb_status cs = check_config(*cfg);
  if (cs != FB_OK) return cs;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return FB_ERR_CUDA;
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FB_ERR_CUDA;
  if (prop.major != 10) return FB_ERR_CUDA;            // built for sm_100a only; no fallback
  fb_ctx* ctx = new (std::nothrow) fb_ctx();
  if (!ctx) return FB_ERR_CUDA;
  ctx->cfg = *cfg;
  ctx->device = device;
  {
    fb_status ss = setup_router_shape(ctx, prop);
    if (ss == FB_OK) ss = ensure_kernel_attributes(device, prop);
    if (ss != FB_OK) { delete ctx; return ss; }
  }
  if (ctx->stages[1] >= 2 && ctx->N % 32 == 0 && ctx->N == cfg->E) {
    const size_t budget_p = static_cast<size_t>(prop.sharedMemPerBlockOptin) - sizeof(fb::PersistShared) - 2048;
    const size_t stage_bytes = fb::kATileBytes + static_cast<size_t>(ctx->N / 2) * fb::kBlockK * 2;
    if (budget_p > 1024 + fb::kPersistScratchBytes + 2 * stage_bytes) {
      int stages = static_cast<int>((budget_p - 1024 - fb::kPersistScratchBytes) / stage_bytes);
      if (stages > fb::kMaxStages) stages = fb::kMaxStages;
      ctx->persist_stages = stages;
      ctx->persist_smem = stages * stage_bytes + fb::kPersistScratchBytes + 1024;
    }
  }

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    delete ctx;
    return FB_ERR_CUDA;
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  bool ok = true;
  if (ctx->persist_stages >= 2) {
    // how many block pairs the GPU holds at once (the grid of the persistent kernel)
    cudaLaunchConfig_t occ;
    memset(&occ, 0, sizeof(occ));
    occ.gridDim = dim3(2 * static_cast<unsigned>(prop.multiProcessorCount), 1, 1);
    occ.blockDim = dim3(fb::kRouterThreads, 1, 1);
    occ.dynamicSmemBytes = ctx->persist_smem;
    cudaLaunchAttribute cl[1];
    cl[0].id = cudaLaunchAttributeClusterDimension;
    cl[0].val.clusterDim.x = 2; cl[0].val.clusterDim.y = 1; cl[0].val.clusterDim.z = 1;
    occ.attrs = cl;
    occ.numAttrs = 1;
    int n_clusters = 0;
    if (ok && cudaOccupancyMaxActiveClusters(&n_clusters, persistent_kernel_fn(cfg->gate == FB_GATE_SIGMOID_GROUP_TOPK, false),
                                             &occ) == cudaSuccess &&
        n_clusters >= 1)
      ctx->max_pairs = n_clusters;
    else
      ctx->persist_stages = 0;                           // not usable here: the one-tile kernel serves every call
    cudaGetLastError();
  }
  if (ctx->stages[1] >= 2) {
    // block pairs of the one-tile pair kernel that the GPU holds at once: the grid of a split launch
    cudaLaunchConfig_t occ;
    memset(&occ, 0, sizeof(occ));
    occ.gridDim = dim3(2 * static_cast<unsigned>(prop.multiProcessorCount), 1, 1);
    occ.blockDim = dim3(fb::kRouterThreads, 1, 1);
    occ.dynamicSmemBytes = ctx->smem_bytes[1];
    cudaLaunchAttribute cl[1];
    cl[0].id = cudaLaunchAttributeClusterDimension;
    cl[0].val.clusterDim.x = 2; cl[0].val.clusterDim.y = 1; cl[0].val.clusterDim.z = 1;
    occ.attrs = cl;
    occ.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, router_split_kernel_fn(0, false), &occ) == cudaSuccess &&
        n_clusters >= 2) {
      ctx->split_pairs = n_clusters;
      const size_t slots = static_cast<size_t>(n_clusters);          // one partial per helper item, at most
      ok = ok && dev_alloc(&ctx->split_partial, slots * 2 * ctx->N * fb::kTileM) &&
           dev_alloc(&ctx->split_flags, slots * 2) &&
           cudaMemset(ctx->split_flags, 0, slots * 2 * sizeof(uint32_t)) == cudaSuccess;
    }
    cudaGetLastError();
  }
  ok = ok && dev_alloc(&ctx->counts_scratch, FB_MAX_EXPERTS) && dev_alloc(&ctx->ticket, 1) &&
       dev_alloc(&ctx->status, 1) &&
       dev_alloc(&ctx->tile_counts, static_cast<size_t>(ctx->max_tiles) * cfg->E) &&
       dev_alloc(&ctx->super_counts,
                 static_cast<size_t>((ctx->max_tiles + fb::kSuperTiles - 1) / fb::kSuperTiles) * cfg->E);
  ok = ok && cudaMemset(ctx->counts_scratch, 0, FB_MAX_EXPERTS * sizeof(uint32_t)) == cudaSuccess &&
       cudaMemset(ctx->ticket, 0, sizeof(uint32_t)) == cudaSuccess &&
       cudaMemset(ctx->status, 0, sizeof(int32_t)) == cudaSuccess;
  if (!ok) { fb_destroy(ctx); return FB_ERR_CUDA; }
  *out = ctx;
  return FB_OK;
}

fb_status fb_destroy(fb_ctx* ctx) {
  if (!ctx) return FB_OK;
  DeviceGuard guard(ctx->device);
  cudaDeviceSynchronize();
  void* ptrs[] = {ctx->split_partial, ctx->split_flags,
                  ctx->counts_scratch, ctx->ticket, ctx->status, ctx->tile_counts, ctx->super_counts, ctx->st_hprev, ctx->st_H,
                  ctx->st_pi, ctx->st_pi_out, ctx->st_counts, ctx->st_swaps, ctx->st_nswaps, ctx->st_load_before,
                  ctx->st_load_after, ctx->st_ids, ctx->st_w, ctx->st_slot_offsets, ctx->st_rank_offsets,
                  ctx->st_perm, ctx->st_inv_perm, ctx->st_rank_load};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  if (ctx->mig_stage) cudaFree(ctx->mig_stage);
  if (ctx->mig_host) cudaFreeHost(ctx->mig_host);
  for (auto& a : ctx->attn) {
    if (a.e0) cudaEventDestroy(a.e0);
    if (a.e1) cudaEventDestroy(a.e1);
  }
  delete ctx;
  return FB_OK;
}

fb_status fb_predict_load(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T, uint32_t* counts,
                          int32_t* topk_ids, float* logits, fb_stream stream_) {
  if (!ctx || !router || !router->W || !counts || T < 0) return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && !x) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  if (T == 0)
    return cudaMemsetAsync(counts, 0, ctx->cfg.E * sizeof(uint32_t), stream) == cudaSuccess ? FB_OK : FB_ERR_CUDA;
  return launch_router(ctx, router, x, T, fb::kModePredict, counts, topk_ids, nullptr, logits, nullptr, stream);
}

fb_status fb_plan_swaps(fb_ctx* ctx, const uint32_t* counts, const int32_t* expert_to_slot, const fb_budget* budget,
                        int32_t layer_id, int32_t* expert_to_slot_out, fb_swap* swaps, int32_t* n_swaps,
                        uint32_t* load_before, uint32_t* load_after, fb_stream stream_) {
  (void)layer_id;   // constant within a call: it leads the tie-break tuple but cannot change the order
  if (!ctx || !counts) return FB_ERR_INVALID_ARG;
  fb::PlanParams pp;
  memset(&pp, 0, sizeof(pp));
  const fb_status st = fill_plan(ctx, budget, expert_to_slot, expert_to_slot_out, swaps, n_swaps, load_before,
                                 load_after, &pp);
  if (st != FB_OK) return st;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  return launch_plan(ctx, pp, counts, static_cast<cudaStream_t>(stream_));
}

fb_status fb_predict_and_plan(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T,
                              const int32_t* expert_to_slot, const fb_budget* budget, int32_t layer_id,
                              uint32_t* counts, int32_t* expert_to_slot_out, fb_swap* swaps, int32_t* n_swaps,
                              uint32_t* load_before, uint32_t* load_after, fb_stream stream_) {
  (void)layer_id;
  if (!ctx || !router || !router->W || !counts || T < 0) return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && !x) return FB_ERR_INVALID_ARG;
  fb::PlanParams pp;
  memset(&pp, 0, sizeof(pp));
  const fb_status st = fill_plan(ctx, budget, expert_to_slot, expert_to_slot_out, swaps, n_swaps, load_before,
                                 load_after, &pp);
  if (st != FB_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  if (T == 0) {
    if (cudaMemsetAsync(counts, 0, ctx->cfg.E * sizeof(uint32_t), stream) != cudaSuccess) return FB_ERR_CUDA;
    return launch_plan(ctx, pp, counts, stream);
  }
  return launch_router(ctx, router, x, T, fb::kModePredictPlan, counts, nullptr, nullptr, nullptr, &pp, stream);
}

fb_status fb_route_dispatch(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T,
                            const int32_t* expert_to_slot, int32_t* topk_ids, float* topk_w, uint32_t* slot_offsets,
                            uint32_t* rank_offsets, int32_t* perm, int32_t* inv_perm, uint32_t* rank_load,
                            float* logits, fb_stream stream_) {
  if (!ctx || !router || !router->W || !expert_to_slot || !slot_offsets || !rank_offsets || !rank_load || T < 0)
    return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && (!x || !topk_ids || !topk_w || !perm || !inv_perm)) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  const fb_config& c = ctx->cfg;
  if (T == 0) {
    if (cudaMemsetAsync(slot_offsets, 0, (c.E + 1) * sizeof(uint32_t), stream) != cudaSuccess ||
        cudaMemsetAsync(rank_offsets, 0, (c.R + 1) * sizeof(uint32_t), stream) != cudaSuccess ||
        cudaMemsetAsync(rank_load, 0, c.R * sizeof(uint32_t), stream) != cudaSuccess)
      return FB_ERR_CUDA;
    return FB_OK;
  }
  const fb_status st = launch_router(ctx, router, x, T, fb::kModeDispatch, nullptr, topk_ids, topk_w, logits,
                                     nullptr, stream);
  if (st != FB_OK) return st;
  return launch_dispatch_index(ctx, T, expert_to_slot, topk_ids, slot_offsets, rank_offsets, perm, inv_perm,
                               rank_load, stream);
}

fb_status fb_layer_step(fb_ctx* ctx, const fb_router* router, const void* h_prev, const void* H, int32_t T,
                        const int32_t* expert_to_slot, const fb_budget* budget, int32_t layer_id,
                        uint32_t* counts, int32_t* expert_to_slot_out, fb_swap* swaps, int32_t* n_swaps,
                        uint32_t* load_before, uint32_t* load_after, int32_t* topk_ids, float* topk_w,
                        uint32_t* slot_offsets, uint32_t* rank_offsets, int32_t* perm, int32_t* inv_perm,
                        uint32_t* rank_load, fb_stream stream_) {
  (void)layer_id;
  if (!ctx || !router || !router->W || !counts || !slot_offsets || !rank_offsets || !rank_load || T < 0)
    return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && (!h_prev || !H || !topk_ids || !topk_w || !perm || !inv_perm)) return FB_ERR_INVALID_ARG;
  if (T == 0) {
    const fb_status st0 = fb_predict_and_plan(ctx, router, h_prev, 0, expert_to_slot, budget, layer_id, counts,
                                              expert_to_slot_out, swaps, n_swaps, load_before, load_after, stream_);
    if (st0 != FB_OK) return st0;
    return fb_route_dispatch(ctx, router, H, 0, expert_to_slot_out, topk_ids, topk_w, slot_offsets, rank_offsets,
                             perm, inv_perm, rank_load, nullptr, stream_);
  }
  fb::PlanParams pp;
  memset(&pp, 0, sizeof(pp));
  fb_status st = fill_plan(ctx, budget, expert_to_slot, expert_to_slot_out, swaps, n_swaps, load_before, load_after,
                           &pp);
  if (st != FB_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  // one launch for both router passes; the dispatch index needs the new placement and follows
  st = launch_router(ctx, router, h_prev, T, fb::kModeLayer, counts, topk_ids, topk_w, nullptr, &pp, stream, H);
  if (st != FB_OK) return st;
  return launch_dispatch_index(ctx, T, expert_to_slot_out, topk_ids, slot_offsets, rank_offsets, perm, inv_perm,
                               rank_load, stream);
}

fb_status fb_layer_step_host(fb_ctx* ctx, const fb_router* router, const void* h_prev_host, const void* H_host,
                             int32_t T, const int32_t* expert_to_slot_host, const fb_budget* budget,
                             int32_t layer_id, uint32_t* counts, int32_t* expert_to_slot_out, fb_swap* swaps,
                             int32_t* n_swaps, uint32_t* load_before, uint32_t* load_after, int32_t* topk_ids,
                             float* topk_w, uint32_t* slot_offsets, uint32_t* rank_offsets, int32_t* perm,
                             int32_t* inv_perm, uint32_t* rank_load, fb_stream stream_) {
  if (!ctx || !router || !expert_to_slot_host || !budget || T < 0) return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && (!h_prev_host || !H_host)) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  const fb_config& c = ctx->cfg;
  const size_t Tm = static_cast<size_t>(c.T_max), E = c.E, R = c.R, k = c.k;
  if (!ctx->staged) {
    const size_t act = Tm * c.d * 2;
    bool ok = cudaMalloc(&ctx->st_hprev, act ? act : 16) == cudaSuccess &&
              cudaMalloc(&ctx->st_H, act ? act : 16) == cudaSuccess;
    ok = ok && dev_alloc(&ctx->st_pi, E) && dev_alloc(&ctx->st_pi_out, E) && dev_alloc(&ctx->st_counts, E) &&
         dev_alloc(&ctx->st_swaps, E / 2 + 1) && dev_alloc(&ctx->st_nswaps, 1) &&
         dev_alloc(&ctx->st_load_before, R) && dev_alloc(&ctx->st_load_after, R) &&
         dev_alloc(&ctx->st_ids, Tm * k) && dev_alloc(&ctx->st_w, Tm * k) &&
         dev_alloc(&ctx->st_slot_offsets, E + 1) && dev_alloc(&ctx->st_rank_offsets, R + 1) &&
         dev_alloc(&ctx->st_perm, Tm * k) && dev_alloc(&ctx->st_inv_perm, Tm * k) &&
         dev_alloc(&ctx->st_rank_load, R);
    if (!ok) return FB_ERR_CUDA;
    ctx->staged = true;
  }
  const size_t act_bytes = static_cast<size_t>(T) * c.d * 2;
  const size_t n_assign = static_cast<size_t>(T) * k;
  bool ok = true;
  if (T > 0) {
    ok = ok && cudaMemcpyAsync(ctx->st_hprev, h_prev_host, act_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ctx->st_H, H_host, act_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(ctx->st_pi, expert_to_slot_host, E * sizeof(int32_t), cudaMemcpyHostToDevice, stream) ==
                 cudaSuccess;
  if (!ok) return FB_ERR_CUDA;
  const fb_status st = fb_layer_step(ctx, router, ctx->st_hprev, ctx->st_H, T, ctx->st_pi, budget, layer_id,
                                     ctx->st_counts, ctx->st_pi_out, ctx->st_swaps, ctx->st_nswaps,
                                     ctx->st_load_before, ctx->st_load_after, ctx->st_ids, ctx->st_w,
                                     ctx->st_slot_offsets, ctx->st_rank_offsets, ctx->st_perm, ctx->st_inv_perm,
                                     ctx->st_rank_load, stream);
  if (st != FB_OK) return st;
  auto back = [&](void* dst, const void* src, size_t bytes) {
    if (dst && bytes) ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  };
  back(counts, ctx->st_counts, E * sizeof(uint32_t));
  back(expert_to_slot_out, ctx->st_pi_out, E * sizeof(int32_t));
  back(swaps, ctx->st_swaps, budget->max_swaps * sizeof(fb_swap));
  back(n_swaps, ctx->st_nswaps, sizeof(int32_t));
  back(load_before, ctx->st_load_before, R * sizeof(uint32_t));
  back(load_after, ctx->st_load_after, R * sizeof(uint32_t));
  back(topk_ids, ctx->st_ids, n_assign * sizeof(int32_t));
  back(topk_w, ctx->st_w, n_assign * sizeof(float));
  back(slot_offsets, ctx->st_slot_offsets, (E + 1) * sizeof(uint32_t));
  back(rank_offsets, ctx->st_rank_offsets, (R + 1) * sizeof(uint32_t));
  back(perm, ctx->st_perm, n_assign * sizeof(int32_t));
  back(inv_perm, ctx->st_inv_perm, n_assign * sizeof(int32_t));
  back(rank_load, ctx->st_rank_load, R * sizeof(uint32_t));
  if (!ok) return FB_ERR_CUDA;
  return cudaStreamSynchronize(stream) == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_device_status(fb_ctx* ctx, int32_t* word, fb_stream stream_) {
  if (!ctx || !word) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FB_ERR_CUDA;
  if (cudaMemcpy(word, ctx->status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return FB_ERR_CUDA;
  if (*word != 0) {
    if (cudaMemset(ctx->status, 0, sizeof(int32_t)) != cudaSuccess) return FB_ERR_CUDA;
    // a launch that gave up may have left partial-tile flags of the k-range split set: re-arm them
    if (ctx->split_flags != nullptr &&
        cudaMemset(ctx->split_flags, 0, static_cast<size_t>(ctx->split_pairs) * 2 * sizeof(uint32_t)) != cudaSuccess)
      return FB_ERR_CUDA;
  }
  return FB_OK;
}

uint64_t fb_launch_count(const fb_ctx* ctx) { return ctx ? ctx->launches : 0; }

fb_status fb_apply_swaps(void* slot_weights, uint64_t expert_bytes, int32_t E, const int32_t* expert_to_slot,
                         const fb_swap* swaps, const int32_t* n_swaps, int32_t max_swaps, int32_t* status_word,
                         fb_stream stream_) {
  if (E < 1 || E > FB_MAX_EXPERTS || max_swaps < 0 || expert_bytes % 16 != 0) return FB_ERR_INVALID_ARG;
  if (max_swaps == 0 || expert_bytes == 0) return FB_OK;
  if (!slot_weights || !expert_to_slot || !swaps || !n_swaps) return FB_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(slot_weights) % 16 != 0) return FB_ERR_INVALID_ARG;
  // the launch goes to the device that holds the weights, whichever device is current
  const int device = device_of(slot_weights);
  if (device < 0) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  fb::MigrateParams mp;
  mp.slot_weights = static_cast<uint8_t*>(slot_weights);
  mp.expert_bytes = expert_bytes;
  mp.E = E;
  mp.expert_to_slot = expert_to_slot;
  mp.swaps = swaps;
  mp.n_swaps = n_swaps;
  mp.status = status_word;
  mp.max_swaps = max_swaps;
  mp.copy_bytes = expert_bytes;
  const uint64_t per_piece = static_cast<uint64_t>(fb::kMigrateThreads) * fb::kMigrateUnroll * 16;
  uint64_t units = (expert_bytes + per_piece - 1) / per_piece * static_cast<uint64_t>(max_swaps);
  if (units > fb::kMigrateBlocks) units = fb::kMigrateBlocks;
  const dim3 grid(static_cast<unsigned>(units), 1, 1);
  fb::fb_swap_weights_kernel<<<grid, fb::kMigrateThreads, 0, static_cast<cudaStream_t>(stream_)>>>(mp);
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_fit_cost_model(uint64_t t_small_ns, uint64_t t_large_ns, uint64_t bytes_small, uint64_t bytes_large,
                            uint64_t* alpha_ns, uint64_t* fs_per_byte) {
  if (!alpha_ns || !fs_per_byte || bytes_large <= bytes_small || t_large_ns <= t_small_ns) return FB_ERR_INVALID_ARG;
  const unsigned __int128 d_bytes = static_cast<unsigned __int128>(2) * (bytes_large - bytes_small);
  const unsigned __int128 d_t = t_large_ns - t_small_ns;
  const unsigned __int128 fs = (d_t * 1000000u + d_bytes - 1) / d_bytes;             // 1 / beta, rounded up
  if (fs > ~static_cast<uint64_t>(0)) return FB_ERR_RANGE;
  // alpha = t_small - 2 S_small * d_t / d_bytes, rounded down, not below zero
  const unsigned __int128 lhs = static_cast<unsigned __int128>(t_small_ns) * d_bytes;
  const unsigned __int128 rhs = static_cast<unsigned __int128>(2) * bytes_small * d_t;
  *alpha_ns = lhs > rhs ? static_cast<uint64_t>((lhs - rhs) / d_bytes) : 0;
  *fs_per_byte = static_cast<uint64_t>(fs);
  return FB_OK;
}

fb_status fb_calibrate_exchange(void* slot_weights, uint64_t bytes_small, uint64_t bytes_large, int32_t reps,
                                uint64_t* alpha_ns, uint64_t* fs_per_byte, uint64_t* t_small_ns_out,
                                uint64_t* t_large_ns_out, fb_stream stream_) {
  if (!slot_weights || !alpha_ns || !fs_per_byte || reps < 1 || reps > 1000 || bytes_small == 0 ||
      bytes_small % 16 != 0 || bytes_large % 16 != 0 || bytes_large <= bytes_small)
    return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int device = device_of(slot_weights);
  if (device < 0) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  // a one-swap plan over two slots: constant data of the library image on this device
  const int32_t* plan = nullptr;                 // [pi: 2][swap: 4][n: 1]
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(const_cast<int32_t**>(&plan)), g_calibration_plan) !=
          cudaSuccess || plan == nullptr)
    return FB_ERR_CUDA;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  bool ok = cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess;
  uint64_t t_ns[2] = {0, 0};
  const uint64_t sizes[2] = {bytes_small, bytes_large};
  for (int which = 0; which < 2 && ok; ++which) {
    // the two images lie bytes_large apart for both sizes: the same addresses are warm in both runs
    float best = 0.0f;
    for (int r = 0; r < reps + 2 && ok; ++r) {
      ok = cudaEventRecord(e0, stream) == cudaSuccess;
      fb::MigrateParams mp;
      mp.slot_weights = static_cast<uint8_t*>(slot_weights);
      mp.expert_bytes = bytes_large;             // slot stride
      mp.E = 2;
      mp.expert_to_slot = plan;
      mp.swaps = reinterpret_cast<const fb_swap*>(plan + 2);
      mp.n_swaps = plan + 6;
      mp.max_swaps = 1;
      mp.status = nullptr;
      mp.copy_bytes = sizes[which];
      const uint64_t per_piece = static_cast<uint64_t>(fb::kMigrateThreads) * fb::kMigrateUnroll * 16;
      uint64_t units = (sizes[which] + per_piece - 1) / per_piece;
      if (units > fb::kMigrateBlocks) units = fb::kMigrateBlocks;
      fb::fb_swap_weights_kernel<<<static_cast<unsigned>(units), fb::kMigrateThreads, 0, stream>>>(mp);
      ok = ok && cudaEventRecord(e1, stream) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess;
      float ms = 0.0f;
      ok = ok && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess;
      if (r >= 2 && (best == 0.0f || ms < best)) best = ms;          // first two runs warm up; keep the fastest
    }
    t_ns[which] = static_cast<uint64_t>(best * 1e6f);
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (!ok) return FB_ERR_CUDA;
  if (t_small_ns_out) *t_small_ns_out = t_ns[0];
  if (t_large_ns_out) *t_large_ns_out = t_ns[1];
  return fb_fit_cost_model(t_ns[0], t_ns[1], bytes_small, bytes_large, alpha_ns, fs_per_byte);
}

fb_status fb_apply_swaps_staged(fb_ctx* ctx, void* slot_weights, uint64_t expert_bytes, const int32_t* expert_to_slot,
                                const fb_swap* swaps, const int32_t* n_swaps, int32_t max_swaps,
                                uint64_t staging_bytes, fb_stream plan_stream_, fb_stream copy_stream_) {
  if (!ctx || max_swaps < 0 || max_swaps > FB_MAX_EXPERTS / 2) return FB_ERR_INVALID_ARG;
  if (max_swaps == 0 || expert_bytes == 0) return FB_OK;
  if (!slot_weights || !expert_to_slot || !swaps || !n_swaps) return FB_ERR_INVALID_ARG;
  cudaStream_t plan_stream = static_cast<cudaStream_t>(plan_stream_);
  cudaStream_t copy_stream = static_cast<cudaStream_t>(copy_stream_);
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  const int E = ctx->cfg.E;
  if (staging_bytes == 0 || staging_bytes > expert_bytes) staging_bytes = expert_bytes;
  // host copy of the plan: [n_swaps][swaps: max_swaps][placement: E]
  const size_t host_bytes = sizeof(int32_t) * (1 + 4 * static_cast<size_t>(FB_MAX_EXPERTS / 2) + FB_MAX_EXPERTS);
  if (!ctx->mig_host && cudaMallocHost(&ctx->mig_host, host_bytes) != cudaSuccess) return FB_ERR_CUDA;
  if (ctx->mig_stage_bytes < staging_bytes) {
    if (ctx->mig_stage) { cudaStreamSynchronize(copy_stream); cudaFree(ctx->mig_stage); ctx->mig_stage = nullptr; }
    if (cudaMalloc(&ctx->mig_stage, staging_bytes) != cudaSuccess) { ctx->mig_stage_bytes = 0; return FB_ERR_CUDA; }
    ctx->mig_stage_bytes = staging_bytes;
  }
  int32_t* h_n = static_cast<int32_t*>(ctx->mig_host);
  fb_swap* h_swaps = reinterpret_cast<fb_swap*>(h_n + 1);
  int32_t* h_pi = h_n + 1 + 4 * (FB_MAX_EXPERTS / 2);
  bool ok = cudaMemcpyAsync(h_n, n_swaps, sizeof(int32_t), cudaMemcpyDeviceToHost, plan_stream) == cudaSuccess &&
            cudaMemcpyAsync(h_swaps, swaps, sizeof(fb_swap) * max_swaps, cudaMemcpyDeviceToHost, plan_stream) ==
                cudaSuccess &&
            cudaMemcpyAsync(h_pi, expert_to_slot, sizeof(int32_t) * E, cudaMemcpyDeviceToHost, plan_stream) ==
                cudaSuccess &&
            cudaStreamSynchronize(plan_stream) == cudaSuccess;       // the host needs the plan to issue the copies
  if (!ok) return FB_ERR_CUDA;
  const int n = *h_n;
  if (n < 0 || n > max_swaps) return FB_ERR_RANGE;
  uint8_t* base = static_cast<uint8_t*>(slot_weights);
  for (int i = 0; i < n; ++i) {
    const int ea = h_swaps[i].expert_src, eb = h_swaps[i].expert_dst;
    if (ea < 0 || ea >= E || eb < 0 || eb >= E || ea == eb) return FB_ERR_RANGE;
    const int pa = h_pi[ea], pb = h_pi[eb];
    if (pa < 0 || pa >= E || pb < 0 || pb >= E || pa == pb) return FB_ERR_BAD_PLACEMENT;
    uint8_t* A = base + static_cast<uint64_t>(pa) * expert_bytes;
    uint8_t* Bp = base + static_cast<uint64_t>(pb) * expert_bytes;
    // pairwise exchange through the bounded staging buffer, one piece at a time
    for (uint64_t off = 0; off < expert_bytes; off += staging_bytes) {
      const uint64_t len = expert_bytes - off < staging_bytes ? expert_bytes - off : staging_bytes;
      ok = ok && cudaMemcpyAsync(ctx->mig_stage, A + off, len, cudaMemcpyDeviceToDevice, copy_stream) == cudaSuccess &&
           cudaMemcpyAsync(A + off, Bp + off, len, cudaMemcpyDeviceToDevice, copy_stream) == cudaSuccess &&
           cudaMemcpyAsync(Bp + off, ctx->mig_stage, len, cudaMemcpyDeviceToDevice, copy_stream) == cudaSuccess;
    }
  }
  return ok ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_row_cosine_mean(const void* a, const void* b, int64_t rows, int32_t n, int32_t dtype,
                             double* row_scratch, double* mean_out, fb_stream stream_) {
  if (rows < 0 || n <= 0 || (dtype != FB_DTYPE_BF16 && dtype != FB_DTYPE_F32) || !mean_out) return FB_ERR_INVALID_ARG;
  if (rows > 0 && (!a || !b || !row_scratch)) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (rows > 0) {
    const unsigned blocks = static_cast<unsigned>((rows + fb::kCosineWarpsPerBlock - 1) / fb::kCosineWarpsPerBlock);
    if (dtype == FB_DTYPE_BF16)
      fb::fb_row_cosine_kernel<__nv_bfloat16><<<blocks, 32 * fb::kCosineWarpsPerBlock, 0, stream>>>(
          static_cast<const __nv_bfloat16*>(a), static_cast<const __nv_bfloat16*>(b), rows, n, row_scratch);
    else
      fb::fb_row_cosine_kernel<float><<<blocks, 32 * fb::kCosineWarpsPerBlock, 0, stream>>>(
          static_cast<const float*>(a), static_cast<const float*>(b), rows, n, row_scratch);
  }
  fb::fb_mean_kernel<<<1, fb::kMeanThreads, 0, stream>>>(row_scratch, rows, mean_out);
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_topk_hits(const int32_t* ids_a, const int32_t* ids_b, int32_t T, int32_t k, uint32_t* hits_out,
                       fb_stream stream_) {
  if (T < 0 || k < 1 || k > FB_MAX_TOPK || !hits_out || (T > 0 && (!ids_a || !ids_b))) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (cudaMemsetAsync(hits_out, 0, sizeof(uint32_t), stream) != cudaSuccess) return FB_ERR_CUDA;
  if (T > 0) fb::fb_topk_hits_kernel<<<(T + 255) / 256, 256, 0, stream>>>(ids_a, ids_b, T, k, hits_out);
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_set_split(fb_ctx* ctx, int32_t mode, int32_t owner_bias_kblocks) {
  if (!ctx || (mode != 0 && mode != 1) || owner_bias_kblocks < -1 || owner_bias_kblocks > 1024) return FB_ERR_INVALID_ARG;
  ctx->split_mode = mode;
  ctx->split_bias = owner_bias_kblocks;
  return FB_OK;
}

fb_status fb_set_stage_limit(fb_ctx* ctx, int32_t stages) {
  if (!ctx || stages < 0 || stages == 1) return FB_ERR_INVALID_ARG;
  ctx->stage_limit = stages;
  return FB_OK;
}

fb_status fb_set_pair_limit(fb_ctx* ctx, int32_t pairs) {
  if (!ctx || pairs < 0) return FB_ERR_INVALID_ARG;
  ctx->pair_limit = pairs;
  return FB_OK;
}

fb_status fb_time_next_router_launch(fb_ctx* ctx, void* event_before, void* event_after) {
  if (!ctx) return FB_ERR_INVALID_ARG;
  ctx->ev_before = static_cast<cudaEvent_t>(event_before);
  ctx->ev_after = static_cast<cudaEvent_t>(event_after);
  return FB_OK;
}

fb_status fb_router_floor(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T, int32_t what,
                          fb_stream stream_) {
  if (!ctx || !router || !router->W || !x || T <= 0 || (what != 1 && what != 2
       )) return FB_ERR_INVALID_ARG;
  if (T > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  return launch_router(ctx, router, x, T, fb::kModePredict, nullptr, nullptr, nullptr, nullptr, nullptr,
                       static_cast<cudaStream_t>(stream_), nullptr, what);
}

int32_t fb_max_pairs(const fb_ctx* ctx) { return ctx ? ctx->max_pairs : 0; }

fb_status fb_dispatch_slot_counts(fb_ctx* ctx, const uint32_t* slot_offsets, uint32_t* slot_counts, fb_stream stream_) {
  if (!ctx || !slot_offsets || !slot_counts) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  fb::fb_slot_counts_kernel<<<1, FB_MAX_EXPERTS, 0, static_cast<cudaStream_t>(stream_)>>>(slot_offsets, ctx->cfg.E,
                                                                                          slot_counts);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_dispatch_globalize(fb_ctx* ctx, int32_t T_local, int32_t world, int32_t rank,
                                const uint32_t* slot_counts_all, const uint32_t* slot_offsets_local,
                                const int32_t* topk_ids, const int32_t* expert_to_slot, int32_t* inv_perm,
                                uint32_t* slot_offsets, uint32_t* rank_offsets, uint32_t* rank_load,
                                fb_stream stream_) {
  if (!ctx || T_local < 0 || world < 1 || world > 4096 || rank < 0 || rank >= world || !slot_counts_all ||
      !slot_offsets_local || !expert_to_slot || !slot_offsets || !rank_offsets || !rank_load)
    return FB_ERR_INVALID_ARG;
  if (T_local > ctx->cfg.T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T_local > 0 && (!topk_ids || !inv_perm)) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  fb::GlobalizeParams gp;
  gp.T = T_local; gp.k = ctx->cfg.k; gp.E = ctx->cfg.E; gp.R = ctx->cfg.R; gp.world = world; gp.rank = rank;
  gp.counts_all = slot_counts_all; gp.local_offsets = slot_offsets_local; gp.topk_ids = topk_ids;
  gp.expert_to_slot = expert_to_slot; gp.inv_perm = inv_perm;
  gp.slot_offsets = slot_offsets; gp.rank_offsets = rank_offsets; gp.rank_load = rank_load;
  const long long n = static_cast<long long>(T_local) * ctx->cfg.k;
  long long blocks = (n + fb::kGlobalizeThreads - 1) / fb::kGlobalizeThreads;
  if (blocks < 1) blocks = 1;
  if (blocks > 2 * ctx->dispatch_blocks_max) blocks = 2 * ctx->dispatch_blocks_max;
  fb::fb_dispatch_globalize_kernel<<<static_cast<unsigned>(blocks), fb::kGlobalizeThreads, 0,
                                     static_cast<cudaStream_t>(stream_)>>>(gp);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_attention_begin(fb_ctx* ctx, int32_t layer_id, int32_t attn_type, fb_stream stream_) {
  if (!ctx || attn_type < 0 || attn_type >= FB_MAX_ATTENTION_TYPES || layer_id < 0) return FB_ERR_INVALID_ARG;
  fb_ctx::AttnSlot& a = ctx->attn[attn_type];
  if (a.layer >= 0) return FB_OK;                      // this type already has its r(l)
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  if (!a.e0 && cudaEventCreate(&a.e0) != cudaSuccess) return FB_ERR_CUDA;
  if (!a.e1 && cudaEventCreate(&a.e1) != cudaSuccess) return FB_ERR_CUDA;
  if (cudaEventRecord(a.e0, static_cast<cudaStream_t>(stream_)) != cudaSuccess) return FB_ERR_CUDA;
  a.layer = layer_id;
  a.open = true;
  return FB_OK;
}

fb_status fb_attention_end(fb_ctx* ctx, int32_t layer_id, int32_t attn_type, fb_stream stream_) {
  if (!ctx || attn_type < 0 || attn_type >= FB_MAX_ATTENTION_TYPES || layer_id < 0) return FB_ERR_INVALID_ARG;
  fb_ctx::AttnSlot& a = ctx->attn[attn_type];
  if (!a.open || a.layer != layer_id) return FB_OK;    // not the layer being measured
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  if (cudaEventRecord(a.e1, static_cast<cudaStream_t>(stream_)) != cudaSuccess) return FB_ERR_CUDA;
  a.open = false;
  a.pending = true;
  return FB_OK;
}

fb_status fb_layer_budget_ns(fb_ctx* ctx, int32_t attn_type, uint64_t delta_ns, uint64_t* budget_ns,
                             int32_t* profiled_layer) {
  if (!ctx || !budget_ns || attn_type < 0 || attn_type >= FB_MAX_ATTENTION_TYPES) return FB_ERR_INVALID_ARG;
  fb_ctx::AttnSlot& a = ctx->attn[attn_type];
  if (a.pending) {
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FB_ERR_CUDA;
    float ms = 0.0f;
    if (cudaEventSynchronize(a.e1) != cudaSuccess || cudaEventElapsedTime(&ms, a.e0, a.e1) != cudaSuccess)
      return FB_ERR_CUDA;
    a.t_ns = static_cast<uint64_t>(static_cast<double>(ms) * 1e6 + 0.5);
    a.pending = false;
    a.has_time = true;
  }
  if (!a.has_time) return FB_ERR_INVALID_ARG;          // never profiled (or the region is still open)
  *budget_ns = fb_budget_ns(a.t_ns, delta_ns);         // Eq. 10
  if (profiled_layer) *profiled_layer = a.layer;
  return FB_OK;
}

fb_status fb_attention_set_time_ns(fb_ctx* ctx, int32_t attn_type, int32_t layer_id, uint64_t t_attn_ns) {
  if (!ctx || attn_type < 0 || attn_type >= FB_MAX_ATTENTION_TYPES || layer_id < 0) return FB_ERR_INVALID_ARG;
  fb_ctx::AttnSlot& a = ctx->attn[attn_type];
  a.layer = layer_id;
  a.t_ns = t_attn_ns;
  a.open = a.pending = false;
  a.has_time = true;
  return FB_OK;
}

fb_status fb_attention_reset(fb_ctx* ctx) {
  if (!ctx) return FB_ERR_INVALID_ARG;
  for (auto& a : ctx->attn) { a.layer = -1; a.open = a.pending = a.has_time = false; a.t_ns = 0; }
  return FB_OK;
}

fb_status fb_standin_attention(float* out, int32_t blocks, int32_t iters, fb_stream stream_) {
  if (!out || blocks < 1 || blocks > 1024 || iters < 0 || iters > (1 << 24)) return FB_ERR_INVALID_ARG;
  const int device = device_of(out);
  if (device < 0) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  static bool raised[64] = {};
  if (device < 64 && !raised[device]) {
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(fb::fb_standin_attention_kernel),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, fb::kStandinSmemBytes) != cudaSuccess)
      return FB_ERR_CUDA;
    raised[device] = true;
  }
  fb::fb_standin_attention_kernel<<<static_cast<unsigned>(blocks), fb::kStandinThreads, fb::kStandinSmemBytes,
                                    static_cast<cudaStream_t>(stream_)>>>(out, iters);
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_clock_probe(uint64_t* samples, int32_t n, uint32_t period_ns, fb_stream stream_) {
  // bounded by construction: at most 65536 samples, at most 100 us apart
  if (!samples || n < 1 || n > 65536 || period_ns > 100000) return FB_ERR_INVALID_ARG;
  const int device = device_of(samples);
  if (device < 0) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  // The split between L1 and shared memory is a per-SM setting that only changes while the SM is
  // idle: a resident block of a kernel that prefers a small shared-memory share would keep the
  // router kernel's blocks (over 200 KB of shared memory each) off its SM for as long as it runs.
  static bool carveout_set[64] = {};
  if (device < 64 && !carveout_set[device]) {
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(fb::fb_clock_probe_kernel),
                             cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
      return FB_ERR_CUDA;
    carveout_set[device] = true;
  }
  fb::fb_clock_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_)>>>(
      reinterpret_cast<unsigned long long*>(samples), n, period_ns);
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

fb_status fb_set_stamp_buffer(fb_ctx* ctx, uint64_t* stamps) {
  if (!ctx) return FB_ERR_INVALID_ARG;
#ifdef FB_TIMING
  ctx->stamps = reinterpret_cast<unsigned long long*>(stamps);
  return FB_OK;
#else
  (void)stamps;
  return FB_ERR_UNSUPPORTED_SHAPE;      // this build carries no stamp code
#endif
}

fb_status fb_selftest_wait_timeout(fb_ctx* ctx, uint64_t limit_ns, uint64_t* waited_ns, fb_stream stream_) {
  if (!ctx || limit_ns == 0 || limit_ns > 100ull * 1000 * 1000) return FB_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return FB_ERR_CUDA;
  fb::fb_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_)>>>(limit_ns, ctx->status, waited_ns);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? FB_OK : FB_ERR_CUDA;
}

uint64_t fb_persistent_launch_count(const fb_ctx* ctx) { return ctx ? ctx->persistent_launches : 0; }

}  // extern "C"

// ---------------------------------------------------------------------------------
// fb_predict_load_static: the prediction pass for callers that must not allocate.
// Its scratch (the cross-block histogram, the finished-block ticket and a status word)
// lives in a fixed array inside the library image instead of in an fb_ctx.
// ---------------------------------------------------------------------------------
namespace {

constexpr int kStaticScratchWords = FB_STATIC_MAX_EXPERTS + 64;
constexpr int kStaticMaxDevices = 64;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) uint32_t g_static_scratch[kStaticScratchWords];

struct StaticState {
  bool ready = false;
  uint32_t* scratch = nullptr;      // device address of g_static_scratch on this device
  fb_ctx ctx;                       // host-side launch state only; owns no device memory
};
StaticState g_static_state[kStaticMaxDevices];

}  // namespace

extern "C" fb_status fb_predict_load_static(const fb_config* cfg, int device, const fb_router* router,
                                            const void* x, int32_t T, uint32_t* counts, int32_t* topk_ids,
                                            int32_t* status_word, fb_stream stream_) {
  if (!cfg || !router || !router->W || !counts || T < 0) return FB_ERR_INVALID_ARG;
  if (cfg->E > FB_STATIC_MAX_EXPERTS) return FB_ERR_UNSUPPORTED_SHAPE;   // scratch array too small
  const fb_status cs = check_config(*cfg);
  if (cs != FB_OK) return cs;
  if (T > cfg->T_max) return FB_ERR_UNSUPPORTED_SHAPE;
  if (T > 0 && !x) return FB_ERR_INVALID_ARG;
  if (device < 0 || device >= kStaticMaxDevices) return FB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(device);
  if (!guard.ok) return FB_ERR_CUDA;
  StaticState& st = g_static_state[device];
  if (!st.ready) {
    // One-time set-up for this device, with the device current.  In host code the name
    // of a __device__ array is only a handle: the address a kernel can use has to be
    // asked for.
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess || prop.major != 10) return FB_ERR_CUDA;
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || addr == nullptr) return FB_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr)
      return FB_ERR_CUDA;
    st.scratch = static_cast<uint32_t*>(addr);
    st.ctx.encode = reinterpret_cast<EncodeTiledFn>(fn);
    st.ctx.device = device;
    st.ctx.cfg.E = -1;                                   // forces the shape-dependent part below
    st.ready = true;
  }
  fb_ctx& ctx = st.ctx;
  if (memcmp(&ctx.cfg, cfg, sizeof(fb_config)) != 0) {
    // shape-dependent launch parameters (host arithmetic and function attributes only)
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FB_ERR_CUDA;
    ctx.cfg = *cfg;
    fb_status ss = setup_router_shape(&ctx, prop);
    if (ss == FB_OK) ss = ensure_kernel_attributes(device, prop);
    if (ss != FB_OK) { ctx.cfg.E = -1; return ss; }
    for (int i = 0; i < kMapCache; ++i) { ctx.x_maps[i] = MapEntry(); ctx.w_maps[i] = MapEntry(); }
  }
  ctx.counts_scratch = st.scratch;
  ctx.ticket = st.scratch + FB_STATIC_MAX_EXPERTS;
  ctx.status = status_word ? status_word : reinterpret_cast<int32_t*>(st.scratch + FB_STATIC_MAX_EXPERTS + 1);
  ctx.tile_counts = nullptr;                             // unused by the prediction pass
  if (T == 0)
    return cudaMemsetAsync(counts, 0, cfg->E * sizeof(uint32_t), stream) == cudaSuccess ? FB_OK : FB_ERR_CUDA;
  // The array keeps whatever the previous call (possibly one that was cut short) left in it.
  if (cudaMemsetAsync(st.scratch, 0, kStaticScratchWords * sizeof(uint32_t), stream) != cudaSuccess)
    return FB_ERR_CUDA;
  return launch_router(&ctx, router, x, T, fb::kModePredict, counts, topk_ids, nullptr, nullptr, nullptr, stream);
}
