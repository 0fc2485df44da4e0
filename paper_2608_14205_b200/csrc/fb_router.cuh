// Fused router kernel: logits = x W^T (+ b) on tcgen05 tensor cores with fp32
// accumulators in tensor memory, fed by TMA; then, straight out of tensor memory, the
// model's gating rule, top-k, and a per-expert histogram (Eqs. 2-5).  The block that
// finishes last publishes the count vector and, when asked, runs the swap planner.
//
// One block owns 128 token rows and all N = pad16(E) expert columns.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns the TMEM allocation),
// warps 2..5 = epilogue, one thread per token row.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fb_planner.cuh"
#include "fb_ptx.cuh"

namespace fb {

constexpr int kTileM = 128;            // token rows per block
constexpr int kBlockK = 64;            // bf16 elements per k-block = one 128-byte swizzled row
constexpr int kUmmaK = 16;             // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxStages = 8;
constexpr int kRouterThreads = 192;
constexpr int kEpilogueThreads = 128;
constexpr int kATileBytes = kTileM * kBlockK * 2;

enum RouterMode : int {
  kModePredict = 0,        // histogram -> counts
  kModePredictPlan = 1,    // histogram -> counts -> planner in the last block
  kModeDispatch = 2        // ids, weights, per-tile histogram for the dispatch index
};

struct RouterParams {
  int32_t T, d, E, N, k;
  int32_t gate, n_group, topk_group, renorm;
  float route_scale;
  int32_t num_kb;                    // ceil(d / 64)
  int32_t stages;
  int32_t tmem_cols;                 // power of two >= max(32, N)
  int32_t mode;
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
};

__device__ __forceinline__ float fb_sigmoid(float z) {
  return __fdividef(1.0f, 1.0f + __expf(-z));
}

struct RouterShared {
  uint64_t full_bar[kMaxStages];
  uint64_t empty_bar[kMaxStages];
  uint64_t accum_bar;
  uint32_t tmem_base;
  int32_t abort_flag;
  int32_t is_last;
  float logit_bias[FB_MAX_EXPERTS];
  float select_bias[FB_MAX_EXPERTS];
  uint32_t hist[FB_MAX_EXPERTS];
  PlanShared plan;
};

// Load columns [c0, c0 + 32) (or 16 when fewer remain) of this warp's 32 rows.
__device__ __forceinline__ void load_chunk(uint32_t taddr, int c0, int N, uint32_t (&r)[32]) {
  if (N - c0 >= 32) tmem_ld_32x32b_x32(taddr + c0, r);
  else tmem_ld_32x32b_x16(taddr + c0, r);
  tmem_ld_wait();
}

__global__ void __launch_bounds__(kRouterThreads, 1)
fb_router_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ RouterParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ RouterShared sh;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int tile = blockIdx.x;
  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.N) * kBlockK * 2;
  const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle atoms need 1024-byte alignment
  volatile int* abort_flag = &sh.abort_flag;

  if (threadIdx.x == 0) {
    sh.abort_flag = 0;
    sh.is_last = 0;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&sh.full_bar[s]), 1);
      mbar_init(smem_u32(&sh.empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&sh.accum_bar), 1);
    fence_mbar_init();
    prefetch_tensormap(&tmap_x);
    prefetch_tensormap(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc<1>(smem_u32(&sh.tmem_base), static_cast<uint32_t>(p.tmem_cols));
    tmem_relinquish<1>();
  }
  if (warp >= 2) {
    const int et = threadIdx.x - 64;
    for (int e = et; e < FB_MAX_EXPERTS; e += kEpilogueThreads) {
      sh.hist[e] = 0;
      sh.logit_bias[e] = (p.logit_bias != nullptr && e < p.E) ? p.logit_bias[e] : 0.0f;
      sh.select_bias[e] = (p.select_bias != nullptr && e < p.E) ? p.select_bias[e] : 0.0f;
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = sh.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_x = l2_policy_evict_first();   // x is streamed once
      const uint64_t pol_w = l2_policy_evict_last();    // W is re-read by every block
      for (int kb = 0; kb < p.num_kb; ++kb) {
        const int s = kb % p.stages;
        const uint32_t phase = static_cast<uint32_t>(kb / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&sh.empty_bar[s]), phase ^ 1u, abort_flag)) break;
        const uint32_t full = smem_u32(&sh.full_bar[s]);
        mbar_arrive_expect_tx(full, stage_bytes);
        const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
        tma_load_2d(a_dst, &tmap_x, full, kb * kBlockK, tile * kTileM, pol_x);
        tma_load_2d(a_dst + kATileBytes, &tmap_w, full, kb * kBlockK, 0, pol_w);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16_f32(kTileM, static_cast<uint32_t>(p.N));
      bool ok = true;
      for (int kb = 0; kb < p.num_kb && ok; ++kb) {
        const int s = kb % p.stages;
        const uint32_t phase = static_cast<uint32_t>(kb / p.stages) & 1u;
        ok = mbar_wait(smem_u32(&sh.full_bar[s]), phase, abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_addr = smem_base + static_cast<uint32_t>(s) * stage_bytes;
        const uint64_t adesc = umma_smem_desc_sw128(a_addr);
        const uint64_t bdesc = umma_smem_desc_sw128(a_addr + kATileBytes);
#pragma unroll
        for (int kk = 0; kk < kBlockK / kUmmaK; ++kk) {
          // advance 16 elements = 32 bytes inside the swizzled row: +2 in the address field
          umma_bf16<1>(tmem_base, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
        }
        umma_commit_1cta(smem_u32(&sh.empty_bar[s]));     // frees the stage when these MMAs retire
      }
      umma_commit_1cta(smem_u32(&sh.accum_bar));          // accumulator complete
    }
  } else {
    // ------------------------------------------------------------ epilogue: one thread per row
    const int et = threadIdx.x - 64;                       // 0..127
    const int quarter = warp & 3;                          // TMEM lanes this warp may touch
    const int row_in_tile = quarter * 32 + lane;
    const long long row = static_cast<long long>(tile) * kTileM + row_in_tile;
    const bool valid = row < p.T;
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const int E = p.E, N = p.N, k = p.k;

    const bool got = mbar_wait(smem_u32(&sh.accum_bar), 0u, abort_flag);
    tcgen05_fence_after();
    TopK top;
    top.init();
    float sm_max = -INFINITY, sm_sum = 0.0f;               // online softmax (weights without renorm)
    if (got) {
      uint32_t r[32];
      if (p.gate == FB_GATE_SOFTMAX_TOPK) {
        for (int c0 = 0; c0 < N; c0 += 32) {
          load_chunk(taddr, c0, N, r);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int e = c0 + j;
            if (e < E) {
              const float z = __uint_as_float(r[j]) + sh.logit_bias[e];
              if (p.logits != nullptr && valid) p.logits[row * E + e] = z;
              if (z > sm_max) { sm_sum = sm_sum * __expf(sm_max - z) + 1.0f; sm_max = z; }
              else sm_sum += __expf(z - sm_max);
              top.insert(z, e);
            }
          }
        }
      } else {
        // pass 1: score every group by the sum of its two largest keys, keep the best groups
        const int gs = E / p.n_group;
        TopK gtop;                                           // FB_MAX_TOPK >= topk_group
        gtop.init();
        int pos = 0, g = 0;
        float m1 = -INFINITY, m2 = -INFINITY;
        for (int c0 = 0; c0 < N; c0 += 32) {
          load_chunk(taddr, c0, N, r);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int e = c0 + j;
            if (e < E) {
              const float z = __uint_as_float(r[j]) + sh.logit_bias[e];
              if (p.logits != nullptr && valid) p.logits[row * E + e] = z;
              const float q = fb_sigmoid(z) + sh.select_bias[e];
              if (q > m1) { m2 = m1; m1 = q; }
              else if (q > m2) m2 = q;
              if (++pos == gs) {
                gtop.insert(gs >= 2 ? m1 + m2 : m1, g);
                ++g; pos = 0; m1 = -INFINITY; m2 = -INFINITY;
              }
            }
          }
        }
        uint32_t keep = 0;
#pragma unroll
        for (int j = 0; j < FB_MAX_TOPK; ++j)
          if (j < p.topk_group) keep |= 1u << gtop.i[j];
        // pass 2: top-k among the experts of the kept groups
        pos = 0; g = 0;
        for (int c0 = 0; c0 < N; c0 += 32) {
          load_chunk(taddr, c0, N, r);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int e = c0 + j;
            if (e < E) {
              if ((keep >> g) & 1u) {
                const float z = __uint_as_float(r[j]) + sh.logit_bias[e];
                top.insert(fb_sigmoid(z) + sh.select_bias[e], e);
              }
              if (++pos == gs) { ++g; pos = 0; }
            }
          }
        }
      }
    }
    tcgen05_fence_before();

    // ---- outputs per row
    if (got && valid) {
      if (p.topk_ids != nullptr) {
#pragma unroll
        for (int j = 0; j < FB_MAX_TOPK; ++j)
          if (j < k) p.topk_ids[row * k + j] = top.i[j];
      }
      if (p.topk_w != nullptr) {
        float w[FB_MAX_TOPK];
        float wsum = 0.0f;
#pragma unroll
        for (int j = 0; j < FB_MAX_TOPK; ++j) {
          if (p.gate == FB_GATE_SOFTMAX_TOPK) w[j] = (j < k) ? __expf(top.v[j] - sm_max) : 0.0f;
          else w[j] = (j < k) ? top.v[j] - sh.select_bias[top.i[j]] : 0.0f;   // unbiased sigmoid score
          wsum += w[j];
        }
        float scale;
        if (p.gate == FB_GATE_SOFTMAX_TOPK) scale = p.renorm ? 1.0f / wsum : 1.0f / sm_sum;
        else scale = p.renorm ? p.route_scale / wsum : p.route_scale;
#pragma unroll
        for (int j = 0; j < FB_MAX_TOPK; ++j)
          if (j < k) p.topk_w[row * k + j] = w[j] * scale;
      }
    }
    // ---- histogram: one shared-memory atomic per distinct expert per warp (Eq. 5)
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) {
      if (j < k) {
        const int e = (got && valid) ? top.i[j] : -1;
        const uint32_t same = __match_any_sync(0xffffffffu, e);
        if (e >= 0 && lane == __ffs(same) - 1) atomicAdd(&sh.hist[e], __popc(same));
      }
    }
    named_bar_sync(kPlanBarrierId, kEpilogueThreads);
    if (p.mode == kModeDispatch) {
      for (int e = et; e < E; e += kEpilogueThreads)
        p.tile_counts[static_cast<size_t>(tile) * E + e] = sh.hist[e];
    } else {
      for (int e = et; e < E; e += kEpilogueThreads) {
        const uint32_t c = sh.hist[e];
        if (c) atomicAdd(&p.counts_scratch[e], c);
      }
      __threadfence();
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      if (et == 0) {
        const uint32_t prev = atomicAdd(p.ticket, 1u);
        sh.is_last = (prev == gridDim.x - 1) ? 1 : 0;
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      if (sh.is_last) {
        // Every other block has published its counts: this one finishes the call.
        __threadfence();
        for (int e = et; e < E; e += kEpilogueThreads) {
          const uint32_t c = __ldcg(&p.counts_scratch[e]);
          p.counts_out[e] = c;
          sh.plan.cnt[e] = c;
          p.counts_scratch[e] = 0;           // ready for the next call
        }
        if (et == 0) *p.ticket = 0;
        if (sh.abort_flag) { if (et == 0) atomicCAS(p.status, 0, FB_ERR_TIMEOUT); }
        named_bar_sync(kPlanBarrierId, kEpilogueThreads);
        if (p.mode == kModePredictPlan) plan_swaps_block(p.plan, sh.plan, et, p.status);
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncthreads();
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(p.status, 0, FB_ERR_TIMEOUT);
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc<1>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
}

// Stand-alone planner: one block of kPlanThreads threads.
__global__ void __launch_bounds__(kPlanThreads, 1)
fb_plan_kernel(const __grid_constant__ PlanParams p, const uint32_t* __restrict__ counts, int32_t* status) {
  __shared__ PlanShared sh;
  const int t = threadIdx.x;
  for (int e = t; e < p.E; e += kPlanThreads) sh.cnt[e] = counts[e];
  named_bar_sync(kPlanBarrierId, kPlanThreads);
  plan_swaps_block(p, sh, t, status);
}

}  // namespace fb
