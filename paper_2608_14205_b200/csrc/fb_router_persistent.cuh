// Persistent variant of the fused router kernel (Eqs. 2-5) for calls with more 128-row
// tiles than the GPU has SM pairs: every cluster of two blocks walks a strided list of
// tile pairs, and the epilogue of one tile runs while the tensor cores already work on the
// next one.
//
// What makes the overlap possible
//   * the epilogue warps copy their share of the finished accumulators from tensor memory
//     into registers (64 columns per thread), hand tensor memory back to the MMA issuers
//     at once, and do all gating / selection work from registers;
//   * the epilogue's shared-memory scratch (group scores, candidate lists) has its own
//     44 KB behind the pipeline stages instead of reusing them.
// Restricted to the gates the ranking selection handles (DeepSeek-V3-like sigmoid gates with
// 32-expert groups, softmax gates over whole 32-column chunks); everything else, and
// every call that fits one tile per block, runs fb_router_kernel.  Arithmetic, summation
// order (even k-blocks in accumulator 0, odd ones in accumulator 1) and tie-breaking are
// those of fb_router_kernel, so both kernels give identical results.
//
// Warp roles as in fb_router_kernel: warp 0 TMA producer, warps 1 and 18 MMA issuers (even
// block of the pair only), warps 2..17 epilogue (4 row quarters x 4 column shares).
#pragma once
#include "fb_router.cuh"

namespace fb {

constexpr int kPersistGroups = 8;            // 32-column chunks (= groups) per row, at most
constexpr size_t kPersistScratchBytes =
    (3 * kPersistGroups * kTileM + 2 * kCandCap * kTileM) * sizeof(float);   // 44 KB
static_assert(2 * kCandCap >= 2 * (kEpiSubs - 1) * FB_MAX_TOPK, "merge lists must fit in the candidate area");
static_assert(2 * kPersistGroups >= 2 * FB_MAX_TOPK, "result lists must fit in the group-score area");
static_assert(kPersistGroups == kBoundRows, "the three tables of best keys lie one after the other");

struct PersistShared {
  uint64_t full_bar[kMaxStages];
  uint64_t empty_bar[kMaxStages];
  // Accumulator sets: one (2 N of the 512 tensor-memory columns each) or, when 4 N <= 512, two that
  // alternate from tile to tile, so that the next tile's MMAs need not wait for the drain.
  uint64_t accum_bar[2];                     // per set: both issuers' commits, once per use
  uint64_t tmem_empty_bar[2];                // per set, even block's copy: all epilogue warps of the pair, once per use
  uint32_t tmem_base;
  int32_t abort_flag;
  int32_t is_last;
  int32_t accum_ok;
  int32_t any_overflow;
  int32_t issuer_progress[2];                // rings with an odd number of stages: see issuer_turn_wait
  float logit_bias[FB_MAX_EXPERTS];
  alignas(16) float select_bias[FB_MAX_EXPERTS];
  uint32_t hist[FB_MAX_EXPERTS];
  uint32_t cand_count[kTileM];
  PlanShared plan;
};

// Host-side test of the gate shapes this kernel supports (same rule as the ranking
// selection of fb_router_kernel, without the cases that need the softmax denominator).
__host__ __device__ inline bool persistent_gate_ok(int E, int k, int gate, int n_group, int topk_group,
                                                   bool want_sum) {
  if (E % 32 != 0 || E / 32 > kPersistGroups) return false;
  if (gate != FB_GATE_SOFTMAX_TOPK)
    return E / n_group == 32 && topk_group <= kEpiSubs && topk_group * 2 >= k;
  return (E / 32) * 2 >= k && !want_sum;
}

__device__ __forceinline__ void ring_advance(int& s, uint32_t& phase, int stages) {
  if (++s == stages) { s = 0; phase ^= 1u; }
}

// kSigmoid: sigmoid + bias group-limited gate (true) or softmax gate (false); kLogitBias: a logit
// bias is given.  One instance per combination keeps code and registers to what it needs.
template <bool kSigmoid, bool kLogitBias>
__global__ void __launch_bounds__(kRouterThreads, 1)
fb_router_persistent_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_x2,
                            const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ RouterParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ PersistShared sh;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = cluster_ctarank();
  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.N / 2) * kBlockK * 2;
  const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  volatile int* abort_flag = &sh.abort_flag;

  // Tile pairs of this cluster: pair_first, pair_first + pair_stride, ...  In kModeLayer the
  // first pairs_per_pass pairs belong to the early pass, the rest to the normal pass.
  const int pairs_per_pass = p.tiles_first / 2;
  const int total_pairs = p.mode == kModeLayer ? 2 * pairs_per_pass : pairs_per_pass;
  const int pair_first = static_cast<int>(blockIdx.x) / 2;
  const int pair_stride = static_cast<int>(gridDim.x) / 2;

  if (threadIdx.x == 0) {
    sh.abort_flag = 0;
    sh.is_last = 0;
    sh.any_overflow = 0;
    sh.issuer_progress[0] = -1;
    sh.issuer_progress[1] = -1;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&sh.full_bar[s]), 1);
      mbar_init(smem_u32(&sh.empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh.accum_bar[a]), 2);
      mbar_init(smem_u32(&sh.tmem_empty_bar[a]), 2 * (kEpilogueThreads / 32));
    }
    fence_mbar_init();
    prefetch_tensormap(&tmap_x);
    if (p.mode == kModeLayer) prefetch_tensormap(&tmap_x2);
    prefetch_tensormap(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc<2>(smem_u32(&sh.tmem_base), static_cast<uint32_t>(p.tmem_cols));
    tmem_relinquish<2>();
  }
  if (warp >= 2) {
    const int et = threadIdx.x - 64;
    for (int e = et; e < FB_MAX_EXPERTS; e += kEpilogueThreads) {
      sh.hist[e] = 0;
      if (e < kTileM) sh.cand_count[e] = 0;
    }
    if (p.mode == kModePredictPlan || p.mode == kModeLayer) plan_clear(sh.plan, et, kEpilogueThreads);
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_arrive(); cluster_wait();          // the partner's barriers and tensor memory are ready too
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

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_x = l2_policy_evict_first();
      const uint64_t pol_w = l2_policy_evict_last();
      int s = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int pt = pair_first; pt < total_pairs && ok; pt += pair_stride) {
        const bool second_pass = pt >= pairs_per_pass;
        const int tile = 2 * (second_pass ? pt - pairs_per_pass : pt) + static_cast<int>(cta_rank);
        const CUtensorMap* xmap = second_pass ? &tmap_x2 : &tmap_x;
        for (int kb = 0; kb < p.num_kb; ++kb) {
          ok = mbar_wait<true>(smem_u32(&sh.empty_bar[s]), phase ^ 1u, abort_flag);
          if (!ok) break;
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
          // both blocks report their bytes to the even block's barrier
          const uint32_t full = map_to_cta(smem_u32(&sh.full_bar[s]), 0u);
          if (cta_rank == 0) mbar_arrive_expect_tx(smem_u32(&sh.full_bar[s]), 2u * stage_bytes);
          tma_load_2d_pair(a_dst, xmap, full, kb * kBlockK, tile * kTileM, pol_x);
          tma_load_2d_pair(a_dst + kATileBytes, &tmap_w, full, kb * kBlockK,
                           static_cast<int32_t>(cta_rank) * (p.N / 2), pol_w);
          ring_advance(s, phase, p.stages);
        }
      }
    }
  } else if (warp == 1 || warp == kSecondIssuerWarp) {
    // ------------------------------------------------------------ MMA issuers (even block only)
    if (lane == 0 && cta_rank == 0) {
      const int first_kb = warp == 1 ? 0 : 1;
      const uint32_t acc_sets = 4 * p.N <= p.tmem_cols ? 2u : 1u;
      const uint32_t idesc = umma_idesc_bf16_f32(kTileM * 2, static_cast<uint32_t>(p.N));
      int s = 0;
      uint32_t phase = 0;
      uint32_t ti = 0;                        // this block pair's tile counter
      bool ok = true;
      int32_t g = 0;                          // ring position: k-blocks of all of this pair's tiles, in order
      const bool odd_ring = (p.stages & 1) != 0;
      volatile int32_t* my_progress = &sh.issuer_progress[warp == 1 ? 0 : 1];
      const volatile int32_t* other_progress = &sh.issuer_progress[warp == 1 ? 1 : 0];
      for (int pt = pair_first; pt < total_pairs && ok; pt += pair_stride, ++ti) {
        const uint32_t set = ti % acc_sets, use = ti / acc_sets;
        const uint32_t acc = tmem_base + set * 2u * static_cast<uint32_t>(p.N) + (warp == 1 ? 0u : static_cast<uint32_t>(p.N));
        if (use != 0) {
          // the set's previous contents must have been read out by both blocks
          ok = mbar_wait<true>(smem_u32(&sh.tmem_empty_bar[set]), (use - 1u) & 1u, abort_flag);
          if (!ok) break;
          tcgen05_fence_after();
        }
        for (int kb = 0; kb < p.num_kb; ++kb, ++g) {
          if ((kb & 1) == first_kb) {
            if (odd_ring && g >= p.stages) {
              // whose was the stage's previous use (ring position g - stages)?  Its k-block index
              // inside its own tile decides, as for every k-block.
              int kbp = kb - p.stages;
              while (kbp < 0) kbp += p.num_kb;
              if ((kbp & 1) != first_kb) ok = issuer_turn_wait(other_progress, g - p.stages, abort_flag);
            }
            ok = ok && mbar_wait<true>(smem_u32(&sh.full_bar[s]), phase, abort_flag);
            if (!ok) break;
            if (odd_ring) *my_progress = g;
            tcgen05_fence_after();
            const uint32_t a_addr = smem_base + static_cast<uint32_t>(s) * stage_bytes;
            const uint64_t adesc = umma_smem_desc_sw128(a_addr);
            const uint64_t bdesc = umma_smem_desc_sw128(a_addr + kATileBytes);
#pragma unroll
            for (int kk = 0; kk < kBlockK / kUmmaK; ++kk)
              umma_bf16<2>(acc, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb != first_kb || kk != 0) ? 1u : 0u);
            umma_commit_pair(smem_u32(&sh.empty_bar[s]), cta_rank);   // frees the stage in both blocks
          }
          ring_advance(s, phase, p.stages);
        }
        if (ok) umma_commit_pair(smem_u32(&sh.accum_bar[set]), cta_rank);   // this issuer's accumulator is complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int et = threadIdx.x - 64;                       // 0 .. kEpilogueThreads-1
    const int quarter = warp & 3;                          // TMEM lanes this warp may touch
    const int sub = (warp - 2) >> 2;                       // owns chunks sub and sub + 4
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t taddr0 = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const uint32_t acc_sets = 4 * p.N <= p.tmem_cols ? 2u : 1u;
    const int E = p.E, N = p.N, k = p.k;
    constexpr bool sigmoid_gate = kSigmoid;
    const int n_chunks = E >> 5;                           // E is a multiple of 32 here
    constexpr bool has_lb = kLogitBias;
    const bool two_acc = p.num_kb > 1;
    // scratch behind the pipeline stages
    float* gscore_s = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)) +
                                               static_cast<size_t>(p.stages) * stage_bytes);   // [8][128]
    float* glow_s = gscore_s + kPersistGroups * kTileM;                                         // [8][128]
    float* third_s = glow_s + kPersistGroups * kTileM;                                          // [8][128]
    // candidates [32][128]: ordered key bits in the high word, ~expert id in the low word
    unsigned long long* cand = reinterpret_cast<unsigned long long*>(third_s + kPersistGroups * kTileM);
    uint32_t* out_hi = reinterpret_cast<uint32_t*>(gscore_s);   // [8][128]: group scores are dead by then
    uint32_t* out_lo = reinterpret_cast<uint32_t*>(glow_s);
    float* merge_v = reinterpret_cast<float*>(cand);            // [3][8][128]: candidates are dead by then
    int32_t* merge_i = reinterpret_cast<int32_t*>(merge_v + (kEpiSubs - 1) * FB_MAX_TOPK * kTileM);

    // biases (read by these warps only, after the first barrier below)
    for (int e = et; e < FB_MAX_EXPERTS; e += kEpilogueThreads) {
      sh.logit_bias[e] = (p.logit_bias != nullptr && e < p.E) ? p.logit_bias[e] : 0.0f;
      sh.select_bias[e] = (p.select_bias != nullptr && e < p.E) ? p.select_bias[e] : 0.0f;
    }
    // any block may turn out to take the last ticket of the early pass
    if (p.mode == kModePredictPlan || p.mode == kModeLayer) plan_load_placement(p.plan, sh.plan, et, kEpilogueThreads);
    uint32_t tiles_done = 0;
    for (int pt = pair_first; pt < total_pairs; pt += pair_stride) {
      const bool second_pass = pt >= pairs_per_pass;
      const int mode = p.mode == kModeLayer ? (second_pass ? kModeDispatch : kModePredictPlan) : p.mode;
      const int tile = 2 * (second_pass ? pt - pairs_per_pass : pt) + static_cast<int>(cta_rank);
      const long long row = static_cast<long long>(tile) * kTileM + row_in_tile;
      const bool valid = row < p.T;
      int32_t* const out_ids = (p.mode == kModeLayer && !second_pass) ? nullptr : p.topk_ids;
      float* const out_w = (p.mode == kModeLayer && !second_pass) ? nullptr : p.topk_w;

      // one thread polls for the finished accumulators, the others sleep at the barrier
      const uint32_t set = tiles_done % acc_sets, use = tiles_done / acc_sets;
      const uint32_t taddr = taddr0 + set * 2u * static_cast<uint32_t>(N);
      if (et == 0) sh.accum_ok = mbar_wait<true>(smem_u32(&sh.accum_bar[set]), use & 1u, abort_flag) ? 1 : 0;
      named_bar_sync(kAccumBarrierId, kEpilogueThreads);
      if (sh.accum_ok == 0) break;
      ++tiles_done;
      tcgen05_fence_after();

      // ---------------- tensor memory -> registers: this thread's row, chunks sub and sub + 4
      float key[2][32];
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const int c = sub + kEpiSubs * ci;
        if (c < n_chunks) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(taddr + c * 32, r);
          tmem_ld_wait();
          if (two_acc) {                                     // add the odd k-blocks' accumulator
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint32_t r2[32];
              tmem_ld_32x32b_x16(taddr + N + c * 32 + 16 * h, r2);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 16; ++j)
                r[16 * h + j] = __float_as_uint(__uint_as_float(r[16 * h + j]) + __uint_as_float(r2[j]));
            }
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) key[ci][j] = __uint_as_float(r[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) key[ci][j] = -INFINITY;
        }
      }
      // the issuers may overwrite the accumulators now
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(smem_u32(&sh.tmem_empty_bar[set]), 0u);

      // ---------------- selection keys in place; best two keys of every chunk
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const int c = sub + kEpiSubs * ci;
        if (c < n_chunks) {
          const int c0 = c * 32;
          if (sigmoid_gate && !has_lb) {
            const float4* sb4 = reinterpret_cast<const float4*>(&sh.select_bias[c0]);
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const float4 b = sb4[j4];
              key[ci][4 * j4 + 0] = fb_sigmoid(key[ci][4 * j4 + 0]) + b.x;
              key[ci][4 * j4 + 1] = fb_sigmoid(key[ci][4 * j4 + 1]) + b.y;
              key[ci][4 * j4 + 2] = fb_sigmoid(key[ci][4 * j4 + 2]) + b.z;
              key[ci][4 * j4 + 3] = fb_sigmoid(key[ci][4 * j4 + 3]) + b.w;
            }
          } else if (sigmoid_gate) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              key[ci][j] = fb_sigmoid(key[ci][j] + sh.logit_bias[c0 + j]) + sh.select_bias[c0 + j];
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) key[ci][j] = key[ci][j] + (has_lb ? sh.logit_bias[c0 + j] : 0.0f);
          }
          // four interleaved running (best, second, third) triples; the third only feeds the
          // softmax gate's bound
          float m1[4], m2[4], m3[4];
#pragma unroll
          for (int a = 0; a < 4; ++a) { m1[a] = -INFINITY; m2[a] = -INFINITY; m3[a] = -INFINITY; }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float t = fminf(m1[j & 3], key[ci][j]);
            if (!sigmoid_gate) m3[j & 3] = fmaxf(m3[j & 3], fminf(m2[j & 3], t));
            m2[j & 3] = fmaxf(m2[j & 3], t);
            m1[j & 3] = fmaxf(m1[j & 3], key[ci][j]);
          }
#pragma unroll
          for (int a = 2; a >= 1; a >>= 1) {
#pragma unroll
            for (int b = 0; b < a; ++b) {
              // best three of two sorted triples
              const float lo1 = fminf(m1[b], m1[b + a]), hi2 = fmaxf(m2[b], m2[b + a]);
              if (!sigmoid_gate) m3[b] = fmaxf(fminf(lo1, hi2), fmaxf(m3[b], m3[b + a]));
              m2[b] = fmaxf(lo1, hi2);
              m1[b] = fmaxf(m1[b], m1[b + a]);
            }
          }
          glow_s[c * kTileM + row_in_tile] = m2[0];
          if (sigmoid_gate) {
            gscore_s[c * kTileM + row_in_tile] = m1[0] + m2[0];   // group score (gs == 32)
          } else {
            gscore_s[c * kTileM + row_in_tile] = m1[0];
            third_s[c * kTileM + row_in_tile] = m3[0];
          }
        }
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);

      // ---------------- choose the groups; lower bound for the k-th key
      uint32_t kept = 0;
      float floor_key = INFINITY;
      if (sigmoid_gate) {
        float sc[kPersistGroups];
#pragma unroll
        for (int g = 0; g < kPersistGroups; ++g) sc[g] = g < n_chunks ? gscore_s[g * kTileM + row_in_tile] : -INFINITY;
#pragma unroll
        for (int g = 0; g < kPersistGroups; ++g) {
          int rank = 0;
#pragma unroll
          for (int h = 0; h < kPersistGroups; ++h)   // a lower-numbered group wins ties
            if (h != g) rank += (h < g ? sc[h] >= sc[g] : sc[h] > sc[g]) ? 1 : 0;
          if (g < n_chunks && rank < p.topk_group) {
            kept |= 1u << g;
            floor_key = fminf(floor_key, glow_s[g * kTileM + row_in_tile]);
          }
        }
      } else {
        // the k-th largest of the chunks' three best keys (3 n_chunks >= k of them)
        floor_key = kth_largest_known(gscore_s, n_chunks, k, row_in_tile);
        kept = (1u << n_chunks) - 1u;
      }
      // ---------------- collect the keys >= floor of this thread's kept chunks (the bound is one of
      // k known keys of the row, so at least k keys qualify)
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const int c = sub + kEpiSubs * ci;
        if (c < n_chunks && ((kept >> c) & 1u)) {
          uint32_t mine = 0;
#pragma unroll
          for (int j = 0; j < 32; ++j) mine += key[ci][j] >= floor_key ? 1u : 0u;
          const uint32_t first = atomicAdd(&sh.cand_count[row_in_tile], mine);
          // predicated stores, no branches: slot address advances past every hit, a hit is stored
          // while the slot is inside the list
          const uint32_t list = smem_u32(cand) + static_cast<uint32_t>(row_in_tile) * 8u;
          const uint32_t list_end = list + kCandCap * kTileM * 8u;
          uint32_t slot = list + first * (kTileM * 8u);
          const uint32_t id0 = ~static_cast<uint32_t>(c * 32);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t hit = key[ci][j] >= floor_key ? 1u : 0u;
            st_shared_v2_if(hit & (slot < list_end ? 1u : 0u), slot, id0 - j, ordered_bits(key[ci][j]));
            slot += hit * (kTileM * 8u);
          }
        }
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);

      // ---------------- rank the candidates (many equal keys can overflow the list: handled below)
      const bool overflow = rank_candidates(cand, sh.cand_count[row_in_tile], sub, row_in_tile, out_hi, out_lo);
      if (overflow) sh.any_overflow = 1;
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      TopK top;
      top.init();
      if (sub == 0) {
        sh.cand_count[row_in_tile] = 0;                      // ready for the next tile
        if (!overflow) read_ranked(top, k, out_hi, out_lo, row_in_tile);
      }
      if (sh.any_overflow != 0) {
        // Some row of the tile had more than kCandCap keys at or above its floor (many equal
        // keys).  Such rows are selected by plain insertion: every thread scans its own kept
        // chunks in ascending expert order, then the row's first thread merges the lists.
        if (overflow) {
#pragma unroll
          for (int ci = 0; ci < 2; ++ci) {
            const int c = sub + kEpiSubs * ci;
            if (c < n_chunks && ((kept >> c) & 1u)) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (key[ci][j] > top.v[FB_MAX_TOPK - 1]) top.insert(key[ci][j], c * 32 + j);
            }
          }
          if (sub != 0) {
#pragma unroll
            for (int j = 0; j < FB_MAX_TOPK; ++j) {
              merge_v[((sub - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile] = top.v[j];
              merge_i[((sub - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile] = top.i[j];
            }
          }
        }
        named_bar_sync(kPlanBarrierId, kEpilogueThreads);
        if (overflow && sub == 0) {
#pragma unroll 1
          for (int s2 = 1; s2 < kEpiSubs; ++s2) {
#pragma unroll 1
            for (int j = 0; j < FB_MAX_TOPK; ++j) {
              const float x = merge_v[((s2 - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile];
              if (x > -INFINITY) top.insert_any_order(x, merge_i[((s2 - 1) * FB_MAX_TOPK + j) * kTileM + row_in_tile]);
            }
          }
        }
      }

      // ---------------- outputs per row
      const bool writer = valid && sub == 0;
      if (writer) {
        // softmax gates reach this kernel only with renormalised weights: no denominator needed
        write_row_outputs(top, p, row, out_ids, out_w, sh.select_bias, 0.0f, 1.0f);
        // ---------------- histogram (Eq. 5)
#pragma unroll
        for (int j = 0; j < FB_MAX_TOPK; ++j)
          if (j < k) atomicAdd(&sh.hist[top.i[j]], 1u);
      }
      named_bar_sync(kPlanBarrierId, kEpilogueThreads);
      if (et == 0) sh.any_overflow = 0;                       // everyone has read it
      if (mode == kModeDispatch) {
        const bool owns = static_cast<long long>(tile) * kTileM < p.T;   // the padding block of an odd pair owns no tile
        for (int e = et; e < E; e += kEpilogueThreads) {
          if (owns) p.tile_counts[static_cast<size_t>(tile) * E + e] = sh.hist[e];
          sh.hist[e] = 0;
        }
      } else if (pt + pair_stride >= pairs_per_pass) {
        // The histogram keeps accumulating over this block's tiles of the pass and is published
        // once, after the last of them (one fence and one ticket per block, not per tile).
        publish_counts(sh, p, et, warp, lane, mode == kModePredictPlan && p.fuse_planner != 0);
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tcgen05_fence_before();
  __syncthreads();
  cluster_arrive(); cluster_wait();          // nobody leaves while the partner may still signal it
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(p.status, 0, FB_ERR_TIMEOUT);
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc<2>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
}

}  // namespace fb
