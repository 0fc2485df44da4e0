// Dispatch index under the committed placement (stage 4 of the method): a stable
// counting sort of the T*k (token, expert) assignments by physical slot.  Positions
// come from prefix sums and population counts only - no atomic decides an output
// position - so the result is unique and reproducible.
//
// Input: the router kernel's top-k ids and its per-tile expert histogram
// tile_counts[tile][e] (tile = 128 consecutive tokens).  One block per tile.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/freebalance.h"

namespace fb {

constexpr int kDispatchThreads = 256;
constexpr int kDispatchTile = 128;     // must equal the router kernel's tile height

struct DispatchParams {
  int32_t T, k, E, R, num_tiles;
  const int32_t* topk_ids;         // [T][k]
  const uint32_t* tile_counts;     // [num_tiles][E]
  const int32_t* expert_to_slot;   // [E]
  uint32_t* slot_offsets;          // [E+1]
  uint32_t* rank_offsets;          // [R+1]
  int32_t* perm;                   // [T*k]
  int32_t* inv_perm;               // [T*k]
  uint32_t* rank_load;             // [R]
  int32_t* status;
};

__global__ void __launch_bounds__(kDispatchThreads)
fb_dispatch_kernel(const __grid_constant__ DispatchParams p) {
  __shared__ int32_t slot_of[FB_MAX_EXPERTS];
  __shared__ int32_t owner[FB_MAX_EXPERTS];
  __shared__ uint32_t before[FB_MAX_EXPERTS];      // assignments to this slot in earlier tiles
  __shared__ uint32_t total[FB_MAX_EXPERTS];       // assignments to this slot in all tiles
  __shared__ uint32_t offs[FB_MAX_EXPERTS + 1];    // exclusive prefix of total over slots
  __shared__ uint32_t mask[FB_MAX_EXPERTS][kDispatchTile / 32];
  __shared__ uint32_t warp_sum[kDispatchThreads / 32];
  __shared__ int32_t bad;

  const int t = threadIdx.x;
  const int tile = blockIdx.x;
  const int E = p.E, k = p.k;
  if (t == 0) bad = 0;
  for (int s = t; s < FB_MAX_EXPERTS; s += kDispatchThreads) {
    owner[s] = -1; before[s] = 0; total[s] = 0;
#pragma unroll
    for (int w = 0; w < kDispatchTile / 32; ++w) mask[s][w] = 0;
  }
  __syncthreads();
  for (int e = t; e < E; e += kDispatchThreads) {
    int s = p.expert_to_slot[e];
    if (s < 0 || s >= E) { bad = 1; s = 0; }
    else if (atomicExch(&owner[s], e) != -1) bad = 1;
    slot_of[e] = s;
  }
  __syncthreads();
  if (bad) {                                    // not a bijection: report, write nothing
    if (t == 0 && tile == 0) atomicCAS(p.status, 0, FB_ERR_BAD_PLACEMENT);
    return;
  }
  // column sums of the per-tile histogram, split at this tile
  for (int e = t; e < E; e += kDispatchThreads) {
    uint32_t bef = 0, tot = 0;
    const uint32_t* col = p.tile_counts + e;
#pragma unroll 8
    for (int tt = 0; tt < p.num_tiles; ++tt) {
      const uint32_t c = col[static_cast<size_t>(tt) * E];
      tot += c;
      if (tt < tile) bef += c;
    }
    before[slot_of[e]] = bef;
    total[slot_of[e]] = tot;
  }
  __syncthreads();
  // exclusive scan of total[] over slots (thread s owns slot s)
  {
    const uint32_t v = (t < E) ? total[t] : 0;
    uint32_t incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t o = __shfl_up_sync(0xffffffffu, incl, off);
      if ((t & 31) >= off) incl += o;
    }
    if ((t & 31) == 31) warp_sum[t >> 5] = incl;
    __syncthreads();
    uint32_t base = 0;
    for (int w = 0; w < (t >> 5); ++w) base += warp_sum[w];
    if (t < E) offs[t] = base + incl - v;
    if (t == E - 1) offs[E] = base + incl;
  }
  __syncthreads();
  if (tile == 0) {
    const int m = E / p.R;
    for (int s = t; s <= E; s += kDispatchThreads) p.slot_offsets[s] = offs[s];
    for (int r = t; r <= p.R; r += kDispatchThreads) p.rank_offsets[r] = offs[r * m];
    for (int r = t; r < p.R; r += kDispatchThreads) p.rank_load[r] = offs[(r + 1) * m] - offs[r * m];
  }
  // rank of each assignment among the rows of this tile that go to the same slot
  const long long i = static_cast<long long>(tile) * kDispatchTile + t;
  const bool active = t < kDispatchTile && i < p.T;
  int32_t my_slot[FB_MAX_TOPK];
#pragma unroll
  for (int j = 0; j < FB_MAX_TOPK; ++j) my_slot[j] = 0;
  if (active) {
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) {
      if (j < k) {
        int e = p.topk_ids[i * k + j];
        e = (e < 0 || e >= E) ? 0 : e;
        my_slot[j] = slot_of[e];
        atomicOr(&mask[my_slot[j]][t >> 5], 1u << (t & 31));
      }
    }
  }
  __syncthreads();
  if (active) {
    const long long n_assign = static_cast<long long>(p.T) * k;
#pragma unroll
    for (int j = 0; j < FB_MAX_TOPK; ++j) {
      if (j < k) {
        const int s = my_slot[j];
        uint32_t ahead = __popc(mask[s][t >> 5] & ((1u << (t & 31)) - 1u));
        for (int w = 0; w < (t >> 5); ++w) ahead += __popc(mask[s][w]);
        const long long pos = static_cast<long long>(offs[s]) + before[s] + ahead;
        const long long flat = i * k + j;
        if (pos < n_assign) {
          p.perm[pos] = static_cast<int32_t>(flat);
          p.inv_perm[flat] = static_cast<int32_t>(pos);
        }
      }
    }
  }
}

}  // namespace fb
