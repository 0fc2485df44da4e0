// Dispatch index under the committed placement (stage 4 of the method): a stable
// counting sort of the T*k (token, expert) assignments by physical slot.  Positions
// come from prefix sums and population counts only - no atomic decides an output
// position - so the result is unique and reproducible.
//
// Input: the router kernel's top-k ids and its per-tile expert histogram
// tile_counts[tile][e] (tile = 128 consecutive tokens).  One block per tile, or per run of
// consecutive tiles when there are more tiles than blocks fit on the GPU at once.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/freebalance.h"
#include "fb_ptx.cuh"

namespace fb {

constexpr int kDispatchThreads = 1024;   // 4 threads per expert column for the tile sums
constexpr int kDispatchTile = 128;     // must equal the router kernel's tile height
constexpr int kSuperTiles = 32;        // tiles per super-block of the two-level tile sums

struct DispatchParams {
  int32_t T, k, E, R, num_tiles;
  const int32_t* topk_ids;         // [T][k]
  const uint32_t* tile_counts;     // [num_tiles][E]
  const uint32_t* super_counts;    // [ceil(num_tiles / 32)][E] sums over 32 tiles, or nullptr (few tiles)
  const int32_t* expert_to_slot;   // [E]
  uint32_t* slot_offsets;          // [E+1]
  uint32_t* rank_offsets;          // [R+1]
  int32_t* perm;                   // [T*k]
  int32_t* inv_perm;               // [T*k]
  uint32_t* rank_load;             // [R]
  int32_t* status;
};

__global__ void __launch_bounds__(kDispatchThreads, 2)
fb_dispatch_kernel(const __grid_constant__ DispatchParams p) {
  __shared__ int32_t slot_of[FB_MAX_EXPERTS];
  __shared__ int32_t owner[FB_MAX_EXPERTS];
  __shared__ uint32_t before[2][FB_MAX_EXPERTS];   // assignments to this slot in earlier tiles (two buffers: see the tile loop)
  __shared__ uint32_t total[FB_MAX_EXPERTS];       // assignments to this slot in all tiles
  __shared__ uint32_t part_before[kDispatchThreads / FB_MAX_EXPERTS][FB_MAX_EXPERTS];
  __shared__ uint32_t part_total[kDispatchThreads / FB_MAX_EXPERTS][FB_MAX_EXPERTS];
  __shared__ uint32_t offs[FB_MAX_EXPERTS + 1];    // exclusive prefix of total over slots
  __shared__ uint32_t mask[3][FB_MAX_EXPERTS][kDispatchTile / 32];
  __shared__ uint32_t warp_sum[FB_MAX_EXPERTS / 32];
  __shared__ int32_t bad;

  const int t = threadIdx.x;
  const int E = p.E, k = p.k;
  // This block's tiles: a contiguous range, so that "assignments in earlier tiles" can be carried
  // from one tile to the next instead of being summed again.
  const int per_block = (p.num_tiles + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int tile_begin = static_cast<int>(blockIdx.x) * per_block;
  const int tile_end = min(p.num_tiles, tile_begin + per_block);
  // The next router kernel of the stream may set itself up while this grid runs (it waits for
  // this grid's completion before it reads anything).
  pdl_launch_dependents();
  if (t == 0) bad = 0;
  for (int s = t; s < FB_MAX_EXPERTS; s += kDispatchThreads) {
    owner[s] = -1; before[0][s] = 0; before[1][s] = 0; total[s] = 0;
#pragma unroll
    for (int w = 0; w < kDispatchTile / 32; ++w) { mask[0][s][w] = 0; mask[1][s][w] = 0; mask[2][s][w] = 0; }
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
    if (t == 0 && blockIdx.x == 0) atomicCAS(p.status, 0, FB_ERR_BAD_PLACEMENT);
    return;
  }
  if (tile_begin >= tile_end) return;
  // Column sums of the per-tile histogram, split at this block's first tile.  The loop is bound
  // by L2 latency, so each column is shared by 4 threads and the loads are issued 32 at a time.
  {
    const int tile = tile_begin;
    constexpr int kParts = kDispatchThreads / FB_MAX_EXPERTS;
    const int e = t % FB_MAX_EXPERTS, part = t / FB_MAX_EXPERTS;
    uint32_t bef = 0, tot = 0;
    if (e < E && p.super_counts != nullptr) {
      // many tiles: whole super-blocks come pre-summed, only this tile's own super-block is walked
      const int n_super = (p.num_tiles + kSuperTiles - 1) / kSuperTiles;
      const int my_super = tile / kSuperTiles;
      for (int sb = part; sb < n_super; sb += kParts) {
        const uint32_t c = __ldg(p.super_counts + static_cast<size_t>(sb) * E + e);
        tot += c;
        if (sb < my_super) bef += c;
      }
      const uint32_t* col = p.tile_counts + e;
      for (int tt = my_super * kSuperTiles + part; tt < tile; tt += kParts)
        bef += __ldg(col + static_cast<size_t>(tt) * E);
    } else if (e < E) {
      const int per = (p.num_tiles + kParts - 1) / kParts;
      const int t0 = part * per, t1 = min(p.num_tiles, t0 + per);
      const uint32_t* col = p.tile_counts + e;
      for (int base = t0; base < t1; base += 32) {
        uint32_t c[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) c[u] = (base + u < t1) ? __ldg(col + static_cast<size_t>(base + u) * E) : 0u;
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          tot += c[u];
          if (base + u < tile) bef += c[u];
        }
      }
    }
    part_before[part][e] = bef;
    part_total[part][e] = tot;
    __syncthreads();
    if (part == 0 && e < E) {
      uint32_t b = 0, a = 0;
#pragma unroll
      for (int q = 0; q < kParts; ++q) { b += part_before[q][e]; a += part_total[q][e]; }
      before[0][slot_of[e]] = b;
      total[slot_of[e]] = a;
    }
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
    if (t < FB_MAX_EXPERTS && (t & 31) == 31) warp_sum[t >> 5] = incl;
    __syncthreads();
    if (t < FB_MAX_EXPERTS) {
      uint32_t base = 0;
      for (int w = 0; w < (t >> 5); ++w) base += warp_sum[w];
      if (t < E) offs[t] = base + incl - v;
      if (t == E - 1) offs[E] = base + incl;
    }
  }
  __syncthreads();
  if (blockIdx.x == 0) {
    const int m = E / p.R;
    for (int s = t; s <= E; s += kDispatchThreads) p.slot_offsets[s] = offs[s];
    for (int r = t; r <= p.R; r += kDispatchThreads) p.rank_offsets[r] = offs[r * m];
    for (int r = t; r < p.R; r += kDispatchThreads) p.rank_load[r] = offs[(r + 1) * m] - offs[r * m];
  }
  // Rank of each assignment among the rows of its tile that go to the same slot.
  // Thread (row, j) = (t % 128, t / 128) owns assignment j of the tile's row.
  static_assert(kDispatchThreads == kDispatchTile * FB_MAX_TOPK, "one thread per assignment of a tile");
  const int row = t % kDispatchTile, j = t / kDispatchTile;
  const long long n_assign = static_cast<long long>(p.T) * k;
  // Tile loop with one barrier per tile.  Tile n reads the earlier-tile counts from buffer n % 2
  // and writes the next tile's into the other one after its barrier (last read before that
  // barrier).  The row masks rotate through three buffers: tile n uses n % 3 and, after its
  // barrier, clears (n + 2) % 3, which tile n - 1 read before that barrier and tile n + 2 will
  // fill after the next one.  The next tile's expert id and this tile's histogram row are loaded
  // one iteration ahead.
  auto load_id = [&](int tile) -> int {
    const long long i = static_cast<long long>(tile) * kDispatchTile + row;
    if (tile >= tile_end || j >= k || i >= p.T) return -1;
    const int e = p.topk_ids[i * k + j];
#ifdef FB_DEBUG
    if (e < 0 || e >= E) atomicCAS(p.status, 0, FB_ERR_INTERNAL);       // an expert id outside [0, E)
#endif
    return (e < 0 || e >= E) ? 0 : e;
  };
  int e_cur = load_id(tile_begin);
  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int n = tile - tile_begin, par = n & 1, mb = n % 3, mb_clear = (n + 2) % 3;
    const int e_next = load_id(tile + 1);
    // this tile's histogram row, needed to step the earlier-tile counts to the next tile
    const uint32_t step = (t < E && tile + 1 < tile_end) ? __ldg(p.tile_counts + static_cast<size_t>(tile) * E + t) : 0u;
    const bool active = e_cur >= 0;
    const int my_slot = active ? slot_of[e_cur] : 0;
    if (active) atomicOr(&mask[mb][my_slot][row >> 5], 1u << (row & 31));
    __syncthreads();
    if (active) {
      uint32_t ahead = __popc(mask[mb][my_slot][row >> 5] & ((1u << (row & 31)) - 1u));
      for (int w = 0; w < (row >> 5); ++w) ahead += __popc(mask[mb][my_slot][w]);
      const long long pos = static_cast<long long>(offs[my_slot]) + before[par][my_slot] + ahead;
      const long long flat = (static_cast<long long>(tile) * kDispatchTile + row) * k + j;
#ifdef FB_DEBUG
      if (pos < 0 || pos >= n_assign || flat >= n_assign || my_slot < 0 || my_slot >= E)
        atomicCAS(p.status, 0, FB_ERR_INTERNAL);                          // a position outside [0, T k) or a slot outside [0, E)
#endif
      if (pos < n_assign) {
        p.perm[pos] = static_cast<int32_t>(flat);
        p.inv_perm[flat] = static_cast<int32_t>(pos);
      }
    }
    if (tile + 1 < tile_end) {
      if (t < E) before[par ^ 1][slot_of[t]] = before[par][slot_of[t]] + step;
      for (int s = t; s < FB_MAX_EXPERTS; s += kDispatchThreads) {
#pragma unroll
        for (int w = 0; w < kDispatchTile / 32; ++w) mask[mb_clear][s][w] = 0;
      }
    }
    e_cur = e_next;
  }
}

// Sums of the per-tile histograms over super-blocks of 32 tiles (only launched when there
// are many tiles, so that the dispatch kernel's blocks need not each walk all of them).
__global__ void __launch_bounds__(FB_MAX_EXPERTS)
fb_tile_sums_kernel(const uint32_t* __restrict__ tile_counts, uint32_t* __restrict__ super_counts,
                    int num_tiles, int E) {
  const int e = threadIdx.x, sb = blockIdx.x;
  if (e >= E) return;
  const int t0 = sb * kSuperTiles, t1 = min(num_tiles, t0 + kSuperTiles);
  uint32_t c[kSuperTiles];
#pragma unroll
  for (int u = 0; u < kSuperTiles; ++u) c[u] = (t0 + u < t1) ? tile_counts[static_cast<size_t>(t0 + u) * E + e] : 0u;
  uint32_t s = 0;
#pragma unroll
  for (int u = 0; u < kSuperTiles; ++u) s += c[u];
  super_counts[static_cast<size_t>(sb) * E + e] = s;
}

// ---- token-sharded dispatch (several GPUs, each with a contiguous token range in rank order)
// A shard's dispatch index is local.  The order of the whole batch is by (slot, token), so in
// slot p the assignments of earlier ranks come first: the whole-batch position of a local
// assignment at local position q in slot p is
//     G[p] + sum_{r' < rank} counts[r'][p] + (q - local_offsets[p]),
// G = exclusive prefix over slots of the counts summed over all ranks.  counts[r][p] is what the
// ranks exchange (an all-gather of E words per rank).

// counts[p] = number of local assignments in slot p
__global__ void fb_slot_counts_kernel(const uint32_t* __restrict__ slot_offsets, int E, uint32_t* __restrict__ counts) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p < E) counts[p] = slot_offsets[p + 1] - slot_offsets[p];
}

constexpr int kGlobalizeThreads = 256;   // >= FB_MAX_EXPERTS: one thread per slot for the shifts

struct GlobalizeParams {
  int32_t T, k, E, R, world, rank;
  const uint32_t* counts_all;        // [world][E]
  const uint32_t* local_offsets;     // [E+1]
  const int32_t* topk_ids;           // [T][k] (local)
  const int32_t* expert_to_slot;     // [E]
  int32_t* inv_perm;                 // [T*k] in: local positions, out: whole-batch positions
  uint32_t* slot_offsets;            // [E+1] out (whole batch)
  uint32_t* rank_offsets;            // [R+1] out
  uint32_t* rank_load;               // [R]   out
};

__global__ void __launch_bounds__(kGlobalizeThreads)
fb_dispatch_globalize_kernel(const __grid_constant__ GlobalizeParams p) {
  __shared__ uint32_t total[FB_MAX_EXPERTS];
  __shared__ uint32_t shift[FB_MAX_EXPERTS];
  __shared__ uint32_t G[FB_MAX_EXPERTS + 1];
  __shared__ int32_t slot_of[FB_MAX_EXPERTS];
  const int t = threadIdx.x;
  uint32_t before = 0;
  if (t < p.E) {
    uint32_t sum = 0;
    for (int r = 0; r < p.world; ++r) {
      const uint32_t c = p.counts_all[static_cast<size_t>(r) * p.E + t];
      if (r < p.rank) before += c;
      sum += c;
    }
    total[t] = sum;
    slot_of[t] = p.expert_to_slot[t];
  }
  __syncthreads();
  if (t == 0) {                                 // at most 256 slots: a serial prefix is cheapest here
    uint32_t run = 0;
    for (int s = 0; s < p.E; ++s) { G[s] = run; run += total[s]; }
    G[p.E] = run;
  }
  __syncthreads();
  if (t < p.E) shift[t] = G[t] + before - p.local_offsets[t];
  if (blockIdx.x == 0) {
    const int m = p.E / p.R;
    for (int s = t; s <= p.E; s += kGlobalizeThreads) p.slot_offsets[s] = G[s];
    for (int r = t; r <= p.R; r += kGlobalizeThreads) p.rank_offsets[r] = G[r == p.R ? p.E : r * m];
    for (int r = t; r < p.R; r += kGlobalizeThreads) p.rank_load[r] = G[(r + 1) * m] - G[r * m];
  }
  __syncthreads();
  const long long n = static_cast<long long>(p.T) * p.k;
  for (long long q = static_cast<long long>(blockIdx.x) * kGlobalizeThreads + t; q < n;
       q += static_cast<long long>(gridDim.x) * kGlobalizeThreads) {
    const int e = p.topk_ids[q];
    const int s = (e >= 0 && e < p.E) ? slot_of[e] : -1;
    if (s >= 0 && s < p.E) p.inv_perm[q] = static_cast<int32_t>(static_cast<uint32_t>(p.inv_perm[q]) + shift[s]);
  }
}

}  // namespace fb
