// Stage 3 of the method on one device (Method overview, "Weight Transfer"): the accepted
// swaps of a plan applied to the expert weights.  Logical EP ranks are a mapping on one GPU
// here, so "exchange expert weights between two ranks" is an exchange of two slot images
// inside one HBM buffer.  Every expert moves at most once per plan, hence the swaps touch
// disjoint slot pairs and all of them run in one launch; the exchange is in place (each
// 16-byte unit is read from both slots and written crosswise by one thread), so no staging
// memory is needed.  The number of swaps is read on the device: the launch can follow the
// planner on the stream without a host round trip.  A fixed grid strides over the
// (swap, 32 KB piece) pairs, so a large capacity with few accepted swaps costs nothing.
//
// HBM bound: 4 * expert_bytes of traffic per swap (two reads, two writes).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/freebalance.h"

namespace fb {

constexpr int kMigrateThreads = 256;
constexpr int kMigrateUnroll = 8;          // 16-byte units per thread and slot in flight
constexpr int kMigrateBlocks = 148 * 8;   // fixed grid: blocks stride over (swap, piece) pairs

struct MigrateParams {
  uint8_t* slot_weights;          // [E][expert_bytes], slot major
  uint64_t expert_bytes;          // distance between slot images, multiple of 16
  uint64_t copy_bytes;            // bytes exchanged per image (= expert_bytes except when calibrating)
  int32_t E;
  const int32_t* expert_to_slot;  // [E] placement BEFORE the plan
  const fb_swap* swaps;           // [max_swaps]
  const int32_t* n_swaps;         // device scalar
  int32_t max_swaps;              // capacity of swaps[]
  int32_t* status;                // optional
};

__global__ void __launch_bounds__(kMigrateThreads)
fb_swap_weights_kernel(const __grid_constant__ MigrateParams p) {
  const int n = min(*p.n_swaps, p.max_swaps);
  const uint64_t n_vec = p.copy_bytes / 16;
  const uint64_t per_piece = static_cast<uint64_t>(kMigrateThreads) * kMigrateUnroll;
  const uint64_t pieces = (n_vec + per_piece - 1) / per_piece;      // per swap
  const uint64_t total = pieces * static_cast<uint64_t>(n > 0 ? n : 0);
  for (uint64_t unit = blockIdx.x; unit < total; unit += gridDim.x) {
    const int s = static_cast<int>(unit / pieces);
    const uint64_t base = (unit - static_cast<uint64_t>(s) * pieces) * per_piece;
    const fb_swap sw = p.swaps[s];
    const int ea = sw.expert_src, eb = sw.expert_dst;
    if (ea < 0 || ea >= p.E || eb < 0 || eb >= p.E || ea == eb) {          // skip the swap, report it
      if (p.status != nullptr && threadIdx.x == 0 && base == 0) atomicCAS(p.status, 0, FB_ERR_RANGE);
      continue;
    }
    const int pa = p.expert_to_slot[ea], pb = p.expert_to_slot[eb];
    if (pa < 0 || pa >= p.E || pb < 0 || pb >= p.E || pa == pb) {
      if (p.status != nullptr && threadIdx.x == 0 && base == 0) atomicCAS(p.status, 0, FB_ERR_BAD_PLACEMENT);
      continue;
    }
    uint4* A = reinterpret_cast<uint4*>(p.slot_weights + static_cast<uint64_t>(pa) * p.expert_bytes);
    uint4* B = reinterpret_cast<uint4*>(p.slot_weights + static_cast<uint64_t>(pb) * p.expert_bytes);
    uint4 a[kMigrateUnroll], b[kMigrateUnroll];
#pragma unroll
    for (int u = 0; u < kMigrateUnroll; ++u) {
      const uint64_t i = base + static_cast<uint64_t>(u) * kMigrateThreads + threadIdx.x;
      if (i < n_vec) { a[u] = __ldcs(A + i); b[u] = __ldcs(B + i); }      // streamed once: evict first
    }
#pragma unroll
    for (int u = 0; u < kMigrateUnroll; ++u) {
      const uint64_t i = base + static_cast<uint64_t>(u) * kMigrateThreads + threadIdx.x;
      if (i < n_vec) { __stcs(A + i, b[u]); __stcs(B + i, a[u]); }
    }
  }
}

}  // namespace fb
