// Work list of the batched expert kernels: items, units and pieces.
//
// An item is (layer, expert, tile of `tok_tile` tokens of that expert's group); its channels are
// cut into at most kUnitsPerItem units of whole channel blocks (`blk_ch` channels each).  Items are
// laid end to end in a fixed order and every CTA takes an equal contiguous range of units; the
// part of an item inside one CTA's range is a piece.
#pragma once

#include "remoe_internal.cuh"

namespace remoe {
namespace {

constexpr int kPlanHeader = 8;                        // ints: n_items, n_units, ...

// ---------------------------------------------------------------------------------- plan
// Item list of one launch, in a fixed order: layer ascending; within a layer the distinct
// requests in request order (those matching the launch's filter), each cut into token tiles;
// then, in the resident phase, the shared experts, each cut into token tiles.
// plan[0] = n_items, plan[1] = n_units; item j at plan[8 + 4j]: {layer, candidate, tile, unit0}
// where candidate < B*K is a distinct-request index and candidate >= B*K a shared expert.
__device__ __forceinline__ int cand_tiles(const BatchArgs& a, int l, int c) {
  const DevStack& d = a.d;
  const int BK = d.B * d.K;
  if (a.layer >= 0 && l != a.layer) return 0;
  if (c >= BK) return a.phase == 0 ? (d.B + a.tok_tile - 1) / a.tok_tile : 0;
  if (c >= trace_n_unique(d.trace)[l]) return 0;
  const int hit = trace_hit(d.trace, d.L, BK)[l * BK + c];
  if (a.phase == 0) {
    if (!hit) return 0;
  } else {
    if (hit || trace_depth(d.trace, d.L, BK)[l * BK + c] != a.depth) return 0;
  }
  return (d.grp_count[l * BK + c] + a.tok_tile - 1) / a.tok_tile;
}

__device__ __forceinline__ int item_units(const BatchArgs& a, bool shared) {
  const DevStack& d = a.d;
  const int blocks = (shared ? d.Is : d.I) / a.blk_ch;
  const int per_unit = (blocks + kUnitsPerItem - 1) / kUnitsPerItem;
  return (blocks + per_unit - 1) / per_unit;
}

__global__ void __launch_bounds__(1024) plan_kernel(BatchArgs a) {
  __shared__ int warp_tot[32];
  __shared__ int s_carry;
  const DevStack& d = a.d;
  const int BK = d.B * d.K, P = BK + d.S;
  const int n_cand = d.L * P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < n_cand; base += 1024) {
    const int c = base + tid;
    const int l = c / P, cc = c % P;
    const int tiles = c < n_cand ? cand_tiles(a, l, cc) : 0;
    int v = tiles;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += t;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
      int w = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += t;
      }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const int first = s_carry + (warp ? warp_tot[warp - 1] : 0) + v - tiles;   // index of my first item
    const int u_r = item_units(a, false), u_s = d.S ? item_units(a, true) : 0;
    for (int t = 0; t < tiles; ++t) {
      const int j = first + t;
      if (j < a.max_items) {
        int* it = a.plan + kPlanHeader + 4 * j;
        it[0] = l; it[1] = cc; it[2] = t; it[3] = cc >= BK ? u_s : u_r;            // unit count for now
      }
    }
    __syncthreads();
    if (tid == 1023) s_carry = first + tiles;
    __syncthreads();
  }
  // Second pass: exclusive prefix of unit counts (items are few thousand at most).
  const int n_items = min(s_carry, a.max_items);
  __syncthreads();
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < n_items; base += 1024) {
    const int j = base + tid;
    const int units = j < n_items ? a.plan[kPlanHeader + 4 * j + 3] : 0;
    int v = units;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += t;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
      int w = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += t;
      }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const int excl = s_carry + (warp ? warp_tot[warp - 1] : 0) + v - units;
    if (j < n_items) a.plan[kPlanHeader + 4 * j + 3] = excl;
    __syncthreads();
    if (tid == 1023) s_carry = excl + units;
    __syncthreads();
  }
  if (tid == 0) {
    a.plan[0] = n_items;
    a.plan[1] = s_carry;
    if (s_carry < 0 || n_items >= a.max_items) atomicCAS(d.err, kErrNone, kErrBadIndex);
  }
}

struct PieceInfo {
  const char* base;       // expert block
  int l, cand, tile, n_tok;
  int blk0, blk1;         // channel-block range [blk0, blk1) of this piece
  int first_unit;
  bool shared;
};

// Decode the piece of item `j` that falls inside units [ua, ub).
__device__ __forceinline__ bool make_piece(const BatchArgs& a, int j, int ua, int ub, PieceInfo& p) {
  const DevStack& d = a.d;
  const int BK = d.B * d.K;
  const int* it = a.plan + kPlanHeader + 4 * j;
  p.l = it[0]; p.cand = it[1]; p.tile = it[2];
  const int unit0 = it[3];
  p.shared = p.cand >= BK;
  const int blocks = (p.shared ? d.Is : d.I) / a.blk_ch;
  const int per_unit = (blocks + kUnitsPerItem - 1) / kUnitsPerItem;
  const int units = (blocks + per_unit - 1) / per_unit;
  const int lo = max(ua, unit0) - unit0, hi = min(ub, unit0 + units) - unit0;
  if (lo >= hi) return false;
  p.first_unit = lo;
  p.blk0 = lo * per_unit;
  p.blk1 = min(blocks, hi * per_unit);
  if (p.shared) {
    p.base = d.shared_blocks + ((size_t)p.l * d.S + (p.cand - BK)) * d.shared_bytes;
    p.n_tok = min(a.tok_tile, d.B - p.tile * a.tok_tile);
  } else {
    const int slot = trace_slot(d.trace, d.L, BK)[p.l * BK + p.cand];
    if (slot < 0 || slot >= d.C) { atomicCAS(d.err, kErrNone, kErrBadIndex); return false; }
    p.base = d.slots + ((size_t)p.l * d.C + slot) * d.slot_bytes;
    p.n_tok = min(a.tok_tile, d.grp_count[p.l * BK + p.cand] - p.tile * a.tok_tile);
  }
  return true;
}


// First item whose unit range reaches past unit `ua`.
__device__ __forceinline__ int first_item(const BatchArgs& a, int n_items, int ua) {
  int lo = 0, hi = n_items - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a.plan[kPlanHeader + 4 * mid + 3] <= ua) lo = mid; else hi = mid - 1;
  }
  return lo;
}

}  // namespace
}  // namespace remoe
