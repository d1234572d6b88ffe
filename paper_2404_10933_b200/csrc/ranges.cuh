// Work distribution of the kernels that stream over a materialised event list.
//
// The list is cut into chunks (one warp's unit of work) and the chunks into contiguous blocks,
// one per warp (scan) or many per warp, claimed on request (expansion); a warp streams a
// block from end to end, which is the access pattern HBM likes best.  Blocks of
// equal length would be balanced if every event cost the same, but a segment boundary costs
// about as much as a thousand events (descriptor, fold reduction, result), and lists of many
// short segments sit next to each other.  So the blocks are balanced by a cost model instead:
//
//     cost = events + kappa * segments
//
// The cumulative cost at the start of segment s is offsets[s] + kappa * s, a non-decreasing
// function of s that every warp can search on its own, so no pre-pass and no scratch are
// needed: block j of W begins where the cumulative cost reaches j / W of the total, rounded
// down to a chunk boundary.
#pragma once

#include "llmem_model.cuh"

namespace llmem {

#ifndef LLMEM_MAX_STREAM_WARPS
#define LLMEM_MAX_STREAM_WARPS 65536
#endif
constexpr int kMaxStreamWarps = LLMEM_MAX_STREAM_WARPS;  // upper bound on the (virtual) warps of a streaming grid

// Warps of a streaming launch.  `resident` is what the GPU holds at once; the grid may hold
// `oversub` times as many, so that the hardware block scheduler hands out the blocks as SMs
// become free (SMs do not all reach HBM at the same rate, and a grid of exactly the resident
// size ends when its slowest SM does).  No warp gets fewer than `min_chunks` chunks unless
// the resident warps alone would.
inline i64 stream_warps(i64 resident, int oversub, i64 nchunks, i64 min_chunks) {
  i64 warps = resident * (oversub < 1 ? 1 : oversub);
  const i64 by_work = nchunks / (min_chunks < 1 ? 1 : min_chunks);
  if (warps > by_work) warps = by_work > resident ? by_work : resident;
  if (warps > kMaxStreamWarps) warps = kMaxStreamWarps;
  if (warps > nchunks) warps = nchunks;
  return warps < 1 ? 1 : warps;
}

// Smallest s in [0, n] with offsets[s + 1] + kappa * (s + 1) > target (n if none), found by
// the whole warp: every round the 32 lanes probe 32 evenly spaced candidates, so a round costs
// one memory latency and shrinks the interval 32-fold.  All lanes return the same value.
__device__ __forceinline__ i64 warp_search_cost(const i64* __restrict__ offsets, i64 n, i64 kappa, i64 target,
                                                int lane) {
  i64 lo = 0, hi = n;  // the answer lies in [lo, hi]
  while (lo < hi) {
    const i64 span = hi - lo;  // candidates lo .. hi-1 (hi itself needs no probe)
    const i64 step = (span + 31) / 32;
    i64 p = lo + (i64)(lane + 1) * step - 1;  // increasing with the lane
    if (p > hi - 1) p = hi - 1;
    const bool beyond = __ldg(offsets + p + 1) + kappa * (p + 1) > target;
    const unsigned ballot = __ballot_sync(0xffffffffu, beyond);
    if (ballot == 0) {
      lo = hi;  // lane 31 probed hi-1 and it does not qualify: the answer is hi
    } else {
      const int first = __ffs(ballot) - 1;
      const i64 p_first = __shfl_sync(0xffffffffu, p, first);
      const i64 p_prev = __shfl_sync(0xffffffffu, p, first > 0 ? first - 1 : 0);
      hi = p_first;
      if (first > 0) lo = p_prev + 1;
    }
  }
  return lo;
}

// Start of block j of n_warps, as an index into the (alignment-shifted) event axis
// [0, v_end), a multiple of `chunk`; block 0 starts at 0 and block n_warps at v_end.  Also
// returns, through *seg_out, the segment that contains that position's first event or
// the first one after it (n if none).
__device__ __forceinline__ i64 warp_block_start(const i64* __restrict__ offsets, i64 n, int shift, i64 v_end,
                                                i64 j, i64 n_warps, i64 kappa, i64 chunk, int lane,
                                                i64* seg_out) {
  i64 pos;
  if (j <= 0) {
    pos = 0;
  } else if (j >= n_warps) {
    pos = v_end;
  } else {
    const i64 total = v_end - shift;
    const i64 total_cost = total + kappa * n;
    const i64 target = (total_cost / n_warps) * j + ((total_cost % n_warps) * j) / n_warps;
    const i64 s = warp_search_cost(offsets, n, kappa, target, lane);
    if (s >= n) {
      pos = v_end;
    } else {
      // the target falls into segment s: kappa of its cost comes first, then one per event
      const i64 seg_lo = __ldg(offsets + s), seg_hi = __ldg(offsets + s + 1);
      i64 into = target - (seg_lo + kappa * s) - kappa;
      if (into < 0) into = 0;
      if (into > seg_hi - seg_lo) into = seg_hi - seg_lo;
      pos = seg_lo + into + shift;
    }
    pos -= pos % chunk;
  }
  if (seg_out) {
    // smallest segment whose (shifted) end lies beyond pos: kappa = 0 turns the search into
    // one on offsets alone
    *seg_out = warp_search_cost(offsets, n, 0, pos - shift, lane);
  }
  return pos;
}

// Scratch layout of the kernels that leave per-warp partial results: a 256-byte header
// (first word: device status), the block starts of all warps (+1 for the end), then one
// head and one tail partial (32 bytes each) per warp.
constexpr size_t kBoundsOffset = 256;
constexpr size_t kPartialsOffset = kBoundsOffset + (size_t)(kMaxStreamWarps + 32) * sizeof(i64);
constexpr size_t kStreamScratchBytes = kPartialsOffset + (size_t)kMaxStreamWarps * 64;

}  // namespace llmem
