// Ordered fold shared by the kernels that compute per-segment peaks from event values:
// the associative, non-commutative operator on (sum, max prefix, arg max), its warp-level
// forms, and the distributed per-warp state that carries a segment across chunks.
#pragma once

#include "llmem_model.cuh"

namespace llmem {

struct Agg {
  i64 sum, mx, idx;  // idx: virtual (alignment-shifted) global index of the first arg max
  i64 valid;         // 0: identity
};

__device__ __forceinline__ Agg agg_identity() { return Agg{0, 0, -1, 0}; }

// ordered fold: a covers earlier events than b
__device__ __forceinline__ Agg agg_fold(const Agg& a, const Agg& b) {
  if (!a.valid) return b;
  if (!b.valid) return a;
  Agg r;
  r.sum = a.sum + b.sum;
  const i64 cand = a.sum + b.mx;
  const bool take = cand > a.mx;  // ties keep the earlier index
  r.mx = take ? cand : a.mx;
  r.idx = take ? b.idx : a.idx;
  r.valid = 1;
  return r;
}

__device__ __forceinline__ Agg agg_shfl_down(const Agg& a, int delta) {
  Agg r;
  r.sum = __shfl_down_sync(0xffffffffu, a.sum, delta);
  r.mx = __shfl_down_sync(0xffffffffu, a.mx, delta);
  r.idx = __shfl_down_sync(0xffffffffu, a.idx, delta);
  r.valid = __shfl_down_sync(0xffffffffu, (int)a.valid, delta);
  return r;
}

// lane 0 receives the in-order fold of all 32 lanes
__device__ __forceinline__ Agg warp_fold(Agg a, int lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    Agg o = agg_shfl_down(a, d);
    if (lane + d < 32) a = agg_fold(a, o);
  }
  return a;
}

// The scan kernel stores the bare result of a finished segment: its largest prefix
// sum and the segment-relative index of the first event attaining it.  The finish
// kernel adds the per-configuration offset.
__device__ __forceinline__ void write_raw(i64 seg, const Agg& a, i64 seg_vstart, i64* __restrict__ peak_out,
                                          i64* __restrict__ index_out) {
  peak_out[seg] = a.valid ? a.mx : 0;
  if (index_out) index_out[seg] = a.valid ? a.idx - seg_vstart : -1;
}

template <bool kRound>
__device__ __forceinline__ i64 ev(i64 d) { return kRound ? page_round_signed(d) : d; }

// In-order fold of tile-local events [lo, hi) by one warp; lanes take contiguous
// chunks of odd length (distinct banks).  `vbase` is the virtual index of tile slot 0.
template <bool kRound>
__device__ __forceinline__ Agg warp_fold_range(const i64* __restrict__ tile, int lo, int hi, int lane, i64 vbase) {
  const int len = hi - lo;
  const int ch = ((len + 31) / 32) | 1;
  const int a = lo + lane * ch;
  const int b = a + ch < hi ? a + ch : hi;
  Agg g = agg_identity();
  if (a < b) {
    i64 s = ev<kRound>(tile[a]), m = s;
    int ix = a;
    for (int j = a + 1; j < b; ++j) {
      s += ev<kRound>(tile[j]);
      if (s > m) { m = s; ix = j; }
    }
    g = Agg{s, m, vbase + ix, 1};
  }
  return warp_fold(g, lane);
}

// Scratch payload: per warp a head partial (segment that began in an earlier warp's
// range) and a tail partial (segment that continues into a later warp's range).
struct WarpPartials {
  Agg head, tail;
};

// Result of the fast path before it is widened to an Agg: chunk-local arg max.
struct Fold3 {
  i64 sum, mx;
  int ix;
};

__device__ __forceinline__ Fold3 fold3(const Fold3& a, const Fold3& b) {
  Fold3 r;
  r.sum = a.sum + b.sum;
  const i64 cand = a.sum + b.mx;
  const bool take = cand > a.mx;
  r.mx = take ? cand : a.mx;
  r.ix = take ? b.ix : a.ix;
  return r;
}

// In-order fold of the 16-byte words [V0, V1) of a lane's span (compile-time bounds).
template <bool kRound, int V0, int V1>
__device__ __forceinline__ Fold3 fold_words(const longlong2* x) {
  Fold3 f;
  f.sum = ev<kRound>(x[V0].x);
  f.mx = f.sum;
  f.ix = 2 * V0;
#pragma unroll
  for (int j = V0; j < V1; ++j) {
    if (j > V0) {
      f.sum += ev<kRound>(x[j].x);
      if (f.sum > f.mx) { f.mx = f.sum; f.ix = 2 * j; }
    }
    f.sum += ev<kRound>(x[j].y);
    if (f.sum > f.mx) { f.mx = f.sum; f.ix = 2 * j + 1; }
  }
  return f;
}


// Fold of the current segment so far, kept distributed over a warp: `base` (the same in
// every lane) is the sum of all events folded; each lane remembers the best prefix value
// it has seen among its own events and where.  Every lane only ever replaces its
// candidate by a strictly larger, later one, and the final reduction prefers the smaller
// index among equals, so the result is the first arg max.
struct SegmentFolder {
  i64 base = 0, best_v = 0, best_i = 0;
  bool lane_has = false, seg_has = false;

  // A chunk whose lanes hold consecutive spans of kPerLane events starting at index t0:
  // `f` is the lane's own fold, with f.ix relative to the lane's span.
  template <int kPerLane>
  __device__ __forceinline__ void add_spans(const Fold3& f, i64 t0, int lane) {
    i64 inc = f.sum;  // prefix of the lane sums across the warp
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const i64 o = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += o;
    }
    const i64 cand = base + (inc - f.sum) + f.mx;
    if (!lane_has || cand > best_v) {
      best_v = cand;
      best_i = t0 + lane * kPerLane + f.ix;
      lane_has = true;
    }
    base += __shfl_sync(0xffffffffu, inc, 31);
    seg_has = true;
  }

  // The same for spans of any length: `ix` is relative to t0, and a lane that holds no
  // events passes has == false (and sum 0).
  __device__ __forceinline__ void add_lane_folds(i64 sum, i64 mx, int ix, bool has, i64 t0, int lane) {
    i64 inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const i64 o = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += o;
    }
    if (has) {
      const i64 cand = base + (inc - sum) + mx;
      if (!lane_has || cand > best_v) {
        best_v = cand;
        best_i = t0 + ix;
        lane_has = true;
      }
    }
    base += __shfl_sync(0xffffffffu, inc, 31);
    if (__any_sync(0xffffffffu, has)) seg_has = true;
  }

  // A piece whose fold lane `src` holds: joins through lane 0's candidate.
  __device__ __forceinline__ void add_from_lane(const Agg& g, int src, int lane) {
    const i64 g_sum = __shfl_sync(0xffffffffu, g.sum, src);
    const i64 g_mx = __shfl_sync(0xffffffffu, g.mx, src);
    const i64 g_idx = __shfl_sync(0xffffffffu, g.idx, src);
    const bool g_valid = __shfl_sync(0xffffffffu, (int)g.valid, src) != 0;
    if (!g_valid) return;
    if (lane == 0) {
      const i64 cand = base + g_mx;
      if (!lane_has || cand > best_v) {
        best_v = cand;
        best_i = g_idx;
        lane_has = true;
      }
    }
    base += g_sum;
    seg_has = true;
  }

  // A piece already folded by the warp (result in lane 0): joins through lane 0's candidate.
  __device__ __forceinline__ void add_piece(const Agg& g, int lane) {
    const i64 g_sum = __shfl_sync(0xffffffffu, g.sum, 0);
    const bool g_valid = __shfl_sync(0xffffffffu, (int)g.valid, 0) != 0;
    if (!g_valid) return;
    if (lane == 0) {
      const i64 cand = base + g.mx;
      if (!lane_has || cand > best_v) {
        best_v = cand;
        best_i = g.idx;
        lane_has = true;
      }
    }
    base += g_sum;
    seg_has = true;
  }

  // A piece whose fold every lane already holds (the same value in all lanes).
  __device__ __forceinline__ void add_uniform(const Agg& g, int lane) {
    if (lane == 0) {
      const i64 cand = base + g.mx;
      if (!lane_has || cand > best_v) {
        best_v = cand;
        best_i = g.idx;
        lane_has = true;
      }
    }
    base += g.sum;
    seg_has = true;
  }

  // All lanes: reduce the state to one Agg (valid in every lane) and reset it.
  __device__ __forceinline__ Agg take() {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      const i64 ov = __shfl_xor_sync(0xffffffffu, best_v, d);
      const i64 oi = __shfl_xor_sync(0xffffffffu, best_i, d);
      const bool oh = __shfl_xor_sync(0xffffffffu, (int)lane_has, d) != 0;
      if (oh && (!lane_has || ov > best_v || (ov == best_v && oi < best_i))) {
        best_v = ov;
        best_i = oi;
        lane_has = true;
      }
    }
    Agg a{base, best_v, best_i, seg_has ? 1 : 0};
    base = 0;
    lane_has = false;
    seg_has = false;
    return a;
  }

  // Segment `seg` (starting at index seg_start) ends here: store its bare result, or, if it
  // began before this warp's range (range_lo), leave the part seen here as the head partial.
  __device__ __forceinline__ void finish_segment(i64 seg, i64 seg_start, i64 range_lo, WarpPartials* my_partials,
                                                 i64* __restrict__ peak_out, i64* __restrict__ index_out, int lane,
                                                 const Guard& g) {
    const Agg run = take();
    if (lane == 0 && in_bounds(seg >= 0 && seg < g.n, g, kSiteResult)) {
      if (seg_start >= range_lo) write_raw(seg, run, seg_start, peak_out, index_out);
      else my_partials->head = run;
    }
  }

  // The warp's range ends while a segment is still open: leave the part seen as a partial.
  __device__ __forceinline__ void finish_range(i64 seg_start, i64 range_lo, WarpPartials* my_partials, int lane) {
    const Agg run = take();
    if (lane == 0 && run.valid) {
      if (seg_start >= range_lo) my_partials->tail = run;
      else my_partials->head = run;
    }
  }
};

// Loads a lane's span of kPerLane events (16-byte words) and folds it as four
// independent in-order chains over quarters of the span.
template <bool kRound, int kPerLane>
__device__ __forceinline__ Fold3 fold_lane_span(const i64* __restrict__ span) {
  constexpr int kVec = kPerLane / 2;
  constexpr int q1 = kVec / 4, q2 = kVec / 2, q3 = (3 * kVec) / 4;
  const longlong2* src = reinterpret_cast<const longlong2*>(span);
  longlong2 x[kVec];
#pragma unroll
  for (int j = 0; j < kVec; ++j) x[j] = src[j];
  const Fold3 f0 = fold_words<kRound, 0, q1>(x), f1 = fold_words<kRound, q1, q2>(x);
  const Fold3 f2 = fold_words<kRound, q2, q3>(x), f3 = fold_words<kRound, q3, kVec>(x);
  return fold3(fold3(f0, f1), fold3(f2, f3));
}

// What a warp reports for one part of a long segment that several warps write (fused.cu): the
// largest prefix sum inside the part, counted from the segment's start, and its position.
struct PartResult {
  i64 mx, idx;
  i64 has;
  i64 sum;  // sum of the part's events (used where the parts' prefix sums are relative to the part)
};

// Segments cut into parts, for the finishing pass: segment i has more than `lane_max` events,
// its parts of `part` events each report to results[first_part[i] ...].
struct PartsOfSegments {
  const i64* first_part = nullptr;  // one entry per segment, stride `stride` bytes; null: no segment is cut
  size_t stride = 0;
  const PartResult* results = nullptr;
  i64 lane_max = 0, part = 1;
  // true: a part's mx counts from the part's own start (the scan of a given list cannot know what
  // precedes the part) and the parts are joined in order with their sums; false: it counts
  // from the segment's start (the expansion knows the runs before the part)
  bool relative = false;
};

// Host launcher of the finishing pass (defined with the scan kernels): one thread per
// segment folds the partials of segments that cross the warps' blocks (block j starts at
// bounds[j], bounds[n_warps] = end), joins the parts of segments written in parts, defines
// empty segments, adds m_base + lm_p (m_base alone for the second estimator, `dnn`) and marks
// inadmissible configurations.
llmem_status launch_scan_finish(const i64* offsets, i64 n, int shift, const llmem_config* cfg, i64* peak_out,
                                i64* index_out, const i64* bounds, i64 n_warps, const WarpPartials* partials,
                                cudaStream_t stream, PartsOfSegments parts = PartsOfSegments(), bool dnn = false);

// Host side of the expansion by segment owners (defined with its kernels): descriptor table,
// list of parts, then every segment written by its owner into delta_out; with `fold` the bare
// per-segment results as well.  `scratch` has llmem_expand_scan's layout, header cleared.
llmem_status expand_by_owners(const llmem_config* cfg, i64 n, const i64* offsets, i64 total_events, i64* delta_out,
                              int round_bits /* bit 0: rounded values, bit 1: second estimator */, bool fold,
                              i64* peak_out, i64* index_out, void* scratch, PartsOfSegments* parts_out,
                              cudaStream_t stream);

}  // namespace llmem
