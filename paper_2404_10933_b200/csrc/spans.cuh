// Expansion of event lists from a table of segment descriptors, for lists of short and
// medium segments.
//
// A list is a sequence of pieces, each the part of one run (equal events, two alternating
// events, or a short period of operator outputs) that is written in one go.  Two ways of
// writing them are provided.  A lane on its own (emit_piece): it owns a whole segment, stages
// its events row by row in shared memory and folds them into its own (sum, largest prefix,
// first position attaining it).  A warp together (emit_piece_by_warp): the lanes share out
// the 16-byte stores of a piece and every lane takes the same fold.  Either way a run of
// period 1 or 2 is folded in closed form, because its prefix sums are arithmetic
// progressions.
//
// Descriptors are read from global memory through the read-only path; nothing of a descriptor
// is kept in shared memory.
#pragma once

#include "expand.cuh"
#include "fold.cuh"

namespace llmem {

// A run record as read from the table.
struct TableRun {
  int cnt, period;
  u32 code;
  int start;
  i64 a, b, c;
  u32 links;
};

// (plain loads: a descriptor may sit in the table in device memory or in a copy of it in
// shared memory)
__device__ __forceinline__ int4 load_run_head(const SegDesc* d, int r) {
  return *reinterpret_cast<const int4*>(&d->run[r]);
}

__device__ __forceinline__ TableRun load_run(const SegDesc* d, int r) {
  const int4* p = reinterpret_cast<const int4*>(&d->run[r]);
  const int4 h = *p;
  const longlong2 ab = *reinterpret_cast<const longlong2*>(p + 1);
  const longlong2 cl = *reinterpret_cast<const longlong2*>(p + 2);
  return TableRun{h.x, h.y, (u32)h.z, h.w, ab.x, ab.y, cl.x, (u32)cl.y};
}

// Asks for the whole of one descriptor to be brought into the L2 cache: its records are read
// one at a time as the walk of the segment reaches them, and the table of a long list is in
// device memory by then, so without this every run would begin with a miss.
__device__ __forceinline__ void prefetch_descriptor(const SegDesc* d) {
  const unsigned char* p = reinterpret_cast<const unsigned char*>(d);
#pragma unroll
  for (int k = 0; k < (int)((sizeof(SegDesc) + 127) / 128); ++k) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p + 128 * k));
  asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p + sizeof(SegDesc) - 16));
}

// init_n, dyn_n, os_n, invalid of a descriptor
__device__ __forceinline__ int4 load_desc_counts(const SegDesc* d) {
  return *(reinterpret_cast<const int4*>(d) + 1);
}

// Run, offset inside it and iteration of event `pos` (0-based inside the segment) of a valid
// descriptor.  Inside an iteration the run is found by bisection on the runs' start positions
// (empty runs share their start with the next run, so the last run that starts at or before
// the position is the non-empty one that holds it).
__device__ __forceinline__ void locate_in_table(const SegDesc* d, const int4& counts, u32 pos,
                                                int* r_out, int* o_out, int* it_out) {
  const u32 init_n = (u32)counts.x, dyn_n = (u32)counts.y, os_n = (u32)counts.z;
  *it_out = 1;
  if (pos < init_n) {
    *r_out = pos < 2 ? 0 : 1;
    *o_out = pos < 2 ? (int)pos : (int)(pos - 2);
    return;
  }
  u32 q = pos - init_n;
  if (q >= dyn_n) {
    q -= dyn_n;
    if (q < os_n) {
      // the embedding tensors' states, then the layers'
      const u32 s_layers = (u32)load_run_head(d, kOsLast).w;
      *r_out = q >= s_layers ? kOsLast : kOsFirst;
      *o_out = (int)(q >= s_layers ? q - s_layers : q);
      return;
    }
    q -= os_n;
    *it_out = 2 + (int)(q / dyn_n);
    q = q % dyn_n;
  }
  int r = kDynFirst;
  u32 base = 0;
#pragma unroll
  for (int step = 8; step >= 1; step >>= 1) {
    if (r + step <= kDynLast) {
      const u32 s = (u32)load_run_head(d, r + step).w;
      if (s <= q) {
        r += step;
        base = s;
      }
    }
  }
  *r_out = r;
  *o_out = (int)(q - base);
}

// A lane's fold of the events it has emitted for its current segment: chunk-local position.
struct LaneFold {
  i64 sum = 0, mx = 0;
  int ix = 0;
  bool has = false;
  __device__ __forceinline__ void offer(i64 value, int index) {
    if (!has || value > mx) {  // later candidates replace only when strictly larger: first arg max
      mx = value;
      ix = index;
      has = true;
    }
  }
};

// Cursor of one lane inside the list: its segment's descriptor and the run it is in.
struct SpanCursor {
  const SegDesc* d;
  int r, rem, phase, period;
  u32 code, links;
  bool first_iter;  // the optimizer states have not been passed yet: they follow this iteration's frees
  i64 a, b, c;

  __device__ __forceinline__ void enter(const TableRun& rn, int r_, int o) {
    r = r_;
    rem = rn.cnt - o;
    period = rn.period;
    code = rn.code;
    links = rn.links;
    a = rn.a;
    b = rn.b;
    c = rn.c;
    phase = rn.period == 1 ? 0 : (rn.period == 2 ? (o & 1) : (int)((u32)o % (u32)rn.period));
  }

  // A stretch of zeros: a segment that has events but no valid descriptor, or positions
  // that no segment covers.
  __device__ __forceinline__ void enter_zeros(i64 remaining) {
    d = nullptr;
    r = 0;
    rem = remaining > 0x7fffffff ? 0x7fffffff : (int)remaining;
    period = 1;
    phase = 0;
    code = 0;
    links = 0;
    first_iter = true;
    a = b = c = 0;
  }

  // Position the cursor on event `pos` of the segment described by `desc`.
  __device__ __forceinline__ void seek(const SegDesc* desc, u32 pos, i64 seg_remaining) {
    const int4 counts = load_desc_counts(desc);
    if (counts.w) {
      enter_zeros(seg_remaining);
      return;
    }
    d = desc;
    int r_, o, it;
    locate_in_table(desc, counts, pos, &r_, &o, &it);
    first_iter = it == 1 && r_ < kOsFirst;
    enter(load_run(desc, r_), r_, o);
  }

  // Position the cursor on the first event of the segment described by `desc`.
  __device__ __forceinline__ void start(const SegDesc* desc, i64 seg_remaining) {
    if (load_desc_counts(desc).w) {
      enter_zeros(seg_remaining);
      return;
    }
    d = desc;
    first_iter = true;
    enter(load_run(desc, 0), 0, 0);
  }

  // Move to the next non-empty run: the record names it (for the first iteration, after whose
  // frees the optimizer states follow, and for the later ones).
  __device__ __forceinline__ void next_run() {
    if (d == nullptr) {  // zeros go on for as long as they are asked for
      rem = 0x7fffffff;
      return;
    }
    const int r_ = (int)((first_iter ? links : (links >> 8)) & 0xffu);
    if (r_ >= kOsFirst) first_iter = false;
    enter(load_run(d, r_), r_, 0);
  }

  __device__ __forceinline__ i64 value(int ph) const {
    const u32 k = (code >> (2 * ph)) & 3u;
    return k == 0 ? a : (k == 1 ? b : c);
  }
};

// One lane emits the next m events (1 <= m <= min(rem, kRowEvents)) of its cursor's run into
// dst[0 .. m), dst being slot `slot` of a 16-byte aligned row (the parity of the slot decides
// where 16-byte stores may start), and folds them into `f`; `at` is the position the first
// of them has in the lane's segment.  The fold takes page-rounded values when the list itself
// is written raw (kRoundFold).  Closed forms as in emit_piece_by_warp below.
constexpr int kRowEvents = 16;  // events a lane stages per step: one 128-byte line
template <bool kFold, bool kRoundFold>
__device__ __forceinline__ void emit_piece(i64* __restrict__ dst, int slot, int at, int m, SpanCursor& cur, LaneFold& f) {
  if (cur.period <= 2) {
    // x0 on the piece's even offsets, x1 on its odd ones (equal for a constant run)
    const bool odd = cur.period == 2 && cur.phase;
    const i64 x0 = odd ? cur.b : cur.a;
    const i64 x1 = cur.period == 2 ? (odd ? cur.a : cur.b) : cur.a;
    const int j0 = slot & 1;
    if (j0) dst[0] = x0;  // brings the rest to a 16-byte boundary
    const i64 e0 = j0 ? x1 : x0, e1 = j0 ? x0 : x1;
    longlong2* v = reinterpret_cast<longlong2*>(dst + j0);
    const int pairs = (m - j0) >> 1;
#pragma unroll
    for (int k = 0; k < kRowEvents / 2; ++k)
      if (k < pairs) v[k] = make_longlong2(e0, e1);
    if (j0 + 2 * pairs < m) dst[j0 + 2 * pairs] = e0;
    if (kFold) {
      const i64 y0 = ev<kRoundFold>(x0), y1 = ev<kRoundFold>(x1);
      const i64 S = y0 + y1, s = f.sum;
      const int n_even = (m + 1) >> 1, n_odd = m >> 1;
      const bool rising = S > 0;
      const int even_at = rising ? 2 * (n_even - 1) : 0, odd_at = rising ? 2 * n_odd - 1 : 1;
      const i64 even_v = s + y0 + (rising ? (i64)(n_even - 1) * S : 0);
      const i64 odd_v = s + (rising ? (i64)n_odd * S : S);
      const bool even_first = even_at < odd_at || n_odd == 0;
      f.offer(even_first ? even_v : odd_v, at + (even_first ? even_at : odd_at));
      if (n_odd > 0) f.offer(even_first ? odd_v : even_v, at + (even_first ? odd_at : even_at));
      f.sum = s + (i64)n_odd * S + ((m & 1) ? y0 : 0);
    }
    if (cur.period == 2) cur.phase ^= (m & 1);
  } else {
    int ph = cur.phase;
    for (int j = 0; j < m; ++j) {
      const i64 x = cur.value(ph);
      dst[j] = x;
      if (kFold) {
        f.sum += ev<kRoundFold>(x);
        f.offer(f.sum, at + j);
      }
      if (++ph == cur.period) ph = 0;
    }
    cur.phase = ph;
  }
  cur.rem -= m;
}

// A fold that every lane of a warp holds alike: the current segment so far, with the global
// position of the first arg max.
struct WarpFold {
  i64 sum = 0, mx = 0, idx = -1;
  bool has = false;
  __device__ __forceinline__ void offer(i64 value, i64 index) {
    if (!has || value > mx) {
      mx = value;
      idx = index;
      has = true;
    }
  }
  // appends a fold of later events
  __device__ __forceinline__ void append(const Agg& g) {
    if (!g.valid) return;
    offer(sum + g.mx, g.idx);
    sum += g.sum;
  }
  __device__ __forceinline__ Agg agg() const { return Agg{sum, mx, idx, has ? 1 : 0}; }
};

// How often the values a, b and c of a periodic run occur among its positions
// [from, from + m), `from` below the period: the 2-bit codes of one period are counted with
// population counts, whole periods by multiplication.
__device__ __forceinline__ void count_kinds(u32 code, u32 period, u32 from, u32 m, u32* n_b, u32* n_c) {
  const u32 low = code & 0x55555555u, high = (code >> 1) & 0x55555555u;
  const u32 is_b = low & ~high, is_c = high & ~low;  // one bit per position, at bit 2 * position
  const unsigned long long all = period >= 16 ? ~0ull : ((1ull << (2 * period)) - 1);
  const u32 per_b = __popc(is_b & (u32)all), per_c = __popc(is_c & (u32)all);
  const u32 to = from + m, whole = to / period, rest = to - whole * period;
  const u32 head = (u32)((1ull << (2 * from)) - 1), tail = (u32)((1ull << (2 * rest)) - 1);
  *n_b = whole * per_b + __popc(is_b & tail) - __popc(is_b & head);
  *n_c = whole * per_c + __popc(is_c & tail) - __popc(is_c & head);
}

// The whole warp emits the next m events (1 <= m <= min(rem, kExpChunk)) of the cursor's run,
// the same cursor in every lane, into chunk-local positions [l0, l0 + m) of buf and folds them
// into `f` (the same in every lane); t0 is the list position of buf[0].
//
// A run of period 1 or 2 is written as 16-byte pairs dealt out to the lanes.  Its prefix sums
// are two arithmetic progressions with the same step S (the sum of the two values): both are
// largest at their last term if S > 0 and at their first otherwise, so two candidates, taken
// in the order of their positions, give the first arg max.
//
// A run of a longer period (operator outputs of a layer, optimizer states of a layer's
// tensors, the logits with their copies) is written position by position.  If its values all
// have one sign the prefix sums are monotone and only the piece's sum is needed, which the
// counts of each value give; a few events are folded one by one; anything else by the lanes
// over consecutive parts of the piece, joined with shuffles.
template <bool kFold, bool kRoundFold>
__device__ __forceinline__ void emit_piece_by_warp(i64* __restrict__ buf, int l0, int m, SpanCursor& cur, WarpFold& f,
                                                   i64 t0, int lane) {
  const i64 at = t0 + l0;
  if (cur.period <= 2) {
    const bool odd = cur.period == 2 && cur.phase;
    const i64 x0 = odd ? cur.b : cur.a;
    const i64 x1 = cur.period == 2 ? (odd ? cur.a : cur.b) : cur.a;
    const int j0 = l0 & 1, end = l0 + m;
    if (j0 && lane == 0) buf[l0] = x0;  // brings the rest to a 16-byte boundary
    const i64 e0 = j0 ? x1 : x0, e1 = j0 ? x0 : x1;
    const int a0 = l0 + j0, pairs = (end - a0) >> 1;
    longlong2* v = reinterpret_cast<longlong2*>(buf + a0);
#pragma unroll 3
    for (int q = lane; q < pairs; q += 32) v[q] = make_longlong2(e0, e1);
    if (((end - a0) & 1) && lane == 31) buf[end - 1] = e0;
    if (!kFold) {
      if (cur.period == 2) cur.phase ^= (m & 1);
      cur.rem -= m;
      return;
    }
    const i64 y0 = ev<kRoundFold>(x0), y1 = ev<kRoundFold>(x1);
    const i64 S = y0 + y1, s = f.sum;
    const int n_even = (m + 1) >> 1, n_odd = m >> 1;
    const bool rising = S > 0;
    // offsets of the two candidates: the ends of the progressions if they rise, else their starts
    const int even_at = rising ? 2 * (n_even - 1) : 0, odd_at = rising ? 2 * n_odd - 1 : 1;
    const i64 even_v = s + y0 + (rising ? (i64)(n_even - 1) * S : 0);
    const i64 odd_v = s + (rising ? (i64)n_odd * S : S);
    const bool even_first = even_at < odd_at || n_odd == 0;
    f.offer(even_first ? even_v : odd_v, at + (even_first ? even_at : odd_at));
    if (n_odd > 0) f.offer(even_first ? odd_v : even_v, at + (even_first ? odd_at : even_at));
    f.sum = s + (i64)n_odd * S + ((m & 1) ? y0 : 0);
    if (cur.period == 2) cur.phase ^= (m & 1);
  } else {
    const u32 period = (u32)cur.period, phase = (u32)cur.phase;
    {
      // position l0 + j holds the value of phase (phase + j) mod period
      u32 ph = phase + (u32)lane;
      ph -= (ph / period) * period;
      const u32 step = 32u % period;
      for (int j = lane; j < m; j += 32) {
        buf[l0 + j] = cur.value((int)ph);
        ph += step;
        if (ph >= period) ph -= period;
      }
    }
    if (!kFold) {
      const u32 after = phase + (u32)m;
      cur.phase = (int)(after - (after / period) * period);
      cur.rem -= m;
      return;
    }
    const i64 ya = ev<kRoundFold>(cur.a), yb = ev<kRoundFold>(cur.b), yc = ev<kRoundFold>(cur.c);
    u32 n_b, n_c;
    count_kinds(cur.code, period, phase, (u32)m, &n_b, &n_c);
    const u32 n_a = (u32)m - n_b - n_c;
    u32 per_b, per_c;
    count_kinds(cur.code, period, 0, period, &per_b, &per_c);
    const bool has_a = per_b + per_c < period, has_b = per_b > 0, has_c = per_c > 0;
    const bool all_up = (!has_a || ya > 0) && (!has_b || yb > 0) && (!has_c || yc > 0);
    const bool all_down = (!has_a || ya < 0) && (!has_b || yb < 0) && (!has_c || yc < 0);
    if (all_up || all_down) {
      const i64 total = (i64)n_a * ya + (i64)n_b * yb + (i64)n_c * yc;
      if (all_up) f.offer(f.sum + total, at + m - 1);
      else f.offer(f.sum + ev<kRoundFold>(cur.value((int)phase)), at);
      f.sum += total;
    } else if (m <= 8) {
      int ph = (int)phase;
      for (int j = 0; j < m; ++j) {
        f.sum += ev<kRoundFold>(cur.value(ph));
        f.offer(f.sum, at + j);
        if (++ph == cur.period) ph = 0;
      }
    } else {
      // lane l takes events [l w, l w + w) of the piece
      const int w = (m + 31) >> 5;
      const int lo = lane * w, hi = lo + w < m ? lo + w : m;
      LaneFold part;
      if (lo < hi) {
        u32 ph = phase + (u32)lo;
        ph -= (ph / period) * period;
        for (int j = lo; j < hi; ++j) {
          part.sum += ev<kRoundFold>(cur.value((int)ph));
          part.offer(part.sum, j);
          if (++ph == period) ph = 0;
        }
      }
      SegmentFolder join;
      join.add_lane_folds(part.sum, part.mx, part.ix, part.has, at, lane);
      f.append(join.take());
    }
    u32 ph = phase + (u32)m;
    cur.phase = (int)(ph - (ph / period) * period);
  }
  cur.rem -= m;
}

// Sum of the next m page-rounded events (1 <= m <= rem) of the cursor's run, which are passed
// over without being written; the cursor moves as in emit_piece_by_warp.
template <bool kRoundFold>
__device__ __forceinline__ i64 skip_piece(int m, SpanCursor& cur) {
  i64 sum;
  if (cur.period <= 2) {
    const bool odd = cur.period == 2 && cur.phase;
    const i64 y0 = ev<kRoundFold>(odd ? cur.b : cur.a);
    const i64 y1 = ev<kRoundFold>(cur.period == 2 ? (odd ? cur.a : cur.b) : cur.a);
    sum = (i64)((m + 1) >> 1) * y0 + (i64)(m >> 1) * y1;
    if (cur.period == 2) cur.phase ^= (m & 1);
  } else {
    const u32 period = (u32)cur.period, phase = (u32)cur.phase;
    u32 n_b, n_c;
    count_kinds(cur.code, period, phase, (u32)m, &n_b, &n_c);
    sum = (i64)((u32)m - n_b - n_c) * ev<kRoundFold>(cur.a) + (i64)n_b * ev<kRoundFold>(cur.b) +
          (i64)n_c * ev<kRoundFold>(cur.c);
    const u32 ph = phase + (u32)m;
    cur.phase = (int)(ph - (ph / period) * period);
  }
  cur.rem -= m;
  return sum;
}

}  // namespace llmem
