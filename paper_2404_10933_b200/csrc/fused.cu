// llmem_expand_scan: materialise the event list and take its segmented prefix-sum + max
// in one pass.  Each warp builds a 576-event chunk in its own shared memory exactly as
// the expansion kernel does (or finds that the buffer already holds it), folds it while it
// is there, and hands it to the TMA engine as one bulk store.  The list is written to HBM
// once (8 bytes per event) and never read back: the scan costs no HBM traffic at all.
#include "llmem_host.h"
#include "expand.cuh"
#include "fold.cuh"
#include "ranges.cuh"
#include "spans.cuh"

// Which kernel takes lists of short segments: 1 the one whose segments each have one owner,
// 0 the one that streams chunks of the list with one cursor per warp.
#ifndef LLMEM_SHORT_LISTS_BY_OWNER
#define LLMEM_SHORT_LISTS_BY_OWNER 1
#endif

// Launch shape (overridable at compile time for tuning sweeps): one CTA per SM, 16 warps
// for lists of short segments (a segment boundary is a long single-lane latency, which more
// warps hide), 12 for lists of long ones (fewer, faster streams write slightly faster).
#ifndef LLMEM_FUSED_WARPS_SHORT
#define LLMEM_FUSED_WARPS_SHORT 16
#endif
#ifndef LLMEM_FUSED_WARPS_LONG
#define LLMEM_FUSED_WARPS_LONG 12
#endif
#ifndef LLMEM_FUSED_LONG_SEGMENT
#define LLMEM_FUSED_LONG_SEGMENT 32768
#endif
#ifndef LLMEM_FUSED_CTAS_PER_SM
#define LLMEM_FUSED_CTAS_PER_SM 1
#endif

namespace llmem {

constexpr int kFusedWarpsShort = LLMEM_FUSED_WARPS_SHORT, kFusedWarpsLong = LLMEM_FUSED_WARPS_LONG;
constexpr i64 kFusedLongSegment = LLMEM_FUSED_LONG_SEGMENT;  // mean events per segment from which the list counts as long
constexpr int kFusedCtasPerSm = LLMEM_FUSED_CTAS_PER_SM;
// What a segment boundary costs this kernel, in events: the kappa of the work split.
#ifndef LLMEM_FUSED_SEGMENT_COST
#define LLMEM_FUSED_SEGMENT_COST 4096
#endif
constexpr i64 kFusedSegmentCost = LLMEM_FUSED_SEGMENT_COST;
// Blocks of work per resident warp and the fewest chunks a block is given (ranges.cuh).
#ifndef LLMEM_FUSED_OVERSUB
#define LLMEM_FUSED_OVERSUB 36
#endif
#ifndef LLMEM_FUSED_MIN_CHUNKS
#define LLMEM_FUSED_MIN_CHUNKS 128
#endif

// Descriptor of every configuration, one thread each.  A thread builds its descriptor in
// shared memory; the descriptors of a CTA's configurations are neighbours in the table, so the
// CTA then copies them out together with coalesced 16-byte stores (written by their builders
// one field at a time they would reach device memory as scattered partial lines, and for
// lists of a few hundred events the table is as large as the list).
constexpr int kDescThreads = 128;
__global__ void __launch_bounds__(kDescThreads)
desc_table_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets, int round,
                  SegDesc* __restrict__ table) {
  extern __shared__ __align__(16) unsigned char desc_stage_raw[];
  SegDesc* stage = reinterpret_cast<SegDesc*>(desc_stage_raw);
  const i64 first = (i64)blockIdx.x * kDescThreads, i = first + threadIdx.x;
  if (i < n) build_desc(stage[threadIdx.x], cfg + i, __ldg(offsets + i), __ldg(offsets + i + 1), round != 0);
  __syncthreads();
  const i64 here = n - first < kDescThreads ? n - first : kDescThreads;
  const int4* src = reinterpret_cast<const int4*>(stage);
  int4* dst = reinterpret_cast<int4*>(table + first);
  const int words = (int)here * (int)(sizeof(SegDesc) / 16);
  for (int k = threadIdx.x; k < words; k += kDescThreads) dst[k] = src[k];
}

// Lists whose segments average fewer events than this get 16 warps per CTA and a descriptor
// table; longer ones 12 warps and descriptors built where they are needed.
inline bool long_segments(i64 n, i64 total_events) { return n > 0 && total_events / n >= kFusedLongSegment; }

constexpr size_t kDescTableOffset = (kStreamScratchBytes + 255) / 256 * 256;

size_t expand_scan_scratch_bytes(long long n, long long total_events) {
  if (n <= 0 || total_events <= 0 || long_segments(n, total_events)) return kStreamScratchBytes;
  // a descriptor per configuration, and room to note the segments that a warp writes
  return kDescTableOffset + (size_t)n * (sizeof(SegDesc) + sizeof(i64));
}

// Fold of a full chunk whose events alternate between two values, v0 on even positions and
// v1 on odd ones (constant runs have v0 == v1): with s = v0 + v1 the prefix sums are
// k s + v0 after position 2k and (k + 1) s after position 2k + 1, both linear in k, so the
// largest one sits at an end of one of the two progressions.  Candidates are taken in
// index order and replaced only by strictly larger ones: the first arg max.
__device__ __forceinline__ Agg fold_alternating_chunk(i64 v0, i64 v1, i64 first_index) {
  constexpr i64 kPairs = kExpChunk / 2;
  const i64 s = v0 + v1;
  i64 mx = v0;
  int ix = 0;
  if (s > mx) { mx = s; ix = 1; }
  const i64 even_last = (kPairs - 1) * s + v0;
  if (even_last > mx) { mx = even_last; ix = kExpChunk - 2; }
  const i64 odd_last = kPairs * s;
  if (odd_last > mx) { mx = odd_last; ix = kExpChunk - 1; }
  return Agg{kPairs * s, mx, first_index + ix, 1};
}

// Bulk stores a warp may have in flight from buffers it is not rewriting.
#ifndef LLMEM_FUSED_INFLIGHT
#define LLMEM_FUSED_INFLIGHT 8
#endif
constexpr int kFusedStoresInFlight = LLMEM_FUSED_INFLIGHT;

// kRoundList: the list is written page-rounded (then the fold takes the values as they
// are); otherwise raw sizes are written and the fold rounds each value as it reads it.
// The peak is always that of the page-rounded list (Section 4.2).
//
// Work distribution: the list is cut into n_blocks contiguous blocks of equal cost (events +
// kappa per segment, ranges.cuh), many more than the grid has warps.  Every warp starts on the
// block of its own number and, when done, claims the next unclaimed one from a counter in the
// scratch header.  SMs do not all reach HBM at the same rate: with blocks handed out on
// request the faster ones take more (a pure bulk-store stream writes 6.3 TB/s when every warp
// gets the same share and 7.2-7.6 TB/s when blocks are claimed).
//
// Almost every chunk of a long list lies inside one run of equal (or two alternating)
// events: parameter chunks, gathered chunks, layer outputs.  Such a chunk repeats the one
// written two chunks earlier from the same buffer, so the buffer is not filled again and
// the chunk's fold is taken in closed form; only the bulk store remains.
template <bool kRoundList, int kFusedWarps>
__global__ void __launch_bounds__(kFusedWarps * 32)
expand_scan_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets, i64 total,
                   i64* __restrict__ out, i64 n_blocks, i64 kappa, int bulk_ok, i64* __restrict__ peak_out,
                   i64* __restrict__ index_out, i64* __restrict__ bounds, WarpPartials* __restrict__ partials,
                   unsigned long long* __restrict__ work_counter, const SegDesc* __restrict__ table) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  ExpandWarpSmem& ws = reinterpret_cast<ExpandWarpSmem*>(smem_raw)[warp];
  // the status word is the first word of the scratch header, the work counter sits kWorkCounterOffset into it
  const Guard g{reinterpret_cast<u32*>(reinterpret_cast<unsigned char*>(work_counter) - kWorkCounterOffset), n, total};
  const i64 resident = (i64)gridDim.x * kFusedWarps;
  i64 desc_seg = -1;
  int parity = 0;
  BufferKeys keys;  // what the two chunk buffers hold
  for (i64 gw = (i64)blockIdx.x * kFusedWarps + warp; gw < n_blocks;) {
    i64 seg;  // smallest segment whose end lies beyond the current position; gs/ge its range
    const i64 b_lo = warp_block_start(offsets, n, 0, total, gw, n_blocks, kappa, kExpChunk, lane, &seg);
    const i64 b_hi = warp_block_start(offsets, n, 0, total, gw + 1, n_blocks, kappa, kExpChunk, lane, nullptr);
    const i64 c_lo = b_lo / kExpChunk, c_hi = (b_hi + kExpChunk - 1) / kExpChunk;
    const i64 range_lo = c_lo * kExpChunk;  // a segment that starts at or after this started in this block
    if (!in_bounds(gw >= 0 && gw < kMaxStreamWarps, g, kSiteBlock)) break;
    WarpPartials* my_partials = partials + gw;
    if (lane == 0) {
      my_partials->head = agg_identity();
      my_partials->tail = agg_identity();
      bounds[gw] = b_lo;
      if (gw == n_blocks - 1) bounds[n_blocks] = total;
    }
    i64 gs = seg < n ? __ldg(offsets + seg) : total;
    i64 ge = seg < n ? __ldg(offsets + seg + 1) : total;
    SegmentFolder folder;
    AlternatingRun ar;  // the alternating run the last such chunk lay in

    for (i64 c = c_lo; c < c_hi; ++c, parity ^= 1) {
      const i64 tb = c * kExpChunk;
      const i64 te = tb + kExpChunk < total ? tb + kExpChunk : total;
      i64* buf = ws.buf[parity];
      // a full chunk inside one segment may repeat the one before
      const bool alternating = seg < n && gs <= tb && tb + kExpChunk <= ge &&
                               chunk_alternates(ar, ws, desc_seg, cfg, table, seg, gs, ge, tb, kRoundList, lane, g);
      if (alternating) {
        prepare_alternating<kFusedStoresInFlight>(ar, keys, parity, buf, lane);
        folder.add_uniform(fold_alternating_chunk(ev<!kRoundList>(ar.x0), ev<!kRoundList>(ar.x1), tb), lane);
        if (ge == te) {
          // the segment ends with this chunk: finish it and move to the next non-empty one
          folder.finish_segment(seg, gs, range_lo, my_partials, peak_out, index_out, lane, g);
          do {
            ++seg;
            gs = seg < n ? __ldg(offsets + seg) : total;
            ge = seg < n ? __ldg(offsets + seg + 1) : total;
          } while (seg < n && ge <= te);
        }
      } else {
        keys.set(parity, -1);
        // the bulk store issued from this buffer two chunks ago must have read it
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
        const i64 span_lo = tb + (i64)lane * kExpPerLane;
        const i64 span_hi = span_lo + kExpPerLane < te ? span_lo + kExpPerLane : te;
        i64 pos = tb;
        while (pos < te) {
          if (seg >= n) {
            // offsets do not cover the rest of the chunk: define it as zeros, part of no segment
            for (i64 e = (span_lo > pos ? span_lo : pos); e < span_hi; ++e) buf[e - tb] = 0;
            break;
          }
          ensure_desc(ws, desc_seg, cfg, table, seg, gs, ge, kRoundList, lane, g);
          const i64 piece_end = ge < te ? ge : te;
          const i64 e = span_lo > pos ? span_lo : pos;
          const i64 e_end = span_hi < piece_end ? span_hi : piece_end;
          if (e < e_end && in_bounds(e >= tb && e_end <= tb + kExpChunk, g, kSiteFill)) {
            if (ws.desc.invalid) {
              for (i64 j = e; j < e_end; ++j) buf[j - tb] = 0;
            } else {
              fill_span(buf + (e - tb), ws.desc, (u32)(e - gs), (int)(e_end - e));
            }
          }
          // fold the piece while it sits in shared memory
          if (pos == tb && piece_end == tb + kExpChunk) {
            // the whole chunk belongs to one segment: every lane folds the span it has just written
            const Fold3 f = fold_lane_span<!kRoundList, kExpPerLane>(buf + lane * kExpPerLane);
            folder.add_spans<kExpPerLane>(f, tb, lane);
          } else {
            __syncwarp();  // the piece is read across lanes
            const Agg g = warp_fold_range<!kRoundList>(buf, (int)(pos - tb), (int)(piece_end - tb), lane, tb);
            folder.add_piece(g, lane);
          }
          pos = piece_end;
          if (ge <= te) {
            // the segment ends inside this chunk: finish it and move to the next non-empty one
            folder.finish_segment(seg, gs, range_lo, my_partials, peak_out, index_out, lane, g);
            do {
              ++seg;
              gs = seg < n ? __ldg(offsets + seg) : total;
              ge = seg < n ? __ldg(offsets + seg + 1) : total;
            } while (seg < n && ge <= pos);
          }
        }
        // generic-proxy writes -> async-proxy read
        if (bulk_ok) fence_async_shared();
        __syncwarp();
      }
      store_chunk(out, tb, (u32)(te - tb), buf, bulk_ok, lane, g);
    }
    // the current segment may continue into the next block
    folder.finish_range(gs, range_lo, my_partials, lane);
    // the first `resident` blocks are taken by number, the others in order of request
    unsigned long long ticket = 0;
    if (lane == 0 && n_blocks > resident) ticket = atomicAdd(work_counter, 1ull);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    gw = n_blocks > resident ? resident + (i64)ticket : n_blocks;
  }
  if (lane == 0) bulk_wait_read<0>();
}


// ---------------------------------------------------------------------------
// Lists of short and medium segments: lane-private spans (spans.cuh)
// ---------------------------------------------------------------------------
// How many segments ahead of the current one the descriptors are asked for.
#ifndef LLMEM_SPANS_PREFETCH
#define LLMEM_SPANS_PREFETCH 3
#endif
constexpr int kPrefetchAhead = LLMEM_SPANS_PREFETCH;

struct SpanWarpSmem {
  alignas(128) i64 buf[2][kExpChunk];
  i64 ends[32];  // ends of the 32 segments from the one the chunk begins in
};

// Does the full chunk [tb, tb + kExpChunk), which lies inside segment `seg` (starting at gs),
// consist of one run of period 1 or 2?  Reads the descriptor table; updates `ar` when the
// chunk enters a new such run.
__device__ __forceinline__ bool chunk_alternates_in_table(AlternatingRun& ar, const SegDesc* __restrict__ table,
                                                          i64 seg, i64 gs, i64 tb, const Guard& g) {
  if (tb + kExpChunk <= ar.end) return true;
  if (!in_bounds(seg >= 0 && seg < g.n, g, kSiteDescriptor)) return false;
  const SegDesc* d = table + seg;
  const int4 counts = load_desc_counts(d);
  if (counts.w) return false;
  int r, o, it;
  locate_in_table(d, counts, (u32)(tb - gs), &r, &o, &it);
  const TableRun rn = load_run(d, r);
  if (rn.cnt - o < kExpChunk || rn.period > 2) return false;
  const bool odd = rn.period == 2 && (o & 1);
  ar.x0 = odd ? rn.b : rn.a;
  ar.x1 = rn.period == 2 ? (odd ? rn.a : rn.b) : rn.a;
  ar.end = tb + (rn.cnt - o);
  ar.key = (seg << 8) | (i64)(r << 1) | (odd ? 1 : 0);
  return true;
}

// One element of the segmented scan over the lanes of a chunk: a fold with chunk-local
// position, bit 0 of `fl` = holds events, bit 1 = a segment boundary lies at or before it.
struct SegScan {
  i64 sum, mx;
  int ix, fl;
};

// `o` covers earlier lanes than `x`
__device__ __forceinline__ void seg_scan_join(SegScan& x, const SegScan& o) {
  if (x.fl & 2) return;  // a boundary in between: the earlier events belong to another segment
  if (o.fl & 1) {
    if (x.fl & 1) {
      const i64 cand = o.sum + x.mx;
      const bool take = cand > o.mx;  // ties keep the earlier position
      x.mx = take ? cand : o.mx;
      x.ix = take ? x.ix : o.ix;
      x.sum += o.sum;
    } else {
      x.sum = o.sum;
      x.mx = o.mx;
      x.ix = o.ix;
    }
  }
  x.fl |= o.fl;
}

__device__ __forceinline__ SegScan seg_scan_shfl_up(const SegScan& x, int d) {
  SegScan o;
  o.sum = __shfl_up_sync(0xffffffffu, x.sum, d);
  o.mx = __shfl_up_sync(0xffffffffu, x.mx, d);
  const int packed = __shfl_up_sync(0xffffffffu, (x.ix << 2) | x.fl, d);
  o.ix = packed >> 2;
  o.fl = packed & 3;
  return o;
}

// The same one-pass expansion + scan for lists whose segments are short: all descriptors come
// from the table, and the warp keeps one cursor (the same in every lane) on the run that holds
// the next event to be written.  A chunk is a sequence of pieces, each the part of one run
// that falls into it: the lanes share out the 16-byte stores of a piece, and its fold is
// taken once, in closed form, by every lane alike, so the segment's fold needs no shuffles
// and a segment boundary costs a result store and the first record of the next descriptor.
// Full chunks inside one run of period 1 or 2 repeat the buffer's content as in the kernel
// above.
template <bool kRoundList, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
expand_scan_spans_kernel(i64 n, const i64* __restrict__ offsets, i64 total, i64* __restrict__ out, i64 n_blocks,
                         i64 kappa, int bulk_ok, i64* __restrict__ peak_out, i64* __restrict__ index_out,
                         i64* __restrict__ bounds, WarpPartials* __restrict__ partials,
                         unsigned long long* __restrict__ work_counter, const SegDesc* __restrict__ table) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  SpanWarpSmem& ws = reinterpret_cast<SpanWarpSmem*>(smem_raw)[warp];
  const Guard g{reinterpret_cast<u32*>(reinterpret_cast<unsigned char*>(work_counter) - kWorkCounterOffset), n, total};
  const i64 resident = (i64)gridDim.x * kWarps;
  int parity = 0;
  BufferKeys keys;
  for (i64 gw = (i64)blockIdx.x * kWarps + warp; gw < n_blocks;) {
    i64 seg;  // smallest segment whose end lies beyond the current position; gs/ge its range
    const i64 b_lo = warp_block_start(offsets, n, 0, total, gw, n_blocks, kappa, kExpChunk, lane, &seg);
    const i64 b_hi = warp_block_start(offsets, n, 0, total, gw + 1, n_blocks, kappa, kExpChunk, lane, nullptr);
    const i64 c_lo = b_lo / kExpChunk, c_hi = (b_hi + kExpChunk - 1) / kExpChunk;
    const i64 range_lo = c_lo * kExpChunk;
    if (!in_bounds(gw >= 0 && gw < kMaxStreamWarps, g, kSiteBlock)) break;
    WarpPartials* my_partials = partials + gw;
    if (lane == 0) {
      my_partials->head = agg_identity();
      my_partials->tail = agg_identity();
      bounds[gw] = b_lo;
      if (gw == n_blocks - 1) bounds[n_blocks] = total;
    }
    i64 gs = seg < n ? __ldg(offsets + seg) : total;
    i64 ge = seg < n ? __ldg(offsets + seg + 1) : total;
    WarpFold open;            // the current segment's events seen so far by this block
    SpanCursor cur;           // the run holding the next event
    bool cur_valid = false;   // false: to be positioned on the next event of segment `seg`

    // segment `seg` ends at the current position: store its result (or leave the part seen
    // here to the finishing pass, if the segment began in an earlier block) and move to the
    // next segment that has events
    auto close_segment = [&](i64 pos) {
      if (lane == 0 && in_bounds(seg >= 0 && seg < n, g, kSiteResult)) {
        if (gs >= range_lo) write_raw(seg, open.agg(), gs, peak_out, index_out);
        else my_partials->head = open.agg();
      }
      open = WarpFold();
      do {
        ++seg;
        gs = seg < n ? __ldg(offsets + seg) : total;
        ge = seg < n ? __ldg(offsets + seg + 1) : total;
      } while (seg < n && ge <= pos);
      cur_valid = false;
      prefetch_descriptors(table, seg + kPrefetchAhead, 1, n, lane);
    };
    prefetch_descriptors(table, seg, 1 + kPrefetchAhead, n, lane);

    for (i64 c = c_lo; c < c_hi; ++c, parity ^= 1) {
      const i64 tb = c * kExpChunk;
      const i64 te = tb + kExpChunk < total ? tb + kExpChunk : total;
      i64* buf = ws.buf[parity];
      if (!cur_valid && seg < n) {
        cur.seek(table + seg, (u32)(tb - gs), ge - tb);
        cur_valid = true;
      }
      // a full chunk inside one run of equal or alternating events repeats the buffer's content
      if (seg < n && tb + kExpChunk <= ge && cur.d != nullptr && cur.period <= 2 && cur.rem >= kExpChunk) {
        const bool odd = cur.period == 2 && cur.phase;
        AlternatingRun ar;
        ar.x0 = odd ? cur.b : cur.a;
        ar.x1 = cur.period == 2 ? (odd ? cur.a : cur.b) : cur.a;
        ar.key = (seg << 8) | (i64)(cur.r << 1) | (odd ? 1 : 0);
        prepare_alternating<kFusedStoresInFlight>(ar, keys, parity, buf, lane);
        open.append(fold_alternating_chunk(ev<!kRoundList>(ar.x0), ev<!kRoundList>(ar.x1), tb));
        cur.rem -= kExpChunk;  // an even number of events: the phase stays
        if (ge == te) close_segment(te);
        else if (cur.rem == 0) cur.next_run();
      } else {
        keys.set(parity, -1);
        // the bulk store issued from this buffer two chunks ago must have read it
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
        i64 pos = tb;
        // every round writes at least one event
        while (pos < te) {
          if (seg >= n) {
            // the offsets do not cover the rest of the chunk: zeros, part of no segment
            for (i64 e = pos + lane; e < te; e += 32) buf[e - tb] = 0;
            break;
          }
          if (!cur_valid) {
            cur.start(table + seg, ge - pos);  // a segment begins here
            cur_valid = true;
          }
          const i64 lim = (te < ge ? te : ge) - pos;  // events left in the chunk and in the segment
          int m = cur.rem < lim ? cur.rem : (int)lim;
          if (m < 1) m = 1;  // never reached with consistent descriptors
          if (in_bounds(pos - tb + m <= kExpChunk, g, kSiteFill))
            emit_piece_by_warp<!kRoundList>(buf, (int)(pos - tb), m, cur, open, tb, lane);
          pos += m;
          if (pos >= ge) close_segment(pos);
          else if (cur.rem <= 0) cur.next_run();
        }
        // generic-proxy writes -> async-proxy read
        if (bulk_ok) fence_async_shared();
        __syncwarp();
      }
      store_chunk(out, tb, (u32)(te - tb), buf, bulk_ok, lane, g);
    }
    // the current segment may continue into the next block
    if (lane == 0 && open.has) {
      if (gs >= range_lo) my_partials->tail = open.agg();
      else my_partials->head = open.agg();
    }
    unsigned long long ticket = 0;
    if (lane == 0 && n_blocks > resident) ticket = atomicAdd(work_counter, 1ull);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    gw = n_blocks > resident ? resident + (i64)ticket : n_blocks;
  }
  if (lane == 0) bulk_wait_read<0>();
}


// ---------------------------------------------------------------------------
// Lists of short and medium segments, every segment written by its owner
// ---------------------------------------------------------------------------
// Segments of up to this many events are written by one lane each, longer ones by a warp.
#ifndef LLMEM_OWNED_LANE_MAX
#define LLMEM_OWNED_LANE_MAX 4096
#endif
#ifndef LLMEM_OWNED_WARPS
#define LLMEM_OWNED_WARPS 16
#endif
#ifndef LLMEM_OWNED_CTAS_PER_SM
#define LLMEM_OWNED_CTAS_PER_SM 1
#endif
constexpr i64 kOwnedLaneMax = LLMEM_OWNED_LANE_MAX;
constexpr int kOwnedWarps = LLMEM_OWNED_WARPS, kOwnedCtasPerSm = LLMEM_OWNED_CTAS_PER_SM;
constexpr int kRowStride = kRowEvents + 2;  // 144 bytes: the lanes' rows fall on distinct banks

struct OwnedWarpSmem {
  alignas(16) i64 rows[32][kRowStride];  // lane l stages its next kRowEvents events in rows[l]
  i64 first[32], last[32];               // range of lane l's segment in the list
};

// One-pass expansion + scan in which every segment has one owner.  The warps of a persistent
// grid claim groups of 32 consecutive segments.  Short segments (most of a list of small
// decoders) are written by one lane each: the lane walks its segment's runs with a cursor of
// its own, stages 16 events (one 128-byte line) at a time in its row of shared memory, folds
// them in closed form, and the warp then stores the 32 staged lines with 16-byte stores, eight
// lanes per line, so that device memory sees whole lines although every lane works on a list
// of its own.  There are no segment boundaries to detect, no partial results to join and no
// idle lanes while 32 lists of a few hundred events go by.  Longer segments of the group are
// then written by the whole warp, one after the other, run by run, with coalesced 16-byte
// stores straight to device memory and the fold taken once per run by all lanes alike.
// Results are the bare ones (largest prefix sum, its position): the finishing pass adds
// m_base + lm_p.
template <bool kRoundList, int kWarps>
__global__ void __launch_bounds__(kWarps * 32, kOwnedCtasPerSm)
expand_scan_owned_kernel(i64 n, const i64* __restrict__ offsets, i64 total, i64* __restrict__ out, i64 n_groups,
                         int par /* positions of this parity are 16-byte aligned in `out` */,
                         i64* __restrict__ peak_out, i64* __restrict__ index_out, i64* __restrict__ bounds,
                         unsigned long long* __restrict__ work_counter, const SegDesc* __restrict__ table,
                         unsigned long long* __restrict__ long_count, i64* __restrict__ long_list) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  OwnedWarpSmem& ws = reinterpret_cast<OwnedWarpSmem*>(smem_raw)[warp];
  const Guard g{reinterpret_cast<u32*>(reinterpret_cast<unsigned char*>(work_counter) - kWorkCounterOffset), n, total};
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    // for the finishing pass: one block of work that owns every segment
    bounds[0] = 0;
    bounds[1] = total;
  }
  const i64 resident = (i64)gridDim.x * kWarps;
  for (i64 group = (i64)blockIdx.x * kWarps + warp; group < n_groups;) {
    const i64 seg = group * 32 + lane;
    const bool have = seg < n;
    const i64 gs = have ? __ldg(offsets + seg) : 0, ge = have ? __ldg(offsets + seg + 1) : 0;
    const bool in_list = have && in_bounds(gs >= 0 && ge <= total, g, kSiteStore);
    const i64 count = in_list ? ge - gs : 0;

    // ---- one lane per short segment ----
    const bool mine = count > 0 && count <= kOwnedLaneMax;
    if (__any_sync(0xffffffffu, mine)) {
      // slot 0 of a lane's rows is the last 16-byte aligned position at or before its segment
      const i64 base = gs - ((gs ^ par) & 1);
      ws.first[lane] = mine ? gs : 0;
      ws.last[lane] = mine ? ge : 0;
      SpanCursor cur;
      cur.enter_zeros(0x7fffffff);
      if (mine) cur.start(table + seg, count);
      LaneFold f;
      i64* row = ws.rows[lane];
      __syncwarp();
      for (i64 step = 0; __any_sync(0xffffffffu, mine && base + step * kRowEvents < ge); ++step) {
        const i64 row0 = base + step * kRowEvents;
        // the slots of this row that belong to the segment
        int q = 0, q_end = 0;
        if (mine && row0 < ge) {
          q = row0 < gs ? (int)(gs - row0) : 0;
          q_end = ge - row0 < kRowEvents ? (int)(ge - row0) : kRowEvents;
        }
        const int q_lo = q;
        // every round each lane with slots left emits one piece: the lanes stay together
        while (__any_sync(0xffffffffu, q < q_end)) {
          if (q < q_end) {
            int m = cur.rem < q_end - q ? cur.rem : q_end - q;
            if (m < 1) m = 1;  // never reached with consistent descriptors
            emit_piece<!kRoundList>(row + q, q, (int)(row0 - gs) + q, m, cur, f);
            q += m;
            if (cur.rem <= 0 && row0 + q < ge) cur.next_run();
          }
        }
        const unsigned full = __ballot_sync(0xffffffffu, q_lo == 0 && q_end == kRowEvents);
        const unsigned partial = __ballot_sync(0xffffffffu, q_lo < q_end) & ~full;
        __syncwarp();
        // whole lines: eight lanes store one line, four lines per pass
#pragma unroll
        for (int pass = 0; pass < 8; ++pass) {
          const int r = (lane >> 3) + 4 * pass, vec = lane & 7;
          if ((full >> r) & 1u) {
            const i64 first = ws.first[r];
            const i64 at = first - ((first ^ par) & 1) + step * kRowEvents + 2 * vec;
            *reinterpret_cast<longlong2*>(out + at) = *reinterpret_cast<const longlong2*>(&ws.rows[r][2 * vec]);
          }
        }
        // the first and the last line of a segment: event by event
        for (unsigned todo = partial; todo; todo &= todo - 1) {
          const int r = __ffs(todo) - 1;
          const i64 first = ws.first[r];
          const i64 at = first - ((first ^ par) & 1) + step * kRowEvents + lane;
          if (lane < kRowEvents && at >= first && at < ws.last[r]) out[at] = ws.rows[r][lane];
        }
        __syncwarp();
      }
      if (mine && in_bounds(seg < g.n, g, kSiteResult))
        write_raw(seg, Agg{f.sum, f.mx, gs + f.ix, f.has ? 1 : 0}, gs, peak_out, index_out);
    }

    // ---- longer segments are left to the kernel below: note them ----
    const unsigned wide = __ballot_sync(0xffffffffu, count > kOwnedLaneMax);
    if (wide) {
      unsigned long long slot = 0;
      if (lane == 0) slot = atomicAdd(long_count, (unsigned long long)__popc(wide));
      slot = __shfl_sync(0xffffffffu, slot, 0);
      if ((wide >> lane) & 1u) long_list[slot + __popc(wide & ((1u << lane) - 1))] = seg;
    }

    unsigned long long ticket = 0;
    if (lane == 0 && n_groups > resident) ticket = atomicAdd(work_counter, 1ull);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    group = n_groups > resident ? resident + (i64)ticket : n_groups;
  }
}


// The longer segments of such a list, noted by the kernel above: the warps of a persistent
// grid claim them one at a time and write each run by run with coalesced 16-byte stores
// straight to device memory; the fold of a run is taken once, in closed form, by all lanes
// alike, so a segment costs a few thousand instructions however long it is.
template <bool kRoundList>
__global__ void __launch_bounds__(256)
expand_scan_long_segments_kernel(i64 n, const i64* __restrict__ offsets, i64 total, i64* __restrict__ out, int par,
                                 i64* __restrict__ peak_out, i64* __restrict__ index_out,
                                 const SegDesc* __restrict__ table, const unsigned long long* __restrict__ long_count,
                                 const i64* __restrict__ long_list, unsigned long long* __restrict__ claim_counter,
                                 u32* __restrict__ status_word) {
  const int lane = threadIdx.x & 31;
  const Guard g{status_word, n, total};
  const i64 n_long = (i64)*long_count;
  const i64 resident = ((i64)gridDim.x * blockDim.x) >> 5;
  for (i64 item = ((i64)blockIdx.x * blockDim.x + threadIdx.x) >> 5; item < n_long;) {
    const i64 s = long_list[item];
    if (in_bounds(s >= 0 && s < n, g, kSiteDescriptor)) {
      const i64 s_lo = __ldg(offsets + s), s_hi = __ldg(offsets + s + 1);
      const i64 base = s_lo - ((s_lo ^ par) & 1);  // the last 16-byte aligned position at or before the segment
      i64* dst = out + base;
      SpanCursor cur;
      cur.start(table + s, s_hi - s_lo);
      WarpFold f;
      if (in_bounds(s_lo >= 0 && s_hi <= total, g, kSiteStore)) {
        for (i64 pos = s_lo; pos < s_hi;) {
          const i64 lim = s_hi - pos;
          int m = cur.rem < lim ? cur.rem : (int)lim;
          if (m < 1) m = 1;  // never reached with consistent descriptors
          emit_piece_by_warp<!kRoundList>(dst, (int)(pos - base), m, cur, f, base, lane);
          pos += m;
          if (cur.rem <= 0 && pos < s_hi) cur.next_run();
        }
        if (lane == 0) write_raw(s, f.agg(), s_lo, peak_out, index_out);
      }
    }
    unsigned long long ticket = 0;
    if (lane == 0) ticket = atomicAdd(claim_counter, 1ull);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    item = resident + (i64)ticket;
  }
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_expand_scan(const llmem_config* cfg, int64_t n, const int64_t* offsets,
                                          int64_t total_events, int64_t* delta_out, int64_t* peak_out,
                                          int64_t* peak_index_out, void* scratch, size_t scratch_bytes,
                                          uint32_t flags, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_expand_scan");
  if (n < 0 || total_events < 0) { set_error("llmem_expand_scan: negative size"); return LLMEM_ERR_ARG; }
  if (n == 0) return LLMEM_OK;
  if (!cfg || !offsets || !peak_out || (total_events > 0 && !delta_out)) {
    set_error("llmem_expand_scan: cfg, offsets, delta_out and peak_out are required");
    return LLMEM_ERR_ARG;
  }
  if (!aligned_to(cfg, 16) || !aligned_to(offsets, 8) || !aligned_to(delta_out, 8) || !aligned_to(peak_out, 8) ||
      !aligned_to(peak_index_out, 8)) {
    set_error("llmem_expand_scan: misaligned pointer");
    return LLMEM_ERR_ARG;
  }
  if (!scratch || !aligned_to(scratch, 256) ||
      scratch_bytes < llmem_scratch_bytes(LLMEM_OP_EXPAND_SCAN, n, total_events)) {
    set_error("llmem_expand_scan: scratch missing, misaligned or smaller than llmem_scratch_bytes()");
    return LLMEM_ERR_SCRATCH;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  i64* bounds = reinterpret_cast<i64*>(static_cast<unsigned char*>(scratch) + kBoundsOffset);
  WarpPartials* partials = reinterpret_cast<WarpPartials*>(static_cast<unsigned char*>(scratch) + kPartialsOffset);
  // the header (status word, work counter) starts every call at zero
  unsigned long long* work_counter = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(scratch) + kWorkCounterOffset);
  if (cudaMemsetAsync(scratch, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_expand_scan (memset)");
  i64 warps = 1;
  if (total_events > 0) {
    const i64 nchunks = (total_events + kExpChunk - 1) / kExpChunk;
    const bool long_list = long_segments(n, total_events);
    const int warps_per_cta = long_list ? kFusedWarpsLong : kFusedWarpsShort;
    const bool round = (flags & LLMEM_FUSE_ROUND) != 0;
    const SegDesc* table = nullptr;
    if (!long_list) {
      SegDesc* t = reinterpret_cast<SegDesc*>(static_cast<unsigned char*>(scratch) + kDescTableOffset);
      const size_t stage_bytes = sizeof(SegDesc) * kDescThreads;
      static thread_local int table_dev = -1;
      int cur_dev = 0;
      cudaGetDevice(&cur_dev);
      if (table_dev != cur_dev) {
        if (cudaFuncSetAttribute(desc_table_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes) != cudaSuccess)
          return check_launch("llmem_expand_scan (shared memory opt-in)");
        table_dev = cur_dev;
      }
      desc_table_kernel<<<(unsigned)((n + kDescThreads - 1) / kDescThreads), kDescThreads, stage_bytes, s>>>(
          cfg, n, reinterpret_cast<const i64*>(offsets), round ? 1 : 0, t);
      llmem_status st = check_launch("llmem_expand_scan (descriptor table)");
      if (st != LLMEM_OK) return st;
      table = t;
    }
    const size_t smem = long_list ? sizeof(ExpandWarpSmem) * warps_per_cta : sizeof(SpanWarpSmem) * warps_per_cta;
    static thread_local int configured_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_dev != dev) {
      const int attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
      const int s_long = (int)(sizeof(ExpandWarpSmem) * kFusedWarpsLong);
      const int s_spans = (int)(sizeof(SpanWarpSmem) * kFusedWarpsShort), s_owned = (int)(sizeof(OwnedWarpSmem) * kOwnedWarps);
      if (cudaFuncSetAttribute(expand_scan_owned_kernel<false, kOwnedWarps>, (cudaFuncAttribute)attr, s_owned) != cudaSuccess ||
          cudaFuncSetAttribute(expand_scan_owned_kernel<true, kOwnedWarps>, (cudaFuncAttribute)attr, s_owned) != cudaSuccess)
        return check_launch("llmem_expand_scan (shared memory opt-in)");
      if (cudaFuncSetAttribute(expand_scan_spans_kernel<false, kFusedWarpsShort>, (cudaFuncAttribute)attr, s_spans) != cudaSuccess ||
          cudaFuncSetAttribute(expand_scan_spans_kernel<true, kFusedWarpsShort>, (cudaFuncAttribute)attr, s_spans) != cudaSuccess ||
          cudaFuncSetAttribute(expand_scan_kernel<false, kFusedWarpsLong>, (cudaFuncAttribute)attr, s_long) != cudaSuccess ||
          cudaFuncSetAttribute(expand_scan_kernel<true, kFusedWarpsLong>, (cudaFuncAttribute)attr, s_long) != cudaSuccess)
        return check_launch("llmem_expand_scan (shared memory opt-in)");
      configured_dev = dev;
    }
    const i64 resident = (i64)sm_count() * kFusedCtasPerSm * warps_per_cta;
    // blocks of work: what the finishing pass calls warps
    warps = stream_warps(resident, LLMEM_FUSED_OVERSUB, nchunks, LLMEM_FUSED_MIN_CHUNKS);
    const unsigned grid = (unsigned)(((warps < resident ? warps : resident) + warps_per_cta - 1) / warps_per_cta);
    const int bulk_ok = aligned_to(delta_out, 16) ? 1 : 0;
#define LLMEM_LAUNCH_FUSED(ROUND, WARPS)                                                                        \
  expand_scan_kernel<ROUND, WARPS><<<grid, WARPS * 32, smem, s>>>(                                              \
      cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out), warps,    \
      kFusedSegmentCost, bulk_ok, reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out),      \
      bounds, partials, work_counter, table)
#define LLMEM_LAUNCH_SPANS(ROUND)                                                                               \
  expand_scan_spans_kernel<ROUND, kFusedWarpsShort><<<grid, kFusedWarpsShort * 32, smem, s>>>(                   \
      n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out), warps,          \
      kFusedSegmentCost, bulk_ok, reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out),      \
      bounds, partials, work_counter, table)
    if (long_list) {
      if (round) LLMEM_LAUNCH_FUSED(true, kFusedWarpsLong); else LLMEM_LAUNCH_FUSED(false, kFusedWarpsLong);
    } else if (LLMEM_SHORT_LISTS_BY_OWNER) {
      // every segment written by its owner: groups of 32 segments, claimed by the warps
      const i64 n_groups = (n + 31) / 32;
      const i64 owned_resident = (i64)sm_count() * kOwnedCtasPerSm * kOwnedWarps;
      const unsigned owned_grid = (unsigned)(((n_groups < owned_resident ? n_groups : owned_resident) + kOwnedWarps - 1) / kOwnedWarps);
      const size_t owned_smem = sizeof(OwnedWarpSmem) * kOwnedWarps;
      // positions of parity `par` are 16-byte aligned in the output
      const int par = aligned_to(delta_out, 16) ? 0 : 1;
      unsigned long long* long_count = work_counter + 1;  // three counters side by side in the header
      unsigned long long* long_claims = work_counter + 2;
      i64* long_list = reinterpret_cast<i64*>(static_cast<unsigned char*>(scratch) + kDescTableOffset + (size_t)n * sizeof(SegDesc));
      u32* status_word = static_cast<u32*>(scratch);
      const unsigned long_grid = (unsigned)sm_count() * 8;  // 64 warps per SM
#define LLMEM_LAUNCH_OWNED(ROUND)                                                                               \
  expand_scan_owned_kernel<ROUND, kOwnedWarps><<<owned_grid, kOwnedWarps * 32, owned_smem, s>>>(                 \
      n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out), n_groups, par,   \
      reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), bounds, work_counter, table,      \
      long_count, long_list);                                                                                     \
  expand_scan_long_segments_kernel<ROUND><<<long_grid, 256, 0, s>>>(                                              \
      n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out), par,             \
      reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), table, long_count, long_list,     \
      long_claims, status_word)
      if (round) { LLMEM_LAUNCH_OWNED(true); } else { LLMEM_LAUNCH_OWNED(false); }
#undef LLMEM_LAUNCH_OWNED
      warps = 1;
    } else {
      if (round) LLMEM_LAUNCH_SPANS(true); else LLMEM_LAUNCH_SPANS(false);
    }
#undef LLMEM_LAUNCH_FUSED
#undef LLMEM_LAUNCH_SPANS
    llmem_status st = check_launch("llmem_expand_scan");
    if (st != LLMEM_OK) return st;
  }
  return launch_scan_finish(reinterpret_cast<const i64*>(offsets), n, 0, cfg, reinterpret_cast<i64*>(peak_out),
                            reinterpret_cast<i64*>(peak_index_out), bounds, warps, partials, s);
}
