// llmem_expand_scan: materialise the event list and take its segmented prefix-sum + max
// in one pass: the list is written to HBM once (8 bytes per event) and never read back, the
// scan costs no HBM traffic at all.
//
// Two kernels share the work by the kind of list.  Lists of long segments (deep, wide
// decoders: tens of thousands of events each) are cut into chunks regardless of segment
// boundaries: each warp builds a 576-event chunk in its own shared memory exactly as the
// expansion kernel does (or finds that the buffer already holds it), folds it while it is
// there, and hands it to the TMA engine as one bulk store.  Lists of short and medium
// segments are written by segment owners: a lane for a short segment, a warp for a part of a
// longer one (expand_scan_owned_kernel).
#include "llmem_host.h"
#include "expand.cuh"
#include "fold.cuh"
#include "ranges.cuh"
#include "spans.cuh"

// Launch shape of the chunk kernel (overridable at compile time for tuning sweeps): one CTA
// per SM, 12 warps.  Lists whose segments average at least LLMEM_FUSED_LONG_SEGMENT events go
// to it, the others to the owner kernel.
#ifndef LLMEM_FUSED_WARPS_LONG
#define LLMEM_FUSED_WARPS_LONG 12
#endif
#ifndef LLMEM_FUSED_LONG_SEGMENT
#define LLMEM_FUSED_LONG_SEGMENT 65536
#endif
#ifndef LLMEM_FUSED_CTAS_PER_SM
#define LLMEM_FUSED_CTAS_PER_SM 1
#endif

namespace llmem {

constexpr int kFusedWarpsLong = LLMEM_FUSED_WARPS_LONG;
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

// Segments of up to this many events are written by one lane each; longer ones are cut into
// parts of this many events, each written by a warp.
#ifndef LLMEM_OWNED_LANE_MAX
#define LLMEM_OWNED_LANE_MAX 2048
#endif
#ifndef LLMEM_OWNED_PART
#define LLMEM_OWNED_PART 8192
#endif
constexpr i64 kOwnedLaneMax = LLMEM_OWNED_LANE_MAX, kOwnedPart = LLMEM_OWNED_PART;
static_assert(LLMEM_OWNED_PART % 16 == 0 && LLMEM_OWNED_PART < (1 << 20), "parts: whole lines, part numbers fit 20 bits");

// Scratch of the owner kernel behind the header, block starts and partials of the chunk
// kernels: one descriptor per configuration, then the list of parts (segment << 20 | part
// number, a segment's parts next to each other) and one result per part.
constexpr size_t kDescTableOffset = (kStreamScratchBytes + 255) / 256 * 256;
inline i64 max_parts(i64 n, i64 total_events) { return total_events / kOwnedPart + n + 1; }

// Descriptor of every configuration, one thread each.  A thread builds its descriptor in
// shared memory; the descriptors of a CTA's configurations are neighbours in the table, so the
// CTA then copies them out together with coalesced 16-byte stores (written by their builders
// one field at a time they would reach device memory as scattered partial lines, and for
// lists of a few hundred events the table is as large as the list).  A thread whose segment
// is too long for a lane also enters the segment's parts into the list of parts.
constexpr int kDescThreads = 128;
__global__ void __launch_bounds__(kDescThreads)
desc_table_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets,
                  int round /* bit 0: rounded values, bit 1: second estimator */,
                  SegDesc* __restrict__ table, unsigned long long* __restrict__ part_count,
                  i64* __restrict__ part_list, i64 part_capacity) {
  extern __shared__ __align__(16) unsigned char desc_stage_raw[];
  SegDesc* stage = reinterpret_cast<SegDesc*>(desc_stage_raw);
  const i64 first = (i64)blockIdx.x * kDescThreads, i = first + threadIdx.x;
  i64 count = 0;
  if (i < n) {
    const i64 lo = __ldg(offsets + i), hi = __ldg(offsets + i + 1);
    build_desc(stage[threadIdx.x], cfg + i, lo, hi, (round & 1) != 0, (round & 2) != 0);
    count = hi - lo;
  }
  // the parts of the longer segments: one addition to the counter per warp
  const int lane = threadIdx.x & 31;
  const i64 parts = part_list != nullptr && count > kOwnedLaneMax ? (count + kOwnedPart - 1) / kOwnedPart : 0;
  i64 before = parts;  // parts of this and the lower lanes
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const i64 o = __shfl_up_sync(0xffffffffu, before, d);
    if (lane >= d) before += o;
  }
  const i64 in_warp = __shfl_sync(0xffffffffu, before, 31);
  if (in_warp > 0) {
    unsigned long long slot0 = 0;
    if (lane == 0) slot0 = atomicAdd(part_count, (unsigned long long)in_warp);
    const i64 slot = (i64)__shfl_sync(0xffffffffu, slot0, 0) + before - parts;
    if (parts > 0 && slot + parts <= part_capacity) {  // always, by the size of the scratch
      for (i64 k = 0; k < parts; ++k) part_list[slot + k] = (i << 20) | k;
      stage[threadIdx.x].first_part = slot;
    }
  }
  __syncthreads();
  const i64 here = n - first < kDescThreads ? n - first : kDescThreads;
  const int4* src = reinterpret_cast<const int4*>(stage);
  int4* dst = reinterpret_cast<int4*>(table + first);
  const int words = (int)here * (int)(sizeof(SegDesc) / 16);
  for (int k = threadIdx.x; k < words; k += kDescThreads) dst[k] = src[k];
}

// Lists whose segments average at least this many events go to the chunk kernel, which builds
// descriptors where it needs them; shorter ones get a descriptor table and the owner kernel.
inline bool long_segments(i64 n, i64 total_events) { return n > 0 && total_events / n >= kFusedLongSegment; }

size_t expand_scan_scratch_bytes(long long n, long long total_events) {
  if (n <= 0 || total_events <= 0 || long_segments(n, total_events)) return kStreamScratchBytes;
  // a descriptor per configuration, the list of parts and a result per part
  return kDescTableOffset + (size_t)n * sizeof(SegDesc) +
         (size_t)max_parts(n, total_events) * (sizeof(i64) + sizeof(PartResult));
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
                   unsigned long long* __restrict__ work_counter, int dnn /* 2: the second estimator's list, else 0 */) {
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
                               chunk_alternates(ar, ws, desc_seg, cfg, seg, gs, ge, tb, (kRoundList ? 1 : 0) | dnn, lane, g);
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
          ensure_desc(ws, desc_seg, cfg, seg, gs, ge, (kRoundList ? 1 : 0) | dnn, lane, g);
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
// Lists of short and medium segments, every segment written by its owner
// ---------------------------------------------------------------------------
#ifndef LLMEM_OWNED_WARPS
#define LLMEM_OWNED_WARPS 16
#endif
#ifndef LLMEM_OWNED_CTAS_PER_SM
#define LLMEM_OWNED_CTAS_PER_SM 1
#endif
constexpr int kOwnedWarps = LLMEM_OWNED_WARPS, kOwnedCtasPerSm = LLMEM_OWNED_CTAS_PER_SM;
constexpr int kRowStride = kRowEvents + 2;  // 144 bytes: the lanes' rows fall on distinct banks

struct OwnedWarpSmem {
  alignas(16) i64 rows[32][kRowStride];  // lane l stages its next kRowEvents events in rows[l]
  i64 first[32], last[32];               // range of lane l's segment in the list
};

// One-pass expansion + scan in which every event has one owner that needs nobody else.  The
// warps of a persistent grid claim items of work from one counter: first the groups of 32
// consecutive segments, then the parts of the longer segments (the list of parts the table
// kernel made).
//
// A part (up to 8192 events of one segment) is written by a whole warp, run by run, with
// coalesced 16-byte stores straight to device memory; the fold of a run is taken once, in
// closed form, by all lanes alike, so a part costs a few thousand instructions however many
// events it has.  The prefix sum at which a part begins is the sum of the runs before it,
// taken from their closed forms.  The finishing pass joins the results of a segment's parts.
//
// In a group, the segments short enough for a lane (most of a list of small decoders) are
// written by one lane each: the lane walks its segment's runs with a cursor of its own, stages
// 16 events (one 128-byte line) at a time in its row of shared memory, folds them in closed
// form, and the warp then stores the 32 staged lines with 16-byte stores, eight lanes per
// line, so that device memory sees whole lines although every lane works on a list of its
// own.  There are no segment boundaries to detect, no partial results to join and no idle
// lanes while 32 lists of a few hundred events go by.
//
// Results are the bare ones (largest prefix sum, its position): the finishing pass adds
// m_base + lm_p.
template <bool kRoundList, int kWarps, bool kFold>
__global__ void __launch_bounds__(kWarps * 32, kOwnedCtasPerSm)
expand_scan_owned_kernel(i64 n, const i64* __restrict__ offsets, i64 total, i64* __restrict__ out, i64 n_groups,
                         int par /* positions of this parity are 16-byte aligned in `out` */,
                         i64* __restrict__ peak_out, i64* __restrict__ index_out, i64* __restrict__ bounds,
                         unsigned long long* __restrict__ work_counter, const SegDesc* __restrict__ table,
                         const unsigned long long* __restrict__ part_count, const i64* __restrict__ part_list,
                         PartResult* __restrict__ part_results, i64 part_capacity) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  OwnedWarpSmem& ws = reinterpret_cast<OwnedWarpSmem*>(smem_raw)[warp];
  const Guard g{reinterpret_cast<u32*>(reinterpret_cast<unsigned char*>(work_counter) - kWorkCounterOffset), n, total};
  if (kFold && blockIdx.x == 0 && threadIdx.x == 0) {
    // for the finishing pass: one block of work that owns every segment
    bounds[0] = 0;
    bounds[1] = total;
  }
  i64 n_parts = (i64)*part_count;
  if (n_parts > part_capacity) n_parts = part_capacity;
  // One queue, handed out item by item from the counter in the scratch header: the groups of
  // short segments first (a group of 32 lists written by lanes takes longer than a part
  // written by a warp, so the items that end the kernel are the short ones), then the parts.
  const i64 n_items = n_groups + n_parts;
  for (;;) {
    unsigned long long ticket = 0;
    if (lane == 0) ticket = atomicAdd(work_counter, 1ull);
    const i64 work = (i64)__shfl_sync(0xffffffffu, ticket, 0);
    if (work >= n_items) break;
    const bool on_groups = work < n_groups;
    const i64 item = on_groups ? work : work - n_groups;
    if (!on_groups) {
      // ---- the whole warp for one part of a longer segment ----
      const i64 entry = part_list[item];
      const i64 s = entry >> 20, k = entry & 0xfffff;
      if (in_bounds(s >= 0 && s < n && k <= item, g, kSiteDescriptor)) {
        const i64 s_lo = __ldg(offsets + s), s_hi = __ldg(offsets + s + 1);
        const i64 lo = s_lo + k * kOwnedPart, hi = lo + kOwnedPart < s_hi ? lo + kOwnedPart : s_hi;
        const i64 parts = (s_hi - s_lo + kOwnedPart - 1) / kOwnedPart;
        if (in_bounds(s_lo >= 0 && s_hi <= total && lo < hi, g, kSiteStore)) {
          const i64 base = lo - ((lo ^ par) & 1);  // the last 16-byte aligned position at or before the part
          i64* dst = out + base;
          // the segment's descriptor, copied to shared memory in one go: the runs before the
          // part are walked through at once, and every record read from device memory would
          // be a miss of its own
          SegDesc* desc = reinterpret_cast<SegDesc*>(&ws.rows[0][0]);
          {
            const int4* src = reinterpret_cast<const int4*>(table + s);
            int4* dst = reinterpret_cast<int4*>(desc);
            for (int w = lane; w < (int)(sizeof(SegDesc) / 16); w += 32) dst[w] = __ldg(src + w);
            __syncwarp();
          }
          SpanCursor cur;
          cur.start(desc, s_hi - s_lo);
          WarpFold f;
          // the prefix sum the part begins at: the runs before it, in closed form
          for (i64 pos = s_lo; pos < lo;) {
            const i64 lim = lo - pos;
            int m = cur.rem < lim ? cur.rem : (int)lim;
            if (m < 1) m = 1;  // never reached with consistent descriptors
            const i64 passed = skip_piece<!kRoundList>(m, cur);
            if (kFold) f.sum += passed;
            pos += m;
            if (cur.rem <= 0) cur.next_run();
          }
          for (i64 pos = lo; pos < hi;) {
            const i64 lim = hi - pos;
            int m = cur.rem < lim ? cur.rem : (int)lim;
            if (m < 1) m = 1;
            emit_piece_by_warp<kFold, !kRoundList>(dst, (int)(pos - base), m, cur, f, base, lane);
            pos += m;
            if (cur.rem <= 0 && pos < hi) cur.next_run();
          }
          // a segment of one part has its result; the parts of a longer one are joined by the
          // finishing pass
          if (kFold && lane == 0) {
            if (parts == 1) {
              write_raw(s, f.agg(), s_lo, peak_out, index_out);
            } else {
              PartResult* mine = part_results + item;
              mine->mx = f.mx;
              mine->idx = f.idx;
              mine->has = f.has ? 1u : 0u;
            }
          }
          __syncwarp();  // the copy of the descriptor is done with
        }
      }
    } else {
      // ---- one lane for each short segment of a group ----
      const i64 seg = item * 32 + lane;
      const bool have = seg < n;
      const i64 gs = have ? __ldg(offsets + seg) : 0, ge = have ? __ldg(offsets + seg + 1) : 0;
      const bool in_list = have && in_bounds(gs >= 0 && ge <= total, g, kSiteStore);
      const i64 count = in_list ? ge - gs : 0;
      const bool mine = count > 0 && count <= kOwnedLaneMax;
      if (__any_sync(0xffffffffu, mine)) {
        // slot 0 of a lane's rows is the last 16-byte aligned position at or before its segment
        const i64 base = gs - ((gs ^ par) & 1);
        ws.first[lane] = mine ? gs : 0;
        ws.last[lane] = mine ? ge : 0;
        SpanCursor cur;
        cur.enter_zeros(0x7fffffff);
        if (mine) {
          prefetch_descriptor(table + seg);
          cur.start(table + seg, count);
        }
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
              emit_piece<kFold, !kRoundList>(row + q, q, (int)(row0 - gs) + q, m, cur, f);
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
        if (kFold && mine && in_bounds(seg < g.n, g, kSiteResult))
          write_raw(seg, Agg{f.sum, f.mx, gs + f.ix, f.has ? 1 : 0}, gs, peak_out, index_out);
      }
    }
  }
}


// Host side of the owner kernel: descriptors of all configurations and the list of parts of
// the longer segments (desc_table_kernel), then every segment written by its owner.  `scratch`
// has the layout of llmem_expand_scan's; its header has been cleared by the caller.  With
// `fold` the bare results go to peak_out / index_out and *parts_out tells the finishing pass
// where the parts of the longer segments reported.
llmem_status expand_by_owners(const llmem_config* cfg, i64 n, const i64* offsets, i64 total_events, i64* delta_out,
                              int round_bits, bool fold, i64* peak_out, i64* index_out, void* scratch,
                              PartsOfSegments* parts_out, cudaStream_t s) {
  const bool round = (round_bits & 1) != 0;
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaGetDevice(&dev);
  if (configured_dev != dev) {
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    const int s_owned = (int)(sizeof(OwnedWarpSmem) * kOwnedWarps);
    if (cudaFuncSetAttribute(expand_scan_owned_kernel<false, kOwnedWarps, false>, attr, s_owned) != cudaSuccess ||
        cudaFuncSetAttribute(expand_scan_owned_kernel<true, kOwnedWarps, false>, attr, s_owned) != cudaSuccess ||
        cudaFuncSetAttribute(expand_scan_owned_kernel<false, kOwnedWarps, true>, attr, s_owned) != cudaSuccess ||
        cudaFuncSetAttribute(expand_scan_owned_kernel<true, kOwnedWarps, true>, attr, s_owned) != cudaSuccess ||
        cudaFuncSetAttribute(desc_table_kernel, attr, (int)(sizeof(SegDesc) * kDescThreads)) != cudaSuccess)
      return check_launch("expansion by segment owners (shared memory opt-in)");
    configured_dev = dev;
  }
  unsigned char* base = static_cast<unsigned char*>(scratch) + kDescTableOffset;
  SegDesc* table = reinterpret_cast<SegDesc*>(base);
  const i64 part_capacity = max_parts(n, total_events);
  i64* part_list = reinterpret_cast<i64*>(base + (size_t)n * sizeof(SegDesc));
  PartResult* part_results = reinterpret_cast<PartResult*>(part_list + part_capacity);
  i64* bounds = reinterpret_cast<i64*>(static_cast<unsigned char*>(scratch) + kBoundsOffset);
  unsigned long long* work_counter = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(scratch) + kWorkCounterOffset);
  unsigned long long* part_count = work_counter + 1;  // beside the work counter in the header
  desc_table_kernel<<<(unsigned)((n + kDescThreads - 1) / kDescThreads), kDescThreads, sizeof(SegDesc) * kDescThreads, s>>>(
      cfg, n, offsets, round_bits, table, part_count, part_list, part_capacity);
  llmem_status st = check_launch("expansion by segment owners (descriptor table)");
  if (st != LLMEM_OK) return st;
  const i64 n_groups = (n + 31) / 32;
  // the number of parts is known on the device only: a persistent grid whatever it is
  const unsigned grid = (unsigned)(sm_count() * kOwnedCtasPerSm);
  const size_t smem = sizeof(OwnedWarpSmem) * kOwnedWarps;
  const int par = aligned_to(delta_out, 16) ? 0 : 1;  // positions of this parity are 16-byte aligned
#define LLMEM_LAUNCH_OWNED(ROUND, FOLD)                                                                          \
  expand_scan_owned_kernel<ROUND, kOwnedWarps, FOLD><<<grid, kOwnedWarps * 32, smem, s>>>(                       \
      n, offsets, total_events, delta_out, n_groups, par, peak_out, index_out, bounds, work_counter, table,       \
      part_count, part_list, part_results, part_capacity)
  if (fold) {
    if (round) LLMEM_LAUNCH_OWNED(true, true); else LLMEM_LAUNCH_OWNED(false, true);
  } else {
    if (round) LLMEM_LAUNCH_OWNED(true, false); else LLMEM_LAUNCH_OWNED(false, false);
  }
#undef LLMEM_LAUNCH_OWNED
  st = check_launch("expansion by segment owners");
  if (st != LLMEM_OK) return st;
  if (parts_out) {
    parts_out->first_part = &table->first_part;
    parts_out->stride = sizeof(SegDesc);
    parts_out->results = part_results;
    parts_out->lane_max = kOwnedLaneMax;
    parts_out->part = kOwnedPart;
  }
  return LLMEM_OK;
}

bool short_segment_list(long long n, long long total_events) { return n > 0 && total_events > 0 && !long_segments(n, total_events); }

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
  i64 warps = 1;  // blocks of work the finishing pass has to look at
  PartsOfSegments parts_of_segments;  // segments written in parts, for the finishing pass
  const bool round = (flags & LLMEM_FUSE_ROUND) != 0;
  const int dnn_bit = (flags & LLMEM_ESTIMATOR_DNNMEM) ? 2 : 0;
  if (dnn_bit && !round) {
    // the fold of a list written raw rounds every value to the 2 MiB page while it reads
    set_error("llmem_expand_scan: LLMEM_ESTIMATOR_DNNMEM needs LLMEM_FUSE_ROUND (the list is written aligned to 512 bytes)");
    return LLMEM_ERR_ARG;
  }
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaGetDevice(&dev);
  if (configured_dev != dev) {
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    const int s_long = (int)(sizeof(ExpandWarpSmem) * kFusedWarpsLong);
    if (cudaFuncSetAttribute(expand_scan_kernel<false, kFusedWarpsLong>, attr, s_long) != cudaSuccess ||
        cudaFuncSetAttribute(expand_scan_kernel<true, kFusedWarpsLong>, attr, s_long) != cudaSuccess)
      return check_launch("llmem_expand_scan (shared memory opt-in)");
    configured_dev = dev;
  }
  if (total_events > 0 && long_segments(n, total_events)) {
    // chunks of the list, claimed block by block by the warps of a persistent grid
    const i64 nchunks = (total_events + kExpChunk - 1) / kExpChunk;
    const size_t smem = sizeof(ExpandWarpSmem) * kFusedWarpsLong;
    const i64 resident = (i64)sm_count() * kFusedCtasPerSm * kFusedWarpsLong;
    warps = stream_warps(resident, LLMEM_FUSED_OVERSUB, nchunks, LLMEM_FUSED_MIN_CHUNKS);
    const unsigned grid = (unsigned)(((warps < resident ? warps : resident) + kFusedWarpsLong - 1) / kFusedWarpsLong);
    const int bulk_ok = aligned_to(delta_out, 16) ? 1 : 0;
#define LLMEM_LAUNCH_FUSED(ROUND)                                                                               \
  expand_scan_kernel<ROUND, kFusedWarpsLong><<<grid, kFusedWarpsLong * 32, smem, s>>>(                           \
      cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out), warps,    \
      kFusedSegmentCost, bulk_ok, reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out),      \
      bounds, partials, work_counter, dnn_bit)
    if (round) LLMEM_LAUNCH_FUSED(true); else LLMEM_LAUNCH_FUSED(false);
#undef LLMEM_LAUNCH_FUSED
    llmem_status st = check_launch("llmem_expand_scan");
    if (st != LLMEM_OK) return st;
  } else if (total_events > 0) {
    llmem_status st = expand_by_owners(cfg, n, reinterpret_cast<const i64*>(offsets), total_events,
                                       reinterpret_cast<i64*>(delta_out), (round ? 1 : 0) | dnn_bit, true, reinterpret_cast<i64*>(peak_out),
                                       reinterpret_cast<i64*>(peak_index_out), scratch, &parts_of_segments, s);
    if (st != LLMEM_OK) return st;
  }
  return launch_scan_finish(reinterpret_cast<const i64*>(offsets), n, 0, cfg, reinterpret_cast<i64*>(peak_out),
                            reinterpret_cast<i64*>(peak_index_out), bounds, warps, partials, s, parts_of_segments, dnn_bit != 0);
}
