// llmem_expand_scan: materialise the event list and take its segmented prefix-sum + max
// in one pass.  Each warp builds a 576-event chunk in its own shared memory exactly as
// the expansion kernel does (or finds that the buffer already holds it), folds it while it
// is there, and hands it to the TMA engine as one bulk store.  The list is written to HBM
// once (8 bytes per event) and never read back: the scan costs no HBM traffic at all.
#include "llmem_host.h"
#include "expand.cuh"
#include "fold.cuh"
#include "ranges.cuh"

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

// Descriptor of every configuration, one thread each: on lists of short segments the warps of
// the expansion cross a segment boundary every few chunks, and building the descriptor there
// (one lane, a thousand dependent instructions) is the larger part of what a boundary costs.
__global__ void __launch_bounds__(128)
desc_table_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets, int round,
                  SegDesc* __restrict__ table) {
  const i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) build_desc(table[i], cfg + i, __ldg(offsets + i), __ldg(offsets + i + 1), round != 0);
}

// Lists whose segments average fewer events than this get 16 warps per CTA and a descriptor
// table; longer ones 12 warps and descriptors built where they are needed.
inline bool long_segments(i64 n, i64 total_events) { return n > 0 && total_events / n >= kFusedLongSegment; }

constexpr size_t kDescTableOffset = (kStreamScratchBytes + 255) / 256 * 256;

size_t expand_scan_scratch_bytes(long long n, long long total_events) {
  if (n <= 0 || total_events <= 0 || long_segments(n, total_events)) return kStreamScratchBytes;
  return kDescTableOffset + (size_t)n * sizeof(SegDesc);
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
      desc_table_kernel<<<(unsigned)((n + 127) / 128), 128, 0, s>>>(cfg, n, reinterpret_cast<const i64*>(offsets),
                                                                  round ? 1 : 0, t);
      llmem_status st = check_launch("llmem_expand_scan (descriptor table)");
      if (st != LLMEM_OK) return st;
      table = t;
    }
    const size_t smem = sizeof(ExpandWarpSmem) * warps_per_cta;
    static thread_local int configured_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_dev != dev) {
      const int attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
      const int s_short = (int)(sizeof(ExpandWarpSmem) * kFusedWarpsShort), s_long = (int)(sizeof(ExpandWarpSmem) * kFusedWarpsLong);
      if (cudaFuncSetAttribute(expand_scan_kernel<false, kFusedWarpsShort>, (cudaFuncAttribute)attr, s_short) != cudaSuccess ||
          cudaFuncSetAttribute(expand_scan_kernel<true, kFusedWarpsShort>, (cudaFuncAttribute)attr, s_short) != cudaSuccess ||
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
    if (long_list) {
      if (round) LLMEM_LAUNCH_FUSED(true, kFusedWarpsLong); else LLMEM_LAUNCH_FUSED(false, kFusedWarpsLong);
    } else {
      if (round) LLMEM_LAUNCH_FUSED(true, kFusedWarpsShort); else LLMEM_LAUNCH_FUSED(false, kFusedWarpsShort);
    }
#undef LLMEM_LAUNCH_FUSED
    llmem_status st = check_launch("llmem_expand_scan");
    if (st != LLMEM_OK) return st;
  }
  return launch_scan_finish(reinterpret_cast<const i64*>(offsets), n, 0, cfg, reinterpret_cast<i64*>(peak_out),
                            reinterpret_cast<i64*>(peak_index_out), bounds, warps, partials, s);
}
