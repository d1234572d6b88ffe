// llmem_expand_scan: materialise the event list and take its segmented prefix-sum + max
// in one pass.  Each warp builds a 576-event chunk in its own shared memory exactly as
// the expansion kernel does, folds it from shared memory while it is still there, and
// hands it to the TMA engine as one bulk store.  The list is written to HBM once
// (8 bytes per event) and never read back: the scan costs no HBM traffic at all.
#include "llmem_host.h"
#include "expand.cuh"
#include "fold.cuh"
#include "ranges.cuh"

// Launch shape (overridable at compile time for tuning sweeps).  The fold adds arithmetic
// to the expansion, so this kernel wants twice the warps of the plain expansion kernel.
#ifndef LLMEM_FUSED_THREADS
#define LLMEM_FUSED_THREADS 512
#endif
#ifndef LLMEM_FUSED_CTAS_PER_SM
#define LLMEM_FUSED_CTAS_PER_SM 1
#endif

namespace llmem {

constexpr int kFusedThreads = LLMEM_FUSED_THREADS;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kFusedCtasPerSm = LLMEM_FUSED_CTAS_PER_SM;
// What a segment boundary costs this kernel, in events: the kappa of the work split.
#ifndef LLMEM_FUSED_SEGMENT_COST
#define LLMEM_FUSED_SEGMENT_COST 4096
#endif
constexpr i64 kFusedSegmentCost = LLMEM_FUSED_SEGMENT_COST;

// kRoundList: the list is written page-rounded (then the fold takes the values as they
// are); otherwise raw sizes are written and the fold rounds each value as it reads it.
// The peak is always that of the page-rounded list (Section 4.2).
template <bool kRoundList>
__global__ void __launch_bounds__(kFusedThreads)
expand_scan_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets, i64 total,
                   i64* __restrict__ out, i64 n_warps, i64 kappa, int bulk_ok, i64* __restrict__ peak_out,
                   i64* __restrict__ index_out, i64* __restrict__ bounds, WarpPartials* __restrict__ partials) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  ExpandWarpSmem& ws = reinterpret_cast<ExpandWarpSmem*>(smem_raw)[warp];
  const i64 gw = (i64)blockIdx.x * kFusedWarps + warp;
  if (gw >= n_warps) return;
  // this warp's block of chunks: balanced by events + kappa per segment (ranges.cuh)
  i64 seg;  // smallest segment whose end lies beyond the current position; gs/ge its range
  const i64 b_lo = warp_block_start(offsets, n, 0, total, gw, n_warps, kappa, kExpChunk, lane, &seg);
  const i64 b_hi = warp_block_start(offsets, n, 0, total, gw + 1, n_warps, kappa, kExpChunk, lane, nullptr);
  const i64 c_lo = b_lo / kExpChunk, c_hi = (b_hi + kExpChunk - 1) / kExpChunk;
  WarpPartials* my_partials = partials + gw;
  if (lane == 0) {
    my_partials->head = agg_identity();
    my_partials->tail = agg_identity();
    bounds[gw] = b_lo;
    if (gw == n_warps - 1) bounds[n_warps] = total;
  }
  if (c_lo >= c_hi) return;
  i64 gs = seg < n ? __ldg(offsets + seg) : total;
  i64 ge = seg < n ? __ldg(offsets + seg + 1) : total;
  i64 desc_seg = -1;
  const i64 range_lo = c_lo * kExpChunk;  // a segment that starts at or after this started in this warp's range
  SegmentFolder folder;

  int parity = 0;
  for (i64 c = c_lo; c < c_hi; ++c, parity ^= 1) {
    const i64 tb = c * kExpChunk;
    const i64 te = tb + kExpChunk < total ? tb + kExpChunk : total;
    i64* buf = ws.buf[parity];
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
      if (desc_seg != seg) {
        __syncwarp();  // every lane is done with the previous descriptor
        if (lane == 0) build_desc(ws.desc, cfg + seg, gs, ge, kRoundList);
        __syncwarp();
        desc_seg = seg;
      }
      const i64 piece_end = ge < te ? ge : te;
      const i64 e = span_lo > pos ? span_lo : pos;
      const i64 e_end = span_hi < piece_end ? span_hi : piece_end;
      if (e < e_end) {
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
        folder.finish_segment(seg, gs, range_lo, my_partials, peak_out, index_out, lane);
        do {
          ++seg;
          gs = seg < n ? __ldg(offsets + seg) : total;
          ge = seg < n ? __ldg(offsets + seg + 1) : total;
        } while (seg < n && ge <= pos);
      }
    }
    // hand the chunk to the TMA engine (generic-proxy writes -> async-proxy read)
    const u32 cnt = (u32)(te - tb);
    if (bulk_ok) {
      fence_async_shared();
      __syncwarp();
      if (lane == 0) {
        const u32 even = cnt & ~1u;
        if (even) bulk_store(out + tb, buf, even * 8u);
        bulk_commit();
        if (cnt & 1u) out[tb + cnt - 1] = buf[cnt - 1];
      }
    } else {
      __syncwarp();
      for (u32 i = lane; i < cnt; i += 32) out[tb + i] = buf[i];
    }
  }
  // the current segment may continue into the next warp's range
  folder.finish_range(gs, range_lo, my_partials, lane);
  if (lane == 0) bulk_wait_read<0>();
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_expand_scan(const llmem_config* cfg, int64_t n, const int64_t* offsets,
                                          int64_t total_events, int64_t* delta_out, int64_t* peak_out,
                                          int64_t* peak_index_out, void* scratch, size_t scratch_bytes,
                                          uint32_t flags, void* cuda_stream) {
  clear_error();
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
  if (cudaMemsetAsync(scratch, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_expand_scan (memset)");
  i64 warps = 1;
  if (total_events > 0) {
    const size_t smem = sizeof(ExpandWarpSmem) * kFusedWarps;
    static thread_local int configured_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_dev != dev) {
      cudaError_t e1 = cudaFuncSetAttribute(expand_scan_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      cudaError_t e2 = cudaFuncSetAttribute(expand_scan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e1 != cudaSuccess || e2 != cudaSuccess) return check_launch("llmem_expand_scan (shared memory opt-in)");
      configured_dev = dev;
    }
    const i64 nchunks = (total_events + kExpChunk - 1) / kExpChunk;
    warps = (i64)sm_count() * kFusedCtasPerSm * kFusedWarps;
    if (warps > kMaxStreamWarps) warps = kMaxStreamWarps;
    if (warps > nchunks) warps = nchunks;
    const i64 grid = (warps + kFusedWarps - 1) / kFusedWarps;
    const int bulk_ok = aligned_to(delta_out, 16) ? 1 : 0;
    if (flags & LLMEM_FUSE_ROUND)
      expand_scan_kernel<true><<<(unsigned)grid, kFusedThreads, smem, s>>>(
          cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out),
          warps, kFusedSegmentCost, bulk_ok, reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out),
          bounds, partials);
    else
      expand_scan_kernel<false><<<(unsigned)grid, kFusedThreads, smem, s>>>(
          cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out),
          warps, kFusedSegmentCost, bulk_ok, reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out),
          bounds, partials);
    llmem_status st = check_launch("llmem_expand_scan");
    if (st != LLMEM_OK) return st;
  }
  return launch_scan_finish(reinterpret_cast<const i64*>(offsets), n, 0, cfg, reinterpret_cast<i64*>(peak_out),
                            reinterpret_cast<i64*>(peak_index_out), bounds, warps, partials, s);
}
