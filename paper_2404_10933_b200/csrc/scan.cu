// Segmented prefix-sum + max over materialised event lists (llmem_scan_peak).
//
// Bound by HBM reads (8 bytes per event).  The event array is cut into flat
// 832-event chunks regardless of segment boundaries, so long and short segments
// load every SM equally.  Every warp of the persistent grid owns a contiguous range
// of chunks and streams it on its own: lane 0 keeps two 1-D TMA bulk copies in
// flight into the warp's private ring of shared-memory stages, each completing on
// an mbarrier; each lane reads 26 consecutive events from a landed stage (thirteen
// 16-byte words, an odd count, hence conflict-free), folds them in order, and the
// warp combines with shuffles.  The fold is the associative, non-commutative
// operator on (sum, max prefix, arg max):  (s1,m1) + (s2,m2) = (s1+s2, max(m1, s1+m2)).
// There is no CTA-wide barrier: the warps of an SM drift apart and cover each
// other's latencies.
//
// Segments that end inside a warp's range are finished by that warp.  A segment
// that crosses warp ranges leaves one partial per warp in scratch; a second, tiny
// kernel folds those in order.  No warp ever waits on another warp.  The only waits
// are on the warp's own mbarriers, and they are bounded: on expiry the kernel
// records LLMEM_ERR_TIMEOUT in the scratch status word, drains its own copies and
// returns.
#include "llmem_host.h"
#include "fold.cuh"
#include "ranges.cuh"

namespace llmem {

// Launch shape (overridable at compile time for tuning sweeps).
#ifndef LLMEM_SCAN_THREADS
#define LLMEM_SCAN_THREADS 256
#endif
#ifndef LLMEM_SCAN_PER_LANE
#define LLMEM_SCAN_PER_LANE 26
#endif
#ifndef LLMEM_SCAN_STAGES
#define LLMEM_SCAN_STAGES 2
#endif
constexpr int kScanThreads = LLMEM_SCAN_THREADS;
constexpr int kScanWarps = kScanThreads / 32;
// events per lane: twice an odd number, so that a lane's span is an odd number of
// 16-byte words and the spans of a quarter-warp fall on distinct banks
constexpr int kScanPerLane = LLMEM_SCAN_PER_LANE;
constexpr int kScanChunk = 32 * kScanPerLane;  // 832 events = 6656 bytes: one warp's unit of work
constexpr int kScanStages = LLMEM_SCAN_STAGES;  // chunks in flight per warp
// What a segment boundary costs the scan, in events (piece fold, reduction, result, next
// offsets): the kappa of the cost-balanced work split.
#ifndef LLMEM_SCAN_SEGMENT_COST
#define LLMEM_SCAN_SEGMENT_COST 3072
#endif
constexpr i64 kScanSegmentCost = LLMEM_SCAN_SEGMENT_COST;
// Virtual warps per resident warp and the fewest chunks a virtual warp is given (ranges.cuh).
#ifndef LLMEM_SCAN_OVERSUB
#define LLMEM_SCAN_OVERSUB 1
#endif
#ifndef LLMEM_SCAN_MIN_CHUNKS
#define LLMEM_SCAN_MIN_CHUNKS 64
#endif
static_assert(kScanPerLane % 2 == 0 && (kScanPerLane / 2) % 2 == 1, "per-lane span: odd number of 16-byte words");

// ---- mbarrier / TMA primitives ---------------------------------------------
__device__ __forceinline__ u32 saddr(const void* p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64* bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(saddr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u64* bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}\n" ::"r"(saddr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(u64* bar, u32 bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n" ::"r"(saddr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, u32 parity) {
  u32 ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(saddr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ u64 global_timer_ns() {
  u64 t;
  asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
  return t;
}

constexpr u64 kWaitLimitNs = 2000000000ull;  // 2 s

// Wait for a phase of an mbarrier, giving up after kWaitLimitNs, or at once when
// `abort_flag` (optional) shows that another lane of the warp has given up.  Returns
// false on give-up and raises the flag.
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity, volatile int* abort_flag,
                                                  u64 limit_ns = kWaitLimitNs) {
  // common case: the data has landed, or lands within a few polls (each try_wait
  // already suspends the thread for a hardware-defined interval)
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  // rare case: keep polling against a wall-clock limit
  const u64 t0 = global_timer_ns();
  for (u32 spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if (abort_flag && *abort_flag) return false;
    if ((spin & 63u) == 63u && global_timer_ns() - t0 > limit_ns) {
      if (abort_flag) *abort_flag = 1;
      return false;
    }
  }
}

__device__ __forceinline__ void bulk_load(void* sdst, const void* gsrc, u32 bytes, u64* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(saddr(sdst)),
      "l"(gsrc), "r"(bytes), "r"(saddr(bar))
      : "memory");
}

// One warp's private shared memory.
struct ScanWarpSmem {
  alignas(128) i64 stage[kScanStages][kScanChunk];
  u64 full[kScanStages];
};

// Per-configuration additive offset m_base + lm_p and admissibility.
__device__ __forceinline__ bool segment_offset(const llmem_config* __restrict__ cfg, i64 seg, i64* off, bool dnn) {
  *off = 0;
  if (!cfg) return true;
  Cfg f = load_cfg(cfg + seg);
  if (dnn) {
    // the second estimator adds the CUDA context alone: the lm_head is one of its events
    DnnPlan p;
    u64 peak;
    if (dnn_full_status(f, &p, &peak) != LLMEM_CFG_OK) return false;
    *off = f.base_bytes;
    return true;
  }
  Plan p;
  u64 peak;
  if (full_status(f, &p, &peak) != LLMEM_CFG_OK) return false;
  *off = (i64)p.offset;
  return true;
}

template <bool kRound>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_kernel(const i64* __restrict__ delta_aligned /* 16-byte aligned base */, int shift /* 0 or 1 */,
            const i64* __restrict__ offsets, i64 n, i64 total,
            i64* __restrict__ peak_out, i64* __restrict__ index_out, i64 n_warps, i64 kappa,
            i64* __restrict__ bounds, WarpPartials* __restrict__ partials, u32* __restrict__ status_word) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  ScanWarpSmem& ws = reinterpret_cast<ScanWarpSmem*>(smem_raw)[warp];
  __shared__ int abort_flags[kScanWarps];
  const i64 gw = (i64)blockIdx.x * kScanWarps + warp;
  // virtual indices: event e lives at v = e + shift, so that v even <=> 16-byte aligned
  const i64 v_begin = shift, v_end = (i64)shift + total;
  if (gw >= n_warps) return;
  const Guard guard{status_word, n, total};
  if (!in_bounds(gw < kMaxStreamWarps, guard, kSiteBlock)) return;
  // this warp's block of chunks: balanced by events + kappa per segment (ranges.cuh)
  i64 seg;  // the segment that contains the first event of the current chunk
  const i64 b_lo = warp_block_start(offsets, n, shift, v_end, gw, n_warps, kappa, kScanChunk, lane, &seg);
  const i64 b_hi = warp_block_start(offsets, n, shift, v_end, gw + 1, n_warps, kappa, kScanChunk, lane, nullptr);
  const i64 c_lo = b_lo / kScanChunk, c_hi = (b_hi + kScanChunk - 1) / kScanChunk;
  if (lane == 0) {
    partials[gw].head = agg_identity();
    partials[gw].tail = agg_identity();
    bounds[gw] = b_lo;
    if (gw == n_warps - 1) bounds[n_warps] = v_end;
  }
  if (c_lo >= c_hi) return;
  if (lane == 0) {
    for (int s = 0; s < kScanStages; ++s) mbar_init(&ws.full[s], 1);
    abort_flags[warp] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();
  volatile int* abort_flag = &abort_flags[warp];

  // lane 0: start the copy of chunk c into stage (c - c_lo) % kScanStages
  auto issue = [&](i64 c) {
    const int s = (int)((c - c_lo) % kScanStages);
    const i64 t0 = c * kScanChunk;
    const i64 v_lo = t0 > v_begin ? t0 : v_begin;
    const i64 v_hi = t0 + kScanChunk < v_end ? t0 + kScanChunk : v_end;
    const i64 a_lo = v_lo + (v_lo & 1), a_hi = v_hi - (v_hi & 1);
    i64* dst = ws.stage[s];
    // ragged first / last element (at most one each): plain loads
    if (a_lo > v_lo) dst[v_lo - t0] = delta_aligned[v_lo];
    if (a_hi < v_hi && v_hi - 1 >= a_lo) dst[v_hi - 1 - t0] = delta_aligned[v_hi - 1];
    if (a_hi > a_lo && in_bounds(a_lo >= v_begin && a_hi <= v_end && a_hi - a_lo <= kScanChunk, guard, kSiteLoad)) {
      const u32 bytes = (u32)((a_hi - a_lo) * 8);
      mbar_arrive_expect_tx(&ws.full[s], bytes);
      bulk_load(dst + (a_lo - t0), delta_aligned + a_lo, bytes, &ws.full[s]);
    } else {
      mbar_arrive(&ws.full[s]);
    }
  };
  if (lane == 0)
    for (i64 c = c_lo; c < c_hi && c < c_lo + kScanStages; ++c) issue(c);

  i64 seg_vstart = seg < n ? __ldg(offsets + seg) + shift : v_end;
  i64 seg_vend = seg < n ? __ldg(offsets + seg + 1) + shift : v_end;
  const i64 warp_vlo = c_lo * kScanChunk;  // segments that start at or after this started in this warp's range
  SegmentFolder folder;
  WarpPartials* my_partials = partials + gw;
  i64 consumed = 0;
  bool aborted = false;
  auto next_segment = [&](i64 pos) {
    do {
      ++seg;
      seg_vstart = seg < n ? __ldg(offsets + seg) + shift : v_end;
      seg_vend = seg < n ? __ldg(offsets + seg + 1) + shift : v_end;
    } while (seg < n && seg_vend <= pos);
  };

  for (i64 c = c_lo; c < c_hi; ++c, ++consumed) {
    const int s = (int)(consumed % kScanStages);
    const u32 par = (u32)((consumed / kScanStages) & 1);
    const i64 t0 = c * kScanChunk;
    const i64 v_lo = t0 > v_begin ? t0 : v_begin;
    const i64 v_hi = t0 + kScanChunk < v_end ? t0 + kScanChunk : v_end;
    const bool ok = mbar_wait_bounded(&ws.full[s], par, abort_flag);
    if (!__all_sync(0xffffffffu, ok)) { aborted = true; break; }
    const i64* tile = ws.stage[s];

    if (v_lo == t0 && v_hi == t0 + kScanChunk && seg < n && seg_vend >= v_hi) {
      // ---------- fast path: the whole chunk lies inside one segment ----------
      const Fold3 f = fold_lane_span<kRound, kScanPerLane>(tile + lane * kScanPerLane);
      // every lane has consumed its part of the stage: refill it
      __syncwarp();
      if (lane == 0 && c + kScanStages < c_hi) issue(c + kScanStages);
      folder.add_spans<kScanPerLane>(f, t0, lane);
      if (seg_vend == v_hi) {
        folder.finish_segment(seg, seg_vstart, warp_vlo, my_partials, peak_out, index_out, lane, guard);
        next_segment(v_hi);
      }
      continue;
    }

    // ---------- slow path: segment boundaries inside the chunk, or a ragged chunk ----------
    i64 pos = v_lo;
    while (pos < v_hi && seg < n) {
      const i64 pb = seg_vend < v_hi ? seg_vend : v_hi;
      Agg g = warp_fold_range<kRound>(tile, (int)(pos - t0), (int)(pb - t0), lane, t0);
      folder.add_piece(g, lane);
      pos = pb;
      if (seg_vend <= v_hi) {
        folder.finish_segment(seg, seg_vstart, warp_vlo, my_partials, peak_out, index_out, lane, guard);
        next_segment(pos);
      }
    }
    __syncwarp();
    if (lane == 0 && c + kScanStages < c_hi) issue(c + kScanStages);
  }

  // the current segment may continue into the next warp's range
  if (!aborted) folder.finish_range(seg_vstart, warp_vlo, my_partials, lane);
  if (lane == 0) {
    // drain: every copy that was issued must have landed before the warp exits
    i64 issued = c_hi - c_lo;
    if (issued > consumed + kScanStages) issued = consumed + kScanStages;
    for (i64 k = consumed; k < issued; ++k)
      mbar_wait_bounded(&ws.full[k % kScanStages], (u32)((k / kScanStages) & 1), nullptr);
    if (aborted || *abort_flag) atomicExch(status_word, (u32)LLMEM_ERR_TIMEOUT);
  }
}

// ---------------------------------------------------------------------------
// Lists of short and medium segments: every segment scanned by its owner
// ---------------------------------------------------------------------------
// Segments of up to this many events are scanned by one lane each; longer ones are cut into
// parts of this many events, each scanned by a warp (a lane's staged lines read about 1.6 TB/s
// whatever the length, a warp's bulk copies 3.3 TB/s on 866-event and 6 TB/s on 3 k-event
// segments: the lanes only pay below a few hundred events).
#ifndef LLMEM_SCAN_LANE_MAX
#define LLMEM_SCAN_LANE_MAX 768
#endif
#ifndef LLMEM_SCAN_PART
#define LLMEM_SCAN_PART 4096
#endif
// Lists whose segments average fewer events than this are scanned by owners.
#ifndef LLMEM_SCAN_OWNED_BELOW
#define LLMEM_SCAN_OWNED_BELOW 8192
#endif
constexpr i64 kScanLaneMax = LLMEM_SCAN_LANE_MAX, kScanPart = LLMEM_SCAN_PART, kScanOwnedBelow = LLMEM_SCAN_OWNED_BELOW;
static_assert(LLMEM_SCAN_PART % 2 == 0 && LLMEM_SCAN_PART < (1 << 20), "parts: 16-byte words, part numbers fit 20 bits");

inline bool scan_by_owners(i64 n, i64 total_events) { return n > 0 && total_events > 0 && total_events / n < kScanOwnedBelow; }
inline i64 scan_max_parts(i64 n, i64 total_events) { return total_events / kScanPart + n + 1; }
// behind the header, block starts and partials of the chunk kernel: the first part of every
// segment, the list of parts, one result per part
constexpr size_t kScanPartsOffset = (kStreamScratchBytes + 255) / 256 * 256;

size_t scan_scratch_bytes(long long n, long long total_events) {
  if (!scan_by_owners(n, total_events)) return kStreamScratchBytes;
  return kScanPartsOffset + (size_t)n * sizeof(i64) + (size_t)scan_max_parts(n, total_events) * (sizeof(i64) + sizeof(PartResult));
}

// One thread per segment: a segment too long for a lane enters its parts into the list of
// parts (segment << 20 | part number, a segment's parts next to each other) and notes where
// they start; the others note -1.
__global__ void __launch_bounds__(256)
scan_parts_kernel(const i64* __restrict__ offsets, i64 n, unsigned long long* __restrict__ part_count,
                  i64* __restrict__ part_list, i64* __restrict__ first_part, i64 part_capacity) {
  const i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  const i64 count = i < n ? __ldg(offsets + i + 1) - __ldg(offsets + i) : 0;
  const i64 parts = count > kScanLaneMax ? (count + kScanPart - 1) / kScanPart : 0;
  i64 before = parts;  // parts of this and the lower lanes
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const i64 o = __shfl_up_sync(0xffffffffu, before, d);
    if (lane >= d) before += o;
  }
  const i64 in_warp = __shfl_sync(0xffffffffu, before, 31);
  i64 slot = -1;
  if (in_warp > 0) {
    unsigned long long slot0 = 0;
    if (lane == 0) slot0 = atomicAdd(part_count, (unsigned long long)in_warp);
    const i64 mine = (i64)__shfl_sync(0xffffffffu, slot0, 0) + before - parts;
    if (parts > 0 && mine + parts <= part_capacity) {  // always, by the size of the scratch
      for (i64 k = 0; k < parts; ++k) part_list[mine + k] = (i << 20) | k;
      slot = mine;
    }
  }
  if (i < n) first_part[i] = slot;
}

// Segmented prefix-sum + max for lists of short and medium segments.  The warps of a persistent
// grid claim items from one counter: first the groups of 32 consecutive segments, then the
// parts of the longer segments.  In a group every segment of up to 768 events is scanned by one
// lane: each step the warp brings the next 128-byte line of all 32 segments into shared memory
// (eight lanes per line: 16-byte loads from 32 different lines in one instruction reach a
// fifth of the bandwidth) and every lane folds its own line in order: no segment boundaries
// to find in a chunk, no pieces to join.  A part is streamed by the whole
// warp through the same two-stage ring of TMA bulk copies as in the kernel above, each lane
// folding 26 consecutive events of a landed chunk; since a part lies inside one segment there
// is only the fast path.  The finishing pass joins the parts of a segment in order.
constexpr int kScanRowEvents = 16;                  // events a lane takes per step: one 128-byte line
constexpr int kScanRowStride = kScanRowEvents + 2;  // 144 bytes: the lanes' rows fall on distinct banks
static_assert(32 * kScanRowStride <= kScanChunk && 64 <= kScanChunk, "rows and segment ranges fit the stages");

#ifndef LLMEM_SCAN_OWNED_WARPS
#define LLMEM_SCAN_OWNED_WARPS 16
#endif
constexpr int kScanOwnedWarps = LLMEM_SCAN_OWNED_WARPS;

template <bool kRound>
__global__ void __launch_bounds__(kScanOwnedWarps * 32, 1)
scan_owned_kernel(const i64* __restrict__ delta_aligned, int shift, const i64* __restrict__ offsets, i64 n, i64 total,
                  i64* __restrict__ peak_out, i64* __restrict__ index_out, i64 n_groups,
                  unsigned long long* __restrict__ work_counter, const unsigned long long* __restrict__ part_count,
                  const i64* __restrict__ part_list, PartResult* __restrict__ part_results, i64 part_capacity,
                  i64* __restrict__ bounds, u32* __restrict__ status_word) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  ScanWarpSmem& ws = reinterpret_cast<ScanWarpSmem*>(smem_raw)[warp];
  __shared__ int abort_flags[kScanOwnedWarps];
  const Guard guard{status_word, n, total};
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    // for the finishing pass: one block of work that owns every segment
    bounds[0] = shift;
    bounds[1] = (i64)shift + total;
  }
  if (lane == 0) {
    for (int s = 0; s < kScanStages; ++s) mbar_init(&ws.full[s], 1);
    abort_flags[warp] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();
  volatile int* abort_flag = &abort_flags[warp];
  u32 phase_bits = 0;  // parity of each stage's next completion
  bool aborted = false;
  i64 n_parts = (i64)*part_count;
  if (n_parts > part_capacity) n_parts = part_capacity;
  // groups first, item by item from the counter (see expand_scan_owned_kernel)
  const i64 n_items = n_groups + n_parts;
  while (!aborted) {
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
      if (in_bounds(s >= 0 && s < n && k <= item, guard, kSiteDescriptor)) {
        const i64 s_lo = __ldg(offsets + s) + shift, s_hi = __ldg(offsets + s + 1) + shift;  // virtual positions
        const i64 lo = s_lo + k * kScanPart, hi = lo + kScanPart < s_hi ? lo + kScanPart : s_hi;
        const i64 parts = (s_hi - s_lo + kScanPart - 1) / kScanPart;
        if (in_bounds(s_lo >= shift && s_hi <= (i64)shift + total && lo < hi, guard, kSiteLoad)) {
          // chunks of the part, from an even position so that the copies start on 16-byte boundaries
          const i64 c0 = lo & ~(i64)1;
          const i64 n_chunks = (hi - c0 + kScanChunk - 1) / kScanChunk;
          auto issue = [&](i64 c) {
            const int st = (int)(c % kScanStages);
            const i64 t0 = c0 + c * kScanChunk;
            const i64 v_lo = t0 > lo ? t0 : lo, v_hi = t0 + kScanChunk < hi ? t0 + kScanChunk : hi;
            const i64 a_lo = v_lo + (v_lo & 1), a_hi = v_hi - (v_hi & 1);
            i64* dst = ws.stage[st];
            if (a_lo > v_lo) dst[v_lo - t0] = delta_aligned[v_lo];
            if (a_hi < v_hi && v_hi - 1 >= a_lo) dst[v_hi - 1 - t0] = delta_aligned[v_hi - 1];
            if (a_hi > a_lo) {
              const u32 bytes = (u32)((a_hi - a_lo) * 8);
              mbar_arrive_expect_tx(&ws.full[st], bytes);
              bulk_load(dst + (a_lo - t0), delta_aligned + a_lo, bytes, &ws.full[st]);
            } else {
              mbar_arrive(&ws.full[st]);
            }
          };
          if (lane == 0)
            for (i64 c = 0; c < n_chunks && c < kScanStages; ++c) issue(c);
          SegmentFolder folder;
          i64 consumed = 0;
          for (i64 c = 0; c < n_chunks; ++c, ++consumed) {
            const int st = (int)(c % kScanStages);
            const bool ok = mbar_wait_bounded(&ws.full[st], (phase_bits >> st) & 1u, abort_flag);
            phase_bits ^= 1u << st;
            if (!__all_sync(0xffffffffu, ok)) { aborted = true; break; }
            const i64* tile = ws.stage[st];
            const i64 t0 = c0 + c * kScanChunk;
            const i64 v_lo = t0 > lo ? t0 : lo, v_hi = t0 + kScanChunk < hi ? t0 + kScanChunk : hi;
            if (v_lo == t0 && v_hi == t0 + kScanChunk) {
              const Fold3 f = fold_lane_span<kRound, kScanPerLane>(tile + lane * kScanPerLane);
              __syncwarp();  // every lane has consumed its part of the stage: refill it
              if (lane == 0 && c + kScanStages < n_chunks) issue(c + kScanStages);
              folder.add_spans<kScanPerLane>(f, t0, lane);
            } else {
              const Agg g = warp_fold_range<kRound>(tile, (int)(v_lo - t0), (int)(v_hi - t0), lane, t0);
              folder.add_piece(g, lane);
              __syncwarp();
              if (lane == 0 && c + kScanStages < n_chunks) issue(c + kScanStages);
            }
          }
          if (aborted) {
            // drain: every copy that was issued must have landed before the warp goes on or exits
            if (lane == 0) {
              i64 issued = n_chunks < consumed + kScanStages ? n_chunks : consumed + kScanStages;
              for (i64 c = consumed; c < issued; ++c) {
                const int st = (int)(c % kScanStages);
                mbar_wait_bounded(&ws.full[st], (phase_bits >> st) & 1u, nullptr);
              }
            }
          } else {
            const Agg whole = folder.take();
            if (lane == 0) {
              if (parts == 1) {
                write_raw(s, whole, s_lo, peak_out, index_out);
              } else {
                PartResult* mine = part_results + item;
                mine->sum = whole.sum;
                mine->mx = whole.mx;
                mine->idx = whole.idx;
                mine->has = whole.valid;
              }
            }
          }
        }
      }
    } else {
      // ---- one lane for each short segment of a group ----
      const i64 seg = item * 32 + lane;
      const bool have = seg < n;
      const i64 gs = have ? __ldg(offsets + seg) + shift : 0, ge = have ? __ldg(offsets + seg + 1) + shift : 0;
      const bool mine = have && ge > gs && ge - gs <= kScanLaneMax &&
                        in_bounds(gs >= shift && ge <= (i64)shift + total, guard, kSiteLoad);
      if (__any_sync(0xffffffffu, mine)) {
        // Rows of 16 events (one 128-byte line), one per lane, in the warp's first stage; the
        // ranges of the lanes' segments in its second.  A step brings the next line of every
        // segment in with 16-byte loads, eight lanes per line, so that device memory is read in
        // whole lines although every lane then folds a list of its own.
        i64(*rows)[kScanRowStride] = reinterpret_cast<i64(*)[kScanRowStride]>(ws.stage[0]);
        i64* first = ws.stage[1];
        i64* last = ws.stage[1] + 32;
        const i64 base = gs & ~(i64)1;  // slot 0 of a lane's rows: the last even position at or before its segment
        first[lane] = mine ? gs : 0;
        last[lane] = mine ? ge : 0;
        __syncwarp();
        i64 sum = 0, mx = 0, idx = -1;
        bool has = false;
        // The lines of the next step are requested before the rows of this one are folded, so
        // that the loads are in flight during the fold.
        longlong2 x[8];
        auto fetch = [&](i64 step) {
#pragma unroll
          for (int pass = 0; pass < 8; ++pass) {
            const int r = (lane >> 3) + 4 * pass, vec = lane & 7;
            const i64 lo_r = first[r], hi_r = last[r];
            const i64 at = (lo_r & ~(i64)1) + step * kScanRowEvents + 2 * vec;
            x[pass] = make_longlong2(0, 0);
            if (at >= lo_r && at + 1 < hi_r) {
              x[pass] = __ldg(reinterpret_cast<const longlong2*>(delta_aligned + at));
            } else {
              if (at >= lo_r && at < hi_r) x[pass].x = __ldg(delta_aligned + at);
              if (at + 1 >= lo_r && at + 1 < hi_r) x[pass].y = __ldg(delta_aligned + at + 1);
            }
          }
        };
        bool more = true;  // the group has a segment with events: step 0 exists
        fetch(0);
        for (i64 step = 0; more; ++step) {
#pragma unroll
          for (int pass = 0; pass < 8; ++pass)
            *reinterpret_cast<longlong2*>(&rows[(lane >> 3) + 4 * pass][2 * (lane & 7)]) = x[pass];
          __syncwarp();
          more = __any_sync(0xffffffffu, mine && base + (step + 1) * kScanRowEvents < ge);
          if (more) fetch(step + 1);
          const i64 row0 = base + step * kScanRowEvents;
          if (mine && row0 < ge) {
            const int q_lo = row0 < gs ? (int)(gs - row0) : 0;
            const int q_end = ge - row0 < kScanRowEvents ? (int)(ge - row0) : kScanRowEvents;
            const i64* row = rows[lane];
            for (int q = q_lo; q < q_end; ++q) {
              sum += ev<kRound>(row[q]);
              if (!has || sum > mx) { mx = sum; idx = row0 + q; has = true; }
            }
          }
          __syncwarp();
        }
        if (mine && in_bounds(seg < guard.n, guard, kSiteResult))
          write_raw(seg, Agg{sum, mx, idx, has ? 1 : 0}, gs, peak_out, index_out);
      }
    }
  }
  if (lane == 0 && (aborted || *abort_flag)) atomicExch(status_word, (u32)LLMEM_ERR_TIMEOUT);
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever
// complete, with the given limit; the wait must give up and the warp records
// LLMEM_ERR_TIMEOUT exactly as the scan kernel would.  Nothing else is touched.
__global__ void __launch_bounds__(32)
wait_limit_selftest_kernel(u32* __restrict__ status_word, u64 limit_ns) {
  __shared__ u64 bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait_bounded(&bar, 0, &abort_flag, limit_ns);
  if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0) atomicExch(status_word, (u32)LLMEM_ERR_TIMEOUT);
}

// Warp whose block [bounds[j], bounds[j+1]) contains event index v: the largest j with
// bounds[j] <= v (blocks may be empty, then several share a start and the last one owns it).
__device__ __forceinline__ i64 owner_of(const i64* __restrict__ bounds, i64 n_warps, i64 v) {
  i64 lo = 0, hi = n_warps - 1;
  while (lo < hi) {
    const i64 mid = lo + (hi - lo + 1) / 2;
    if (__ldg(bounds + mid) <= v) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

// Finish, one thread per segment: fold the partials of segments that cross warp
// ranges, define empty segments, add m_base + lm_p, and mark inadmissible
// configurations.
__global__ void __launch_bounds__(256)
scan_finish_kernel(const i64* __restrict__ offsets, i64 n, int shift, const llmem_config* __restrict__ cfg,
                   i64* __restrict__ peak_out, i64* __restrict__ index_out, const i64* __restrict__ bounds,
                   i64 n_warps, const WarpPartials* __restrict__ partials, PartsOfSegments parts, bool dnn) {
  for (i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (i64)gridDim.x * blockDim.x) {
    const i64 a = offsets[i] + shift, b = offsets[i + 1] + shift;
    i64 mx = 0, idx = -1;
    if (b > a) {
      const i64 ca = owner_of(bounds, n_warps, a), cb = owner_of(bounds, n_warps, b - 1);
      const i64 n_parts = parts.first_part != nullptr && b - a > parts.lane_max ? (b - a + parts.part - 1) / parts.part : 1;
      if (n_parts > 1) {
        // written in parts: theirs are prefix sums from the segment's start, so the first of the
        // largest is the segment's
        const i64 first = *reinterpret_cast<const i64*>(reinterpret_cast<const unsigned char*>(parts.first_part) + (size_t)i * parts.stride);
        bool has = false;
        i64 before = 0;  // sum of the parts already joined
        for (i64 j = 0; j < n_parts && first >= 0; ++j) {
          const PartResult r = parts.results[first + j];
          const i64 base = parts.relative ? before : 0;
          if (r.has && (!has || base + r.mx > mx)) {
            mx = base + r.mx;
            idx = r.idx - a;
            has = true;
          }
          before += r.sum;
        }
      } else if (ca == cb) {  // finished by the warp that owns it
        mx = peak_out[i];
        if (index_out) idx = index_out[i];
      } else {
        Agg g = partials[ca].tail;
        for (i64 c = ca + 1; c <= cb; ++c) g = agg_fold(g, partials[c].head);
        mx = g.valid ? g.mx : 0;
        idx = g.valid ? g.idx - a : -1;
      }
    }
    i64 off;
    const bool ok = segment_offset(cfg, i, &off, dnn);
    peak_out[i] = ok ? off + mx : -1;
    if (index_out) index_out[i] = ok ? idx : -1;
  }
}

llmem_status launch_scan_finish(const i64* offsets, i64 n, int shift, const llmem_config* cfg, i64* peak_out,
                                i64* index_out, const i64* bounds, i64 n_warps, const WarpPartials* partials,
                                cudaStream_t stream, PartsOfSegments parts, bool dnn) {
  i64 blocks = (n + 255) / 256;
  const i64 cap = (i64)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  scan_finish_kernel<<<(unsigned)blocks, 256, 0, stream>>>(offsets, n, shift, cfg, peak_out, index_out, bounds,
                                                          n_warps < 1 ? 1 : n_warps, partials, parts, dnn);
  return check_launch("llmem_scan_peak (finish)");
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_scan_peak(const int64_t* delta, const int64_t* offsets, int64_t n,
                                        int64_t total_events, const llmem_config* cfg,
                                        int64_t* peak_out, int64_t* peak_index_out, void* scratch,
                                        size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_scan_peak");
  if (n < 0 || total_events < 0) { set_error("llmem_scan_peak: negative size"); return LLMEM_ERR_ARG; }
  if (n == 0) return LLMEM_OK;
  if (!offsets || !peak_out || (total_events > 0 && !delta)) {
    set_error("llmem_scan_peak: delta, offsets and peak_out are required");
    return LLMEM_ERR_ARG;
  }
  if (!aligned_to(delta, 8) || !aligned_to(offsets, 8) || !aligned_to(peak_out, 8) ||
      !aligned_to(peak_index_out, 8) || !aligned_to(cfg, 16)) {
    set_error("llmem_scan_peak: misaligned pointer");
    return LLMEM_ERR_ARG;
  }
  if (!scratch || !aligned_to(scratch, 256) ||
      scratch_bytes < llmem_scratch_bytes(LLMEM_OP_SCAN_PEAK, n, total_events)) {
    set_error("llmem_scan_peak: scratch missing, misaligned or smaller than llmem_scratch_bytes()");
    return LLMEM_ERR_SCRATCH;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  u32* status_word = static_cast<u32*>(scratch);
  i64* bounds = reinterpret_cast<i64*>(static_cast<unsigned char*>(scratch) + kBoundsOffset);
  WarpPartials* partials = reinterpret_cast<WarpPartials*>(static_cast<unsigned char*>(scratch) + kPartialsOffset);
  if (cudaMemsetAsync(status_word, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_scan_peak (memset)");

  const int shift = aligned_to(delta, 16) ? 0 : 1;
  const i64* delta_aligned = reinterpret_cast<const i64*>(delta) - shift;
  const bool round = (flags & LLMEM_FUSE_ROUND) != 0;
  const bool dnn = (flags & LLMEM_ESTIMATOR_DNNMEM) != 0;
  if (dnn && round) {
    set_error("llmem_scan_peak: LLMEM_FUSE_ROUND rounds to the 2 MiB page; lists of the second estimator are written aligned");
    return LLMEM_ERR_ARG;
  }
  i64 warps = 1;
  PartsOfSegments parts_of_segments;
  if (scan_by_owners(n, total_events)) {
    // lists of short and medium segments: every segment scanned by its owner
    const size_t smem = sizeof(ScanWarpSmem) * kScanOwnedWarps;
    static thread_local int owned_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (owned_dev != dev) {
      cudaError_t e1 = cudaFuncSetAttribute(scan_owned_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      cudaError_t e2 = cudaFuncSetAttribute(scan_owned_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e1 != cudaSuccess || e2 != cudaSuccess) return check_launch("llmem_scan_peak (shared memory opt-in)");
      owned_dev = dev;
    }
    unsigned char* base = static_cast<unsigned char*>(scratch) + kScanPartsOffset;
    i64* first_part = reinterpret_cast<i64*>(base);
    const i64 part_capacity = scan_max_parts(n, total_events);
    i64* part_list = first_part + n;
    PartResult* part_results = reinterpret_cast<PartResult*>(part_list + part_capacity);
    unsigned long long* work_counter = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(scratch) + kWorkCounterOffset);
    unsigned long long* part_count = work_counter + 1;
    scan_parts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(reinterpret_cast<const i64*>(offsets), n, part_count, part_list,
                                                                 first_part, part_capacity);
    llmem_status st = check_launch("llmem_scan_peak (parts)");
    if (st != LLMEM_OK) return st;
    const i64 n_groups = (n + 31) / 32;
    const unsigned grid = (unsigned)sm_count();
    if (round)
      scan_owned_kernel<true><<<grid, kScanOwnedWarps * 32, smem, s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events, reinterpret_cast<i64*>(peak_out),
          reinterpret_cast<i64*>(peak_index_out), n_groups, work_counter, part_count, part_list, part_results, part_capacity,
          bounds, status_word);
    else
      scan_owned_kernel<false><<<grid, kScanOwnedWarps * 32, smem, s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events, reinterpret_cast<i64*>(peak_out),
          reinterpret_cast<i64*>(peak_index_out), n_groups, work_counter, part_count, part_list, part_results, part_capacity,
          bounds, status_word);
    st = check_launch("llmem_scan_peak");
    if (st != LLMEM_OK) return st;
    parts_of_segments.first_part = first_part;
    parts_of_segments.stride = sizeof(i64);
    parts_of_segments.results = part_results;
    parts_of_segments.lane_max = kScanLaneMax;
    parts_of_segments.part = kScanPart;
    parts_of_segments.relative = true;
  } else if (total_events > 0) {
    const size_t smem = sizeof(ScanWarpSmem) * kScanWarps;
    static thread_local int configured_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_dev != dev) {
      cudaError_t e1 = cudaFuncSetAttribute(scan_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      cudaError_t e2 = cudaFuncSetAttribute(scan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e1 != cudaSuccess || e2 != cudaSuccess) return check_launch("llmem_scan_peak (shared memory opt-in)");
      configured_dev = dev;
    }
    const i64 nchunks = (total_events + shift + kScanChunk - 1) / kScanChunk;
    warps = stream_warps((i64)sm_count() * kScanWarps, LLMEM_SCAN_OVERSUB, nchunks, LLMEM_SCAN_MIN_CHUNKS);
    const i64 grid = (warps + kScanWarps - 1) / kScanWarps;
    if (round)
      scan_kernel<true><<<(unsigned)grid, kScanThreads, smem, s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events,
          reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), warps, kScanSegmentCost, bounds,
          partials, status_word);
    else
      scan_kernel<false><<<(unsigned)grid, kScanThreads, smem, s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events,
          reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), warps, kScanSegmentCost, bounds,
          partials, status_word);
    llmem_status st = check_launch("llmem_scan_peak");
    if (st != LLMEM_OK) return st;
  }
  return launch_scan_finish(reinterpret_cast<const i64*>(offsets), n, shift, cfg, reinterpret_cast<i64*>(peak_out),
                            reinterpret_cast<i64*>(peak_index_out), bounds, warps, partials, s, parts_of_segments, dnn);
}

extern "C" llmem_status llmem_selftest_wait_limit(void* scratch, size_t scratch_bytes, uint32_t limit_ms,
                                                  void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_selftest_wait_limit");
  if (!scratch || !aligned_to(scratch, 256) || scratch_bytes < kScratchHeader) {
    set_error("llmem_selftest_wait_limit: scratch of at least 256 bytes, 256-byte aligned, is required");
    return LLMEM_ERR_SCRATCH;
  }
  if (limit_ms < 1 || limit_ms > 2000) {
    set_error("llmem_selftest_wait_limit: limit_ms must be in 1 .. 2000");
    return LLMEM_ERR_ARG;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(scratch, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_selftest_wait_limit (memset)");
  wait_limit_selftest_kernel<<<1, 32, 0, s>>>(static_cast<u32*>(scratch), (u64)limit_ms * 1000000ull);
  return check_launch("llmem_selftest_wait_limit");
}
