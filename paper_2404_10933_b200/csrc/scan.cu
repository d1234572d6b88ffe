// Segmented prefix-sum + max over materialised event lists (llmem_scan_peak).
//
// Bound by HBM reads (8 bytes per event).  The event array is cut into flat tiles
// regardless of segment boundaries, so long and short segments load every SM
// equally.  Each persistent CTA owns a contiguous range of tiles.  A producer lane
// streams tiles into a ring of shared-memory stages with 1-D TMA bulk copies
// completing on mbarriers; 256 consumer threads each read 18 consecutive events
// from the stage (nine 16-byte words, an odd count, hence conflict-free), fold them
// in order, and combine across the warp with shuffles and across warps through
// shared memory.  The fold is the associative, non-commutative operator on
// (sum, max prefix, arg max):  (s1,m1) + (s2,m2) = (s1+s2, max(m1, s1+m2)).
//
// Segments that end inside a CTA's range are finished by that CTA.  A segment that
// crosses CTA ranges leaves one partial per CTA in scratch; a second, tiny kernel
// folds those in order.  No CTA ever waits on another CTA.  The only waits are on
// the CTA's own mbarriers, and they are bounded: on expiry the kernel records
// LLMEM_ERR_TIMEOUT in the scratch status word, drains its own copies and returns.
#include "llmem_host.h"
#include "llmem_model.cuh"

namespace llmem {

constexpr int kScanConsumers = 256;
constexpr int kScanWarps = kScanConsumers / 32;
constexpr int kScanThreads = kScanConsumers + 32;  // + one producer warp
constexpr int kScanPerThread = 18;
constexpr int kScanTile = kScanConsumers * kScanPerThread;  // 4608 events = 36 KiB
constexpr int kScanStages = 4;

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

// Wait for a phase of an mbarrier, giving up after kWaitLimitNs or when another
// thread of the CTA has given up.  Returns false on give-up.
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const u64 t0 = global_timer_ns();
  for (u32 spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((spin & 63u) == 63u && global_timer_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
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

__device__ __forceinline__ void consumer_barrier() {
  asm volatile("bar.sync 1, %0;\n" ::"n"(kScanConsumers) : "memory");
}

struct ScanSmem {
  alignas(128) i64 stage[kScanStages][kScanTile];
  u64 full[kScanStages];
  u64 empty[kScanStages];
  Agg warp_agg[2][kScanWarps];
  Agg head, tail;     // slow path: partial of a segment entering / leaving the tile
  i64 next_seg;       // slow path: broadcast of the segment that contains the next tile
  int abort_flag;
};

// Per-configuration additive offset m_base + lm_p and admissibility.
__device__ __forceinline__ bool segment_offset(const llmem_config* __restrict__ cfg, i64 seg, i64* off) {
  *off = 0;
  if (!cfg) return true;
  Cfg f = load_cfg(cfg + seg);
  Plan p;
  u64 peak;
  if (full_status(f, &p, &peak) != LLMEM_CFG_OK) return false;
  *off = (i64)p.offset;
  return true;
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

// Scratch payload: per CTA a head partial (segment that began in an earlier CTA's
// range) and a tail partial (segment that continues into a later CTA's range).
struct CtaPartials {
  Agg head, tail;
};

template <bool kRound>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_kernel(const i64* __restrict__ delta_aligned /* 16-byte aligned base */, int shift /* 0 or 1 */,
            const i64* __restrict__ offsets, i64 n, i64 total,
            i64* __restrict__ peak_out, i64* __restrict__ index_out, i64 tiles_per_cta,
            CtaPartials* __restrict__ partials, u32* __restrict__ status_word) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  ScanSmem& sm = *reinterpret_cast<ScanSmem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // virtual indices: event e lives at v = e + shift, so that v even <=> 16-byte aligned
  const i64 v_begin = shift, v_end = (i64)shift + total;
  const i64 ntiles = (v_end + kScanTile - 1) / kScanTile;
  const i64 tile_lo = (i64)blockIdx.x * tiles_per_cta;
  const i64 tile_hi = tile_lo + tiles_per_cta < ntiles ? tile_lo + tiles_per_cta : ntiles;

  if (tid == 0) {
    partials[blockIdx.x].head = agg_identity();
    partials[blockIdx.x].tail = agg_identity();
    for (int s = 0; s < kScanStages; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], kScanWarps);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();
  if (tile_lo >= tile_hi) return;
  volatile int* abort_flag = &sm.abort_flag;

  if (warp == kScanWarps) {
    // ---------------- producer ----------------
    if (lane == 0) {
      i64 issued = 0;
      for (i64 t = tile_lo; t < tile_hi; ++t, ++issued) {
        const int s = (int)(issued % kScanStages);
        const u32 par = (u32)((issued / kScanStages) & 1);
        if (!mbar_wait_bounded(&sm.empty[s], par ^ 1u, abort_flag)) break;
        const i64 t0 = t * kScanTile;
        const i64 v_lo = t0 > v_begin ? t0 : v_begin;
        const i64 v_hi = t0 + kScanTile < v_end ? t0 + kScanTile : v_end;
        const i64 a_lo = v_lo + (v_lo & 1), a_hi = v_hi - (v_hi & 1);
        i64* dst = sm.stage[s];
        // ragged first / last element (at most one each): plain loads
        if (a_lo > v_lo) dst[v_lo - t0] = delta_aligned[v_lo];
        if (a_hi < v_hi && v_hi - 1 >= a_lo) dst[v_hi - 1 - t0] = delta_aligned[v_hi - 1];
        if (a_hi > a_lo) {
          const u32 bytes = (u32)((a_hi - a_lo) * 8);
          mbar_arrive_expect_tx(&sm.full[s], bytes);
          bulk_load(dst + (a_lo - t0), delta_aligned + a_lo, bytes, &sm.full[s]);
        } else {
          mbar_arrive(&sm.full[s]);
        }
      }
      // drain: every copy that was issued must have landed before the CTA exits
      const i64 first = issued > kScanStages ? issued - kScanStages : 0;
      for (i64 k = first; k < issued; ++k)
        mbar_wait_bounded(&sm.full[k % kScanStages], (u32)((k / kScanStages) & 1), abort_flag);
      if (*abort_flag) atomicExch(status_word, (u32)LLMEM_ERR_TIMEOUT);
    }
    return;
  }

  // ---------------- consumers ----------------
  // seg: the segment that contains the first event of the current tile
  i64 seg, seg_vstart, seg_vend;
  {
    const i64 first_v = tile_lo * kScanTile > v_begin ? tile_lo * kScanTile : v_begin;
    i64 lo = 0, hi = n;  // smallest s with offsets[s+1] + shift > first_v
    while (lo < hi) {
      const i64 mid = lo + (hi - lo) / 2;
      if (__ldg(offsets + mid + 1) + shift > first_v) hi = mid;
      else lo = mid + 1;
    }
    seg = lo;
    seg_vstart = seg < n ? __ldg(offsets + seg) + shift : v_end;
    seg_vend = seg < n ? __ldg(offsets + seg + 1) + shift : v_end;
  }
  const i64 cta_vlo = tile_lo * kScanTile;  // segments that start at or after this started in this CTA
  Agg run = agg_identity();                 // thread 0: fold of the current segment so far
  int fast_parity = 0;
  bool aborted = false;

  i64 it = 0;
  for (i64 t = tile_lo; t < tile_hi; ++t, ++it) {
    const int s = (int)(it % kScanStages);
    const u32 par = (u32)((it / kScanStages) & 1);
    const i64 t0 = t * kScanTile;
    const i64 v_lo = t0 > v_begin ? t0 : v_begin;
    const i64 v_hi = t0 + kScanTile < v_end ? t0 + kScanTile : v_end;
    // On expiry the wait raises the CTA's abort flag; control still runs to the next
    // consumer barrier, after which every consumer sees the flag and leaves together.
    mbar_wait_bounded(&sm.full[s], par, abort_flag);
    const i64* tile = sm.stage[s];

    if (v_lo == t0 && v_hi == t0 + kScanTile && seg < n && seg_vend >= v_hi) {
      // ---------- fast path: the whole tile lies inside one segment ----------
      const longlong2* src = reinterpret_cast<const longlong2*>(tile + tid * kScanPerThread);
      longlong2 x[kScanPerThread / 2];
#pragma unroll
      for (int j = 0; j < kScanPerThread / 2; ++j) x[j] = src[j];
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[s]);  // the stage may be refilled
      i64 sum = ev<kRound>(x[0].x), mx = sum;
      int ix = 0;
      {
        sum += ev<kRound>(x[0].y);
        if (sum > mx) { mx = sum; ix = 1; }
      }
#pragma unroll
      for (int j = 1; j < kScanPerThread / 2; ++j) {
        sum += ev<kRound>(x[j].x);
        if (sum > mx) { mx = sum; ix = 2 * j; }
        sum += ev<kRound>(x[j].y);
        if (sum > mx) { mx = sum; ix = 2 * j + 1; }
      }
      Agg g{sum, mx, t0 + (i64)tid * kScanPerThread + ix, 1};
      g = warp_fold(g, lane);
      if (lane == 0) sm.warp_agg[fast_parity][warp] = g;
      consumer_barrier();
      if (*abort_flag) { aborted = true; break; }
      if (tid == 0) {
#pragma unroll
        for (int w = 0; w < kScanWarps; ++w) run = agg_fold(run, sm.warp_agg[fast_parity][w]);
      }
      fast_parity ^= 1;
      if (seg_vend == v_hi) {
        // the segment ends exactly with the tile
        if (tid == 0) {
          if (seg_vstart >= cta_vlo) write_raw(seg, run, seg_vstart, peak_out, index_out);
          else partials[blockIdx.x].head = run;
          run = agg_identity();
        }
        do {
          ++seg;
          seg_vstart = seg < n ? __ldg(offsets + seg) + shift : v_end;
          seg_vend = seg < n ? __ldg(offsets + seg + 1) + shift : v_end;
        } while (seg < n && seg_vend <= v_hi);
      }
      continue;
    }

    // ---------- slow path: segment boundaries inside the tile, or a ragged tile ----------
    if (tid == 0) {
      sm.head = agg_identity();
      sm.tail = agg_identity();
    }
    consumer_barrier();
    // pieces: segments seg, seg+1, ... that begin before v_hi; warps take them round-robin
    for (i64 sg = seg + warp; sg < n; sg += kScanWarps) {
      const i64 a = __ldg(offsets + sg) + shift, b = __ldg(offsets + sg + 1) + shift;
      if (a >= v_hi) break;
      if (b <= a || b <= v_lo) continue;  // empty, or (only with inconsistent offsets) already past
      const i64 pa = a > v_lo ? a : v_lo, pb = b < v_hi ? b : v_hi;
      Agg g = warp_fold_range<kRound>(tile, (int)(pa - t0), (int)(pb - t0), lane, t0);
      if (lane == 0) {
        const bool starts_here = a >= v_lo, ends_here = b <= v_hi;
        if (starts_here && ends_here) write_raw(sg, g, a, peak_out, index_out);
        else if (!starts_here) sm.head = g;
        else sm.tail = g;
      }
    }
    consumer_barrier();
    if (tid == 0) {
      // the segment that entered the tile
      if (seg < n && seg_vstart < v_lo) {
        run = agg_fold(run, sm.head);
        if (seg_vend <= v_hi) {
          if (seg_vstart >= cta_vlo) write_raw(seg, run, seg_vstart, peak_out, index_out);
          else partials[blockIdx.x].head = run;
          run = agg_identity();
        }
      }
      // the segment that leaves the tile (it began inside it)
      if (sm.tail.valid) run = sm.tail;
      // which segment contains the first event of the next tile
      i64 sg = seg;
      while (sg < n && __ldg(offsets + sg + 1) + shift <= v_hi) ++sg;
      sm.next_seg = sg;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[s]);
    consumer_barrier();
    if (*abort_flag) { aborted = true; break; }
    seg = sm.next_seg;
    seg_vstart = seg < n ? __ldg(offsets + seg) + shift : v_end;
    seg_vend = seg < n ? __ldg(offsets + seg + 1) + shift : v_end;
  }

  if (tid == 0 && !aborted && run.valid) {
    // the current segment continues into the next CTA's range
    if (seg_vstart >= cta_vlo) partials[blockIdx.x].tail = run;
    else partials[blockIdx.x].head = run;
  }
}

// Finish, one thread per segment: fold the partials of segments that cross CTA
// ranges, define empty segments, add m_base + lm_p, and mark inadmissible
// configurations.
__global__ void __launch_bounds__(256)
scan_finish_kernel(const i64* __restrict__ offsets, i64 n, int shift, const llmem_config* __restrict__ cfg,
                   i64* __restrict__ peak_out, i64* __restrict__ index_out, i64 tiles_per_cta,
                   const CtaPartials* __restrict__ partials) {
  for (i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (i64)gridDim.x * blockDim.x) {
    const i64 a = offsets[i] + shift, b = offsets[i + 1] + shift;
    i64 mx = 0, idx = -1;
    if (b > a) {
      const i64 ca = (a / kScanTile) / tiles_per_cta, cb = ((b - 1) / kScanTile) / tiles_per_cta;
      if (ca == cb) {  // finished by the CTA that owns it
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
    const bool ok = segment_offset(cfg, i, &off);
    peak_out[i] = ok ? off + mx : -1;
    if (index_out) index_out[i] = ok ? idx : -1;
  }
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_scan_peak(const int64_t* delta, const int64_t* offsets, int64_t n,
                                        int64_t total_events, const llmem_config* cfg,
                                        int64_t* peak_out, int64_t* peak_index_out, void* scratch,
                                        size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  clear_error();
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
  CtaPartials* partials = reinterpret_cast<CtaPartials*>(static_cast<unsigned char*>(scratch) + kScratchHeader);
  if (cudaMemsetAsync(status_word, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_scan_peak (memset)");

  const int shift = aligned_to(delta, 16) ? 0 : 1;
  const i64* delta_aligned = reinterpret_cast<const i64*>(delta) - shift;
  const bool round = (flags & LLMEM_FUSE_ROUND) != 0;
  i64 tiles_per_cta = 1;
  if (total_events > 0) {
    static thread_local int configured_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_dev != dev) {
      cudaError_t e1 = cudaFuncSetAttribute(scan_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScanSmem));
      cudaError_t e2 = cudaFuncSetAttribute(scan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScanSmem));
      if (e1 != cudaSuccess || e2 != cudaSuccess) return check_launch("llmem_scan_peak (shared memory opt-in)");
      configured_dev = dev;
    }
    const i64 ntiles = (total_events + shift + kScanTile - 1) / kScanTile;
    i64 grid = sm_count();
    if (grid > kMaxScanCtas) grid = kMaxScanCtas;
    if (grid > ntiles) grid = ntiles;
    tiles_per_cta = (ntiles + grid - 1) / grid;
    grid = (ntiles + tiles_per_cta - 1) / tiles_per_cta;
    if (round)
      scan_kernel<true><<<(unsigned)grid, kScanThreads, sizeof(ScanSmem), s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events,
          reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), tiles_per_cta, partials, status_word);
    else
      scan_kernel<false><<<(unsigned)grid, kScanThreads, sizeof(ScanSmem), s>>>(
          delta_aligned, shift, reinterpret_cast<const i64*>(offsets), n, total_events,
          reinterpret_cast<i64*>(peak_out), reinterpret_cast<i64*>(peak_index_out), tiles_per_cta, partials, status_word);
    llmem_status st = check_launch("llmem_scan_peak");
    if (st != LLMEM_OK) return st;
  }
  i64 blocks = (n + 255) / 256;
  const i64 cap = (i64)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  scan_finish_kernel<<<(unsigned)blocks, 256, 0, s>>>(
      reinterpret_cast<const i64*>(offsets), n, shift, cfg, reinterpret_cast<i64*>(peak_out),
      reinterpret_cast<i64*>(peak_index_out), tiles_per_cta, partials);
  return check_launch("llmem_scan_peak (finish)");
}
