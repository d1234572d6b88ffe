// Materialised event lists: per-configuration event counts and their exclusive
// scan, the expansion kernel that writes every signed delta, and in-place page
// rounding.  The expansion is bound by HBM writes (8 bytes per event): each warp
// builds 576-event chunks of deltas in its own shared memory and hands each to the
// TMA engine as one bulk store, double-buffered so that filling the next chunk
// overlaps the store.
#include <mutex>

#include "llmem_host.h"
#include "expand.cuh"
#include "fold.cuh"
#include "ranges.cuh"

namespace llmem {

// ---------------------------------------------------------------------------
// event counts + exclusive scan
// ---------------------------------------------------------------------------
constexpr int kCountThreads = 256;
constexpr int kCountItems = 4;
constexpr int kCountBlock = kCountThreads * kCountItems;  // configurations per CTA

__device__ __forceinline__ u64 warp_inclusive_scan(u64 v, int lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    u64 o = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v += o;
  }
  return v;
}

// Exclusive scan of one value per thread across a CTA of kCountThreads threads;
// returns the exclusive prefix and the CTA total.
__device__ __forceinline__ u64 block_exclusive_scan(u64 v, u64* total, u64* smem /* >= 9 */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  u64 inc = warp_inclusive_scan(v, lane);
  if (lane == 31) smem[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    u64 w = lane < (kCountThreads / 32) ? smem[lane] : 0;
    u64 winc = warp_inclusive_scan(w, lane);
    if (lane < (kCountThreads / 32)) smem[lane] = winc - w;
    if (lane == (kCountThreads / 32) - 1) smem[kCountThreads / 32] = winc;
  }
  __syncthreads();
  u64 r = smem[warp] + inc - v;
  *total = smem[kCountThreads / 32];
  __syncthreads();
  return r;
}

// Pass 1: counts, CTA-local exclusive offsets, per-CTA totals.
template <bool kDnn>
__global__ void __launch_bounds__(kCountThreads)
count_kernel(const llmem_config* __restrict__ cfg, i64 n, i64* __restrict__ offsets,
             uint8_t* __restrict__ status_out, u64* __restrict__ block_sums) {
  __shared__ u64 smem[16];
  const i64 base = (i64)blockIdx.x * kCountBlock + (i64)threadIdx.x * kCountItems;
  u64 c[kCountItems];
  u64 sum = 0;
#pragma unroll
  for (int j = 0; j < kCountItems; ++j) {
    c[j] = 0;
    const i64 i = base + j;
    if (i < n) {
      Cfg f = load_cfg(cfg + i);
      int st = check_fields(f, true, true);
      if (kDnn) {
        // the list of the second estimator (Section 3.1)
        DnnPlan p;
        u64 peak;
        st = dnn_full_status(f, &p, &peak);
        if (st == LLMEM_CFG_OK) c[j] = p.count;
      } else if (st == LLMEM_CFG_OK) {
        Plan p = make_plan(f, f.method);
        st = p.status;
        if (st == LLMEM_CFG_OK) {
          // the byte guard: the peak itself must stay below 2^62
          StaticSums s = make_static_sums(p, f.pos_len > 0);
          Dyn d = make_dyn(p, (u64)f.batch);
          bool fw;
          u64 rel = relative_peak(p, s, sat_add(s.gather, dyn_sum(p, d)), &fw);
          if (sat_add(p.offset, rel) >= kSat) st = LLMEM_CFG_OVERFLOW;
          else c[j] = p.count;
        }
      }
      if (status_out) status_out[i] = (uint8_t)st;
    }
    sum += c[j];
  }
  u64 total;
  u64 excl = block_exclusive_scan(sum, &total, smem);
#pragma unroll
  for (int j = 0; j < kCountItems; ++j) {
    const i64 i = base + j;
    if (i < n) offsets[i] = (i64)excl;
    excl += c[j];
  }
  if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
}

// Pass 2 (one CTA): exclusive scan of the per-CTA totals in place; the grand total
// goes to block_sums[nblocks].
__global__ void __launch_bounds__(kCountThreads)
scan_block_sums_kernel(u64* __restrict__ block_sums, i64 nblocks) {
  __shared__ u64 smem[16];
  u64 carry = 0;
  for (i64 base = 0; base < nblocks; base += kCountThreads) {
    const i64 i = base + threadIdx.x;
    u64 v = i < nblocks ? block_sums[i] : 0;
    u64 total;
    u64 excl = block_exclusive_scan(v, &total, smem);
    if (i < nblocks) block_sums[i] = carry + excl;
    carry += total;
  }
  if (threadIdx.x == 0) block_sums[nblocks] = carry;
}

// Pass 3: add each CTA's base; write offsets[n].
__global__ void __launch_bounds__(256)
add_block_base_kernel(i64* __restrict__ offsets, i64 n, const u64* __restrict__ block_sums, i64 nblocks) {
  for (i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x; i <= n; i += (i64)gridDim.x * blockDim.x) {
    if (i == n) offsets[n] = (i64)block_sums[nblocks];
    else offsets[i] += (i64)block_sums[i / kCountBlock];
  }
}

// ---------------------------------------------------------------------------
// slabs: cutting a grid whose lists do not fit the device at once
// ---------------------------------------------------------------------------
// One warp cuts configurations [first, n) into contiguous slabs of at most max_events events,
// greedily: every slab takes as many configurations as fit; one with more events than that is
// a slab of its own.  The end of a slab is found by the warp's 32-ary search on the offsets.
__global__ void __launch_bounds__(32)
slab_bounds_kernel(const i64* __restrict__ offsets, i64 n, i64 max_events, i64 first, i64* __restrict__ bounds_out,
                   i64* __restrict__ events_out, i64 max_slabs, i64* __restrict__ count_out) {
  const int lane = threadIdx.x;
  i64 a = first, slabs = 0;
  if (lane == 0) {
    bounds_out[0] = first;
    events_out[0] = __ldg(offsets + first);
  }
  while (a < n && slabs < max_slabs) {
    // smallest s with offsets[s + 1] > offsets[a] + max_events: configurations a .. s-1 fit
    const i64 target = __ldg(offsets + a) + max_events;
    i64 b = warp_search_cost(offsets, n, 0, target, lane);
    if (b < a + 1) b = a + 1;
    if (b > n) b = n;
    ++slabs;
    if (lane == 0) {
      bounds_out[slabs] = b;
      events_out[slabs] = __ldg(offsets + b);
    }
    a = b;
  }
  if (lane == 0) *count_out = a < n ? -1 : slabs;
}

// ---------------------------------------------------------------------------
// expansion (run tables, cursor and store primitives: expand.cuh)
// ---------------------------------------------------------------------------
// The list is cut into n_blocks contiguous blocks of equal cost (events + kappa per segment,
// ranges.cuh), many more than the grid has warps; every warp streams one block of 576-event
// chunks at a time on its own: no CTA-wide barrier anywhere, so the warps of an SM drift
// apart and cover each other's latencies.  Lane l owns events [18 l, 18 l + 18) of a chunk.
// With a work counter (caller-provided scratch) the grid is persistent and a warp that has
// finished its block claims the next unclaimed one; without, the grid has one warp per block
// and the hardware block scheduler hands out the CTAs.  Either way SMs that reach HBM faster
// take more of the list.
//
// A full chunk inside one run of equal or two alternating events repeats the chunk written
// from the same buffer two chunks earlier: the buffer is left as it is and only the bulk
// store is issued.
__global__ void __launch_bounds__(kExpThreads)
expand_kernel(const llmem_config* __restrict__ cfg, i64 n, const i64* __restrict__ offsets, i64 total,
              i64* __restrict__ out, i64 n_blocks, i64 kappa, int round /* bit 0: rounded values, bit 1: second estimator */,
              int bulk_ok,
              unsigned long long* __restrict__ work_counter, u32* __restrict__ status_word) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  ExpandWarpSmem& ws = reinterpret_cast<ExpandWarpSmem*>(smem_raw)[warp];
  const Guard g{status_word, n, total};
  const i64 resident = (i64)gridDim.x * kExpWarps;
  i64 desc_seg = -1;  // segment described by ws.desc
  int parity = 0;
  BufferKeys keys;  // what the two chunk buffers hold
  for (i64 gw = (i64)blockIdx.x * kExpWarps + warp; gw < n_blocks;) {
    i64 seg;  // smallest segment whose end lies beyond the current position; gs/ge its range
    const i64 b_lo = warp_block_start(offsets, n, 0, total, gw, n_blocks, kappa, kExpChunk, lane, &seg);
    const i64 b_hi = warp_block_start(offsets, n, 0, total, gw + 1, n_blocks, kappa, kExpChunk, lane, nullptr);
    const i64 c_lo = b_lo / kExpChunk, c_hi = (b_hi + kExpChunk - 1) / kExpChunk;
    i64 gs = seg < n ? __ldg(offsets + seg) : total;
    i64 ge = seg < n ? __ldg(offsets + seg + 1) : total;
    AlternatingRun ar;  // the alternating run the last such chunk lay in

    for (i64 c = c_lo; c < c_hi; ++c, parity ^= 1) {
      const i64 tb = c * kExpChunk;
      const i64 te = tb + kExpChunk < total ? tb + kExpChunk : total;
      i64* buf = ws.buf[parity];
      // a full chunk inside one segment may repeat the one before
      const bool alternating = seg < n && gs <= tb && tb + kExpChunk <= ge &&
                               chunk_alternates(ar, ws, desc_seg, cfg, seg, gs, ge, tb, round, lane, g);
      if (alternating) {
        prepare_alternating<kExpStoresInFlight>(ar, keys, parity, buf, lane);
        if (ge == te) {
          // the segment ends with this chunk: move to the next non-empty one
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
            // offsets do not cover the rest of the chunk: define it as zeros
            for (i64 e = (span_lo > pos ? span_lo : pos); e < span_hi; ++e) buf[e - tb] = 0;
            break;
          }
          ensure_desc(ws, desc_seg, cfg, seg, gs, ge, round, lane, g);
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
          pos = piece_end;
          if (ge <= te) {
            // the segment ends inside this chunk: move to the next non-empty one
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
    if (work_counter == nullptr) break;  // one block per warp
    // the first `resident` blocks are taken by number, the others in order of request
    unsigned long long ticket = 0;
    if (lane == 0) ticket = atomicAdd(work_counter, 1ull);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    gw = resident + (i64)ticket;
  }
  if (lane == 0) bulk_wait_read<0>();
}

// ---------------------------------------------------------------------------
// rounding in place
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
round_kernel(i64* __restrict__ delta, i64 total) {
  // 16-byte vectors over the aligned middle, scalars for a ragged first / last element
  const i64 head = ((reinterpret_cast<uintptr_t>(delta) & 15) != 0 && total > 0) ? 1 : 0;
  const i64 nvec = (total - head) / 2;
  longlong2* v = reinterpret_cast<longlong2*>(delta + head);
  const i64 stride = (i64)gridDim.x * blockDim.x;
  const i64 t0 = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  for (i64 i = t0; i < nvec; i += stride) {
    longlong2 x = v[i];
    x.x = page_round_signed(x.x);
    x.y = page_round_signed(x.y);
    v[i] = x;
  }
  if (t0 == 0) {
    if (head) delta[0] = page_round_signed(delta[0]);
    const i64 tail = head + 2 * nvec;
    if (tail < total) delta[tail] = page_round_signed(delta[tail]);
  }
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_event_counts(const llmem_config* cfg, int64_t n, int64_t* offsets_out,
                                           uint8_t* status_out, void* scratch, size_t scratch_bytes,
                                           uint32_t flags, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_event_counts");
  if (n < 0) { set_error("llmem_event_counts: n < 0"); return LLMEM_ERR_ARG; }
  if (!offsets_out || !aligned_to(offsets_out, 8)) { set_error("llmem_event_counts: offsets_out is required"); return LLMEM_ERR_ARG; }
  if (n > 0 && (!cfg || !aligned_to(cfg, 16))) { set_error("llmem_event_counts: cfg must be a 16-byte aligned device pointer"); return LLMEM_ERR_ARG; }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (n == 0) {
    if (cudaMemsetAsync(offsets_out, 0, sizeof(int64_t), s) != cudaSuccess) return check_launch("llmem_event_counts");
    return LLMEM_OK;
  }
  if (!scratch || !aligned_to(scratch, 256) ||
      scratch_bytes < llmem_scratch_bytes(LLMEM_OP_EVENT_COUNTS, n, 0)) {
    set_error("llmem_event_counts: scratch missing, misaligned or smaller than llmem_scratch_bytes()");
    return LLMEM_ERR_SCRATCH;
  }
  u64* block_sums = reinterpret_cast<u64*>(static_cast<unsigned char*>(scratch) + kScratchHeader);
  const i64 nblocks = (n + kCountBlock - 1) / kCountBlock;
  if (flags & LLMEM_ESTIMATOR_DNNMEM)
    count_kernel<true><<<(unsigned)nblocks, kCountThreads, 0, s>>>(cfg, n, reinterpret_cast<i64*>(offsets_out), status_out, block_sums);
  else
    count_kernel<false><<<(unsigned)nblocks, kCountThreads, 0, s>>>(cfg, n, reinterpret_cast<i64*>(offsets_out), status_out, block_sums);
  scan_block_sums_kernel<<<1, kCountThreads, 0, s>>>(block_sums, nblocks);
  i64 blocks3 = (n + 1 + 255) / 256;
  const i64 cap3 = (i64)sm_count() * 8;
  if (blocks3 > cap3) blocks3 = cap3;
  add_block_base_kernel<<<(unsigned)blocks3, 256, 0, s>>>(reinterpret_cast<i64*>(offsets_out), n, block_sums, nblocks);
  return check_launch("llmem_event_counts");
}

// ---------------------------------------------------------------------------
// llmem_event_counts_static: the same three kernels, with the per-CTA partial sums
// kept in a file-scope device array instead of caller-provided scratch.
// ---------------------------------------------------------------------------
namespace llmem {

constexpr i64 kStaticMaxConfigs = LLMEM_STATIC_MAX_CONFIGS;
constexpr i64 kStaticSums = kStaticMaxConfigs / kCountBlock + 1;  // 4096 CTA totals + the grand total
static_assert(kStaticMaxConfigs % kCountBlock == 0, "limit is a whole number of CTAs");

// Lives in the module image of every device that loads the library (about 32 KiB)
// until the process exits.  Shared by all calls of the entry point below.
static __device__ __align__(256) unsigned long long g_static_block_sums[kStaticSums];

constexpr int kMaxDevices = 64;
static u64* g_static_ptr[kMaxDevices];  // device address of the array, per device ordinal
static std::mutex g_static_mutex;

// In host code `g_static_block_sums` names a host-side shadow of the symbol, not
// device memory; the address a kernel may dereference has to be asked for, with the
// device in question current.
static llmem_status static_sums_address(u64** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_error("llmem_event_counts_static: cudaGetDevice: %s", cudaGetErrorString(e)); return LLMEM_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) { set_error("llmem_event_counts_static: device ordinal %d beyond %d", dev, kMaxDevices - 1); return LLMEM_ERR_ARG; }
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_block_sums);
    if (e != cudaSuccess || !p) {
      set_error("llmem_event_counts_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
      return LLMEM_ERR_CUDA;
    }
    g_static_ptr[dev] = static_cast<u64*>(p);
  }
  *out = g_static_ptr[dev];
  return LLMEM_OK;
}

}  // namespace llmem

extern "C" llmem_status llmem_event_counts_static(const llmem_config* cfg, int64_t n, int64_t* offsets_out,
                                                  uint8_t* status_out, uint32_t flags, void* cuda_stream) {
  clear_error();
  if (n < 0) { set_error("llmem_event_counts_static: n < 0"); return LLMEM_ERR_ARG; }
  if (n > kStaticMaxConfigs) {
    set_error("llmem_event_counts_static: n = %lld exceeds LLMEM_STATIC_MAX_CONFIGS = %lld; split the batch or "
              "use llmem_event_counts with caller-provided scratch", (long long)n, (long long)kStaticMaxConfigs);
    return LLMEM_ERR_ARG;
  }
  if (!offsets_out || !aligned_to(offsets_out, 8)) { set_error("llmem_event_counts_static: offsets_out is required"); return LLMEM_ERR_ARG; }
  if (n > 0 && (!cfg || !aligned_to(cfg, 16))) { set_error("llmem_event_counts_static: cfg must be a 16-byte aligned device pointer"); return LLMEM_ERR_ARG; }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (n == 0) {
    if (cudaMemsetAsync(offsets_out, 0, sizeof(int64_t), s) != cudaSuccess) return check_launch("llmem_event_counts_static");
    return LLMEM_OK;
  }
  u64* block_sums = nullptr;
  llmem_status st = static_sums_address(&block_sums);
  if (st != LLMEM_OK) return st;
  // Nothing in the array has to start at zero: pass 1 writes entries [0, nblocks), pass 2
  // rewrites them and writes entry [nblocks], and no pass reads an entry this call has not
  // written.  What an earlier call left beyond nblocks is never looked at.
  const i64 nblocks = (n + kCountBlock - 1) / kCountBlock;
  if (flags & LLMEM_ESTIMATOR_DNNMEM)
    count_kernel<true><<<(unsigned)nblocks, kCountThreads, 0, s>>>(cfg, n, reinterpret_cast<i64*>(offsets_out), status_out, block_sums);
  else
    count_kernel<false><<<(unsigned)nblocks, kCountThreads, 0, s>>>(cfg, n, reinterpret_cast<i64*>(offsets_out), status_out, block_sums);
  scan_block_sums_kernel<<<1, kCountThreads, 0, s>>>(block_sums, nblocks);
  i64 blocks3 = (n + 1 + 255) / 256;
  const i64 cap3 = (i64)sm_count() * 8;
  if (blocks3 > cap3) blocks3 = cap3;
  add_block_base_kernel<<<(unsigned)blocks3, 256, 0, s>>>(reinterpret_cast<i64*>(offsets_out), n, block_sums, nblocks);
  return check_launch("llmem_event_counts_static");
}

extern "C" llmem_status llmem_slab_bounds(const int64_t* offsets, int64_t n, int64_t max_events, int64_t first,
                                          int64_t* bounds_out, int64_t* events_out, int64_t max_slabs,
                                          int64_t* count_out, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_slab_bounds");
  if (n < 0 || max_events < 1 || first < 0 || first > n || max_slabs < 1) {
    set_error("llmem_slab_bounds: n >= 0, max_events >= 1, 0 <= first <= n and max_slabs >= 1 are required");
    return LLMEM_ERR_ARG;
  }
  if (!offsets || !bounds_out || !events_out || !count_out || !aligned_to(offsets, 8) || !aligned_to(bounds_out, 8) ||
      !aligned_to(events_out, 8) || !aligned_to(count_out, 8)) {
    set_error("llmem_slab_bounds: offsets, bounds_out, events_out and count_out must be 8-byte aligned device pointers");
    return LLMEM_ERR_ARG;
  }
  slab_bounds_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      reinterpret_cast<const i64*>(offsets), n, max_events, first, reinterpret_cast<i64*>(bounds_out),
      reinterpret_cast<i64*>(events_out), max_slabs, reinterpret_cast<i64*>(count_out));
  return check_launch("llmem_slab_bounds");
}

extern "C" llmem_status llmem_expand_events(const llmem_config* cfg, int64_t n, const int64_t* offsets,
                                            int64_t total_events, int64_t* delta_out, void* scratch,
                                            size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_expand_events");
  if (n < 0 || total_events < 0) { set_error("llmem_expand_events: negative size"); return LLMEM_ERR_ARG; }
  if (total_events == 0) return LLMEM_OK;
  if (!cfg || !offsets || !delta_out) { set_error("llmem_expand_events: cfg, offsets and delta_out are required"); return LLMEM_ERR_ARG; }
  if (!aligned_to(cfg, 16) || !aligned_to(offsets, 8) || !aligned_to(delta_out, 8)) {
    set_error("llmem_expand_events: misaligned pointer");
    return LLMEM_ERR_ARG;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // bit 0: values page-rounded (aligned to 512 bytes under the second estimator); bit 1: the second estimator's list
  const int round_bits = ((flags & LLMEM_FUSE_ROUND) ? 1 : 0) | ((flags & LLMEM_ESTIMATOR_DNNMEM) ? 2 : 0);
  if (short_segment_list(n, total_events) && scratch && aligned_to(scratch, 256) &&
      scratch_bytes >= expand_scan_scratch_bytes(n, total_events)) {
    // lists of short segments: every segment written by its owner, a lane or a warp
    if (cudaMemsetAsync(scratch, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_expand_events (memset)");
    return expand_by_owners(cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out),
                            round_bits, false, nullptr, nullptr, scratch, nullptr, s);
  }
  const size_t smem = sizeof(ExpandWarpSmem) * kExpWarps;
  static thread_local int configured_dev = -1;
  int dev = 0;
  cudaGetDevice(&dev);
  if (configured_dev != dev) {
    if (cudaFuncSetAttribute(expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return check_launch("llmem_expand_events (shared memory opt-in)");
    configured_dev = dev;
  }
  const i64 nchunks = (total_events + kExpChunk - 1) / kExpChunk;
  const i64 resident = (i64)sm_count() * kExpCtasPerSm * kExpWarps;
  const i64 blocks = stream_warps(resident, LLMEM_EXP_OVERSUB, nchunks, LLMEM_EXP_MIN_CHUNKS);
  // with scratch the warps of a persistent grid claim blocks from a counter in its header
  unsigned long long* work_counter = nullptr;
  u32* status_word = nullptr;  // only written by checked builds
  if (scratch && aligned_to(scratch, 256) && scratch_bytes >= kScratchHeader) {
    if (cudaMemsetAsync(scratch, 0, kScratchHeader, s) != cudaSuccess) return check_launch("llmem_expand_events (memset)");
    status_word = static_cast<u32*>(scratch);
    if (blocks > resident)
      work_counter = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(scratch) + kWorkCounterOffset);
  }
  const i64 grid_warps = work_counter ? resident : blocks;
  const i64 grid = (grid_warps + kExpWarps - 1) / kExpWarps;
  expand_kernel<<<(unsigned)grid, kExpThreads, smem, s>>>(
      cfg, n, reinterpret_cast<const i64*>(offsets), total_events, reinterpret_cast<i64*>(delta_out),
      blocks, kExpSegmentCost, round_bits, aligned_to(delta_out, 16) ? 1 : 0, work_counter,
      status_word);
  return check_launch("llmem_expand_events");
}

extern "C" llmem_status llmem_round_events(int64_t* delta, int64_t total_events, void* scratch,
                                           size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  (void)scratch; (void)scratch_bytes; (void)flags;
  clear_error();
  TraceRange trace("llmem_round_events");
  if (total_events < 0) { set_error("llmem_round_events: negative size"); return LLMEM_ERR_ARG; }
  if (total_events == 0) return LLMEM_OK;
  if (!delta || !aligned_to(delta, 8)) { set_error("llmem_round_events: delta must be an 8-byte aligned device pointer"); return LLMEM_ERR_ARG; }
  i64 blocks = (total_events / 2 + 255) / 256;
  const i64 cap = (i64)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  round_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(reinterpret_cast<i64*>(delta), total_events);
  return check_launch("llmem_round_events");
}
