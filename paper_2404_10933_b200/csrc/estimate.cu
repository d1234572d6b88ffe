// Fused kernels: peak estimation without a materialised event list, largest-batch
// search and Algorithm 1.  One thread evaluates one configuration (four threads per
// shape in the selection kernel); identical consecutive events are summed as
// count * rounded size, which is exact because all allocations of an iteration
// precede its frees.  The work is plain 64-bit integer arithmetic; global traffic is
// 64 bytes in and a few bytes out per configuration.
#include "llmem_host.h"
#include "llmem_model.cuh"

// Resident CTAs per SM the register allocation of the per-configuration kernels aims at
// (overridable at compile time for tuning sweeps).
#ifndef LLMEM_EST_MIN_CTAS
#define LLMEM_EST_MIN_CTAS 3
#endif
#ifndef LLMEM_EST_THREADS
#define LLMEM_EST_THREADS 256
#endif
// CTAs per SM the estimate's grid is capped at (its threads stride over the configurations)
#ifndef LLMEM_EST_GRID_CTAS
#define LLMEM_EST_GRID_CTAS 32
#endif
// the same for the two search kernels
#ifndef LLMEM_SEARCH_GRID_CTAS
#define LLMEM_SEARCH_GRID_CTAS 256
#endif
#ifndef LLMEM_SEARCH_MIN_CTAS
#define LLMEM_SEARCH_MIN_CTAS 4
#endif

namespace llmem {

// Peak of one admissible plan at a given batch: m_base + lm_p + largest prefix sum.
// Returns kSat when the value does not fit below 2^62.
struct Search {
  Plan p;
  StaticSums s;
  __device__ __forceinline__ u64 peak(u64 batch, Dyn* d_out, bool* first_wins) const {
    Dyn d = make_dyn(p, batch);
    if (d_out) *d_out = d;
    u64 rel = relative_peak(p, s, sat_add(s.gather, dyn_sum(p, d)), first_wins);
    return sat_add(p.offset, rel);
  }
};

// The batch search of Section 6 in units of pages.  Every rounded event is a multiple
// of cu_p = 2^21, so  peak(b) <= capacity  <=>  pages(b) <= (capacity - m_base - lm_p) >> 21.
// Batches whose raw sizes would reach 2^62 bytes are excluded up front (they cannot fit
// any capacity), which leaves plain, unchecked 64-bit arithmetic inside the probes; the
// one division a probe would need, floor(out / tp) for the TP backward buffer, is done
// with a per-configuration reciprocal.
struct PageSearch {
  u64 out1, logit1, shift1;  // bytes per sample of a layer output / the logits / a shifted copy
  u64 attn1, ffn1;           // bytes per sample of a score-sized / ffn-sized operator output
  u32 n_attn, n_ffn;         // how many of those are kept over all layers (0 with checkpointing)
  u64 q1, recip;             // floor(out1 / tp), ceil(2^64 / tp)
  u64 fixed_a, fixed_b;      // pages that do not depend on the batch (see pages())
  u64 offset;                // m_base + lm_p
  u32 r1;                    // out1 mod tp
  u32 n_out, n_back;         // outputs kept per iteration; TP backward buffers (0 if none or tp = 1)
  int b_safe;                // probes stay within 1..b_safe; 0: nothing can fit
  bool single_iter;
  double rate_up, rate_dn;   // cu_p / W for a W not above, and one not below, the bytes a sample adds
  double dyn_events;         // N: at least the number of batch-dependent events of one iteration

  // `too_large`: one of the batch-independent sums (or the per-sample score size) reached 2^62
  // `big_limit` = floor((2^62 - 1) / bmax), the same for every configuration of a call
  __device__ __forceinline__ void init(const Plan& p, const StaticSums& s, int bmax, bool too_large, u64 big_limit) {
    out1 = p.out1; logit1 = p.logit1; shift1 = p.shift1;
    offset = p.offset;
    n_out = (u32)(p.e_n + p.L * p.n_x);
    n_attn = (u32)(p.L * p.n_attn);
    n_ffn = (u32)(p.L * p.n_ffn);
    attn1 = n_attn ? p.attn1 : 0;
    ffn1 = n_ffn ? p.ffn1 : 0;
    n_back = (p.tpback && p.tp > 1) ? (u32)p.L : 0u;
    q1 = 0; r1 = 0; recip = 0;
    if (n_back) {
      recip = p.tp_recip;             // ceil(2^64 / tp), tp >= 2
      q1 = __umul64hi(out1, recip);   // floor(out1 / tp): exact, out1 < 2^48
      r1 = (u32)(out1 - q1 * p.tp);
    }
    single_iter = p.iters < 2;
    if (too_large) {
      b_safe = 0;
      fixed_a = fixed_b = 0;
      rate_up = rate_dn = dyn_events = 0.0;
      return;
    }
    const u64 init_p = s.init >> 21, os_p = s.os >> 21, gat_p = s.gather >> 21;
    // one iteration: max(init + gather + dyn, init + os); otherwise init + os + gather + dyn
    fixed_a = single_iter ? init_p + gat_p : init_p + os_p + gat_p;
    fixed_b = init_p + os_p;
    u64 big = out1 > logit1 ? out1 : logit1;  // >= 2
    if (attn1 > big) big = attn1;
    if (ffn1 > big) big = ffn1;
    // the largest b <= bmax with b * big < 2^62: bmax itself unless a per-sample size is huge
    b_safe = big <= big_limit ? bmax : (int)((kSat - 1) / big);
    // bytes one more sample adds to the batch-dependent events, without the backward buffers;
    // those add  out - floor(out / tp)  per layer, which lies between b (out1 - q1 - 1) and
    // b (out1 - q1)
    const double w = (double)n_out * (double)out1 + (double)logit1 + 2.0 * (double)shift1 +
                     (double)n_attn * (double)attn1 + (double)n_ffn * (double)ffn1;
    const double back_hi = n_back ? (double)(out1 - q1) : 0.0;  // out1 >= 2 q1 >= q1 + 1 when tp >= 2
    rate_up = (double)kPage / (w + (double)n_back * (back_hi - (n_back ? 1.0 : 0.0)));
    rate_dn = (double)kPage / (w + (double)n_back * back_hi);
    dyn_events = (double)(n_out + n_attn + n_ffn + 2 * n_back + 3);
  }

  template <bool kActs>
  __device__ __forceinline__ u64 pages(u32 b) const {
    const u64 out = (u64)b * out1, logit = (u64)b * logit1, shift = (u64)b * shift1;
    u64 dyn = (u64)n_out * ((out + (kPage - 1)) >> 21) + ((logit + (kPage - 1)) >> 21) +
              2 * ((shift + (kPage - 1)) >> 21);
    if (kActs) {
      dyn += (u64)n_attn * (((u64)b * attn1 + (kPage - 1)) >> 21) + (u64)n_ffn * (((u64)b * ffn1 + (kPage - 1)) >> 21);
    }
    if (n_back) {
      // floor(out / tp) = b q1 + floor(b r1 / tp); b r1 < 2^34, exact with the 64-bit reciprocal
      const u64 back = out - ((u64)b * q1 + __umul64hi((u64)b * r1, recip));
      dyn += (u64)n_back * ((back + (kPage - 1)) >> 21);
    }
    const u64 t = fixed_a + dyn;
    return single_iter ? (t > fixed_b ? t : fixed_b) : t;
  }

  // Section 6: the largest b in 1..bmax with peak(b) <= capacity.  Algorithm 1
  // increments b until the peak exceeds m_total; the peak never decreases with b, so any
  // search that ends with "b fits, b + 1 does not" finds the same b.  The page count is
  // almost linear in b: with W the bytes all batch-dependent events take per sample and N
  // their number,  b W / cu_p <= dyn pages(b) < b W / cu_p + N  (every event rounds up by
  // less than a page).  So with R pages of room nothing above R cu_p / W fits and everything
  // up to (R - N) cu_p / W does.  Both bounds are computed in double precision: the sums and
  // products behind them are of positive terms, fewer than twenty roundings of 2^-53 each,
  // and the bounds are widened by 2^-40, far more than that, before they are cut to integers,
  // so the bracket is certain.  For most shapes it holds one candidate and no probe is needed;
  // otherwise it is bisected with exact page counts.
  __device__ __forceinline__ int largest_batch(i64 capacity) const {
    const u64 cap = capacity >= (i64)kSat ? kSat - 1 : (u64)(capacity < 0 ? 0 : capacity);
    if (capacity < 0 || cap < offset || b_safe == 0) return 0;
    const u64 budget = (cap - offset) >> 21;
    if (budget < fixed_a || (single_iter && budget < fixed_b)) return 0;  // pages(b) is at least that
    // the operator-output terms are decided once, outside the probe loop
    return n_attn ? guided<true>(budget) : guided<false>(budget);
  }

  template <bool kActs>
  __device__ __forceinline__ int guided(u64 budget) const {
    const double room = (double)(budget - fixed_a);  // below 2^41: exact
    const double up = room * rate_up * (1.0 + 0x1p-40);
    int hi = up >= (double)b_safe ? b_safe : (int)up;  // nothing above hi fits
    const double dn = (room - dyn_events) * rate_dn * (1.0 - 0x1p-40);
    int lo = dn < 1.0 ? 0 : (dn >= (double)hi ? hi : (int)dn);  // lo fits (or is 0)
    while (lo < hi) {
      const int mid = lo + (hi - lo + 1) / 2;
      if (pages<kActs>((u32)mid) <= budget) lo = mid;
      else hi = mid - 1;
    }
    return lo;
  }
};

// ---------------------------------------------------------------------------
// llmem_estimate_batch
// ---------------------------------------------------------------------------
// One configuration: status, peak and its position.
__device__ __forceinline__ void estimate_one(const Cfg& f, i64* pk_out, i64* ix_out, int* st_out) {
  int st = check_fields(f, true, true);
  i64 pk = -1, ix = -1;
  if (st == LLMEM_CFG_OK) {
    // only the peak is wanted: plain sums and products that remember whether one was too large
    StickyMath m;
    const Plan p = make_plan(m, f, f.method);
    st = p.status;
    if (st == LLMEM_CFG_OK) {
      const StaticSums s = make_static_sums(m, p, f.pos_len > 0);
      const Dyn d = make_dyn(m, p, (u64)f.batch);
      bool first_wins;
      const u64 rel = relative_peak(m, p, s, m.add(s.gather, dyn_sum(m, p, d)), &first_wins);
      const u64 total = m.add(p.offset, rel);
      if (m.too_large(total)) {
        st = LLMEM_CFG_OVERFLOW;
      } else {
        pk = (i64)total;
        // position of the peak: the last allocation of non-zero size in the
        // iteration that attains it, or the last optimizer-state allocation
        const u64 init_n = 2 + 2 * (u64)p.C;
        const u64 gpart = p.gather ? 1 + (u64)p.C : 0;
        const u64 outs = (u64)p.e_n + (u64)p.L * (u64)(p.n_x + p.n_attn + p.n_ffn);
        const u64 allocs = gpart + outs + 3 + (p.tpback ? (u64)p.L : 0);
        const u64 os_n = (u64)p.e_n + (u64)p.K * (u64)p.L;
        const u64 last = (p.tpback && d.back > 0) ? allocs - 1
                         : (d.shift > 0 ? gpart + outs + 2 : gpart + outs);
        if (p.iters >= 2) ix = (i64)(init_n + 2 * allocs + os_n + last);
        else if (first_wins) ix = (i64)(init_n + last);
        else ix = (i64)(init_n + 2 * allocs + os_n - 1);
      }
    }
  }
  *pk_out = pk;
  *ix_out = ix;
  *st_out = st;
}

// One thread per configuration.  The lanes of a warp hold configurations of different methods,
// so the model forms the quotients by the partition degrees in every lane and selects (a
// division that three lanes in four need is not worth a branch): on a random mix of the four
// methods 29.6 of 32 lanes are busy per instruction.  Handing the configurations of a CTA's
// tile out in the order of a counting sort by method was tried before that and lost to the
// barriers of the sort.
// The same for the DNNMem-style estimator of Section 3.1: the list only grows, so the peak is
// the total and sits at the last event of non-zero size (the second shifted copy, or the
// logits when the sequence has one token).
__device__ __forceinline__ void dnn_estimate_one(const Cfg& f, i64* pk_out, i64* ix_out, int* st_out) {
  DnnPlan p;
  u64 peak;
  const int st = dnn_full_status(f, &p, &peak);
  *st_out = st;
  *pk_out = st == LLMEM_CFG_OK ? (i64)peak : -1;
  *ix_out = st == LLMEM_CFG_OK ? (i64)(p.shift > 0 ? p.count - 1 : p.count - 3) : -1;
}

template <bool kDnn>
__global__ void __launch_bounds__(LLMEM_EST_THREADS, LLMEM_EST_MIN_CTAS)
estimate_kernel(const llmem_config* __restrict__ cfg, i64 n, i64* __restrict__ peak_out,
                i64* __restrict__ index_out, uint8_t* __restrict__ status_out) {
  for (i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (i64)gridDim.x * blockDim.x) {
    const Cfg f = load_cfg(cfg + i);
    i64 pk, ix;
    int st;
    if (kDnn) dnn_estimate_one(f, &pk, &ix, &st);
    else estimate_one(f, &pk, &ix, &st);
    peak_out[i] = pk;
    if (index_out) index_out[i] = ix;
    if (status_out) status_out[i] = (uint8_t)st;
  }
}

// ---------------------------------------------------------------------------
// llmem_max_batch: one thread per shape, capacities innermost (the peak curve
// does not depend on the capacity, so the plan is built once)
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256, LLMEM_SEARCH_MIN_CTAS)
max_batch_kernel(const llmem_config* __restrict__ shape, i64 n, const i64* __restrict__ caps,
                 int n_cap, int bmax, u64 big_limit, int* __restrict__ bs_out, uint8_t* __restrict__ status_out) {
  for (i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (i64)gridDim.x * blockDim.x) {
    Cfg f = load_cfg(shape + i);
    int st = check_fields(f, false, true);
    PageSearch q;
    if (st == LLMEM_CFG_OK) {
      StickyMath m;
      const Plan p = make_plan(m, f, f.method);
      st = p.status;
      if (st == LLMEM_CFG_OK) {
        const StaticSums s = make_static_sums(m, p, f.pos_len > 0);
        q.init(p, s, bmax, m.too_large(0), big_limit);
      }
    }
    int* out = bs_out + i * n_cap;
    if (st != LLMEM_CFG_OK) {
      for (int m = 0; m < n_cap; ++m) out[m] = -1;
    } else {
      for (int m = 0; m < n_cap; ++m) out[m] = q.largest_batch(__ldg(caps + m));
    }
    if (status_out) status_out[i] = (uint8_t)st;
  }
}

// ---------------------------------------------------------------------------
// llmem_select_method: four lanes per shape, lane k searching method k; the
// quad exchanges its four batches by shuffle and lane 0 takes the decision.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256, LLMEM_SEARCH_MIN_CTAS)
select_kernel(const llmem_config* __restrict__ shape, i64 n, const i64* __restrict__ caps, int n_cap,
              int bmax, u64 big_limit, u32 flags, int* __restrict__ method_out, int* __restrict__ batch_out,
              int* __restrict__ bs_list_out, uint8_t* __restrict__ status_out) {
  const i64 quads_per_grid = ((i64)gridDim.x * blockDim.x) >> 2;
  const u32 k = threadIdx.x & 3;  // method of this lane
  const u32 quad_base = (threadIdx.x & 31) & ~3u;
  // n rounded up so that whole warps stay in the loop (shuffles need all lanes)
  const i64 n_warp_rounded = (n + 7) & ~(i64)7;
  for (i64 i = ((i64)blockIdx.x * blockDim.x + threadIdx.x) >> 2; i < n_warp_rounded; i += quads_per_grid) {
    const bool live = i < n;
    int st = LLMEM_CFG_FIELD;
    PageSearch q;
    bool usable = false;
    u32 gpu_n = 1, tp_n = 1;
    if (live) {
      Cfg f = load_cfg(shape + i);
      st = check_fields(f, false, false);
      gpu_n = f.gpu_n;
      tp_n = f.tp_n;
      if (st == LLMEM_CFG_OK) {
        StickyMath m;
        const Plan p = make_plan(m, f, k);
        usable = p.status == LLMEM_CFG_OK;  // a method that cannot be configured scores 0
        if (usable) {
          const StaticSums s = make_static_sums(m, p, f.pos_len > 0);
          q.init(p, s, bmax, m.too_large(0), big_limit);
        }
      }
    }
    for (int m = 0; m < n_cap; ++m) {
      int bs = 0;
      if (usable) bs = q.largest_batch(__ldg(caps + m));
      int b0 = __shfl_sync(0xffffffffu, bs, quad_base + 0);
      int b1 = __shfl_sync(0xffffffffu, bs, quad_base + 1);
      int b2 = __shfl_sync(0xffffffffu, bs, quad_base + 2);
      int b3 = __shfl_sync(0xffffffffu, bs, quad_base + 3);
      if (!live) continue;
      const i64 o = i * n_cap + m;
      if (st != LLMEM_CFG_OK) {
        if (k == 0) { method_out[o] = -1; batch_out[o] = -1; }
        if (bs_list_out) bs_list_out[4 * o + k] = -1;
        continue;
      }
      if (bs_list_out) bs_list_out[4 * o + k] = bs;
      if (k == 0) {
        // scores doubled so that CDP's factor 1.5 stays integral; dp_n = gpu_n / tp_n
        const i64 nn = gpu_n;
        i64 e0 = 3 * (i64)b0 * nn, e1 = 2 * (i64)b1 * nn, e2 = 2 * (i64)b2;
        i64 e3 = b3 > 0 ? 2 * (i64)b3 * (nn / tp_n) : 0;
        int idx = 0, bb = b0;
        i64 best = e0;
        if (e1 > best) { best = e1; idx = 1; bb = b1; }
        if (e2 > best) { best = e2; idx = 2; bb = b2; }
        if (e3 > best) { best = e3; idx = 3; bb = b3; }
        const bool keep = (flags & LLMEM_SELECT_ALLZERO) ? (best != 0) : (e2 != 0);
        method_out[o] = keep ? idx : LLMEM_METHOD_OFFLOAD;
        batch_out[o] = keep ? bb : 0;
      }
    }
    if (live && k == 0 && status_out) status_out[i] = (uint8_t)st;
  }
}

// ---------------------------------------------------------------------------
// llmem_select_segmented: the decision of Algorithm 1 over arbitrary candidate groups.
// One thread per (group, capacity); capacities vary fastest so that a warp reads
// contiguous rows of the batch matrix.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
select_segmented_kernel(const llmem_config* __restrict__ item_cfg, const int* __restrict__ bs,
                        const i64* __restrict__ group_offsets, i64 n_groups, int n_cap,
                        i64* __restrict__ item_out, int* __restrict__ method_out, int* __restrict__ batch_out) {
  const i64 total = n_groups * n_cap;
  for (i64 o = (i64)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (i64)gridDim.x * blockDim.x) {
    const i64 g = o / n_cap;
    const int m = (int)(o - g * n_cap);
    const i64 lo = __ldg(group_offsets + g), hi = __ldg(group_offsets + g + 1);
    i64 best_item = -1;
    u64 best_score = 0;  // doubled, so that CDP's factor 1.5 stays integral
    int best_method = LLMEM_METHOD_OFFLOAD, best_batch = 0;
    for (i64 i = lo; i < hi; ++i) {
      const int b = __ldg(bs + i * n_cap + m);
      if (b <= 0) continue;  // does not fit, or not admissible: score 0
      // bytes 48..51 of the record: method, gpu_n, tp_n, lm_bytes
      const u32 w = __ldg(reinterpret_cast<const u32*>(item_cfg + i) + 12);
      const u32 method = w & 0xff, n = (w >> 8) & 0xff, t = (w >> 16) & 0xff;
      u64 score = 0;
      if (method == LLMEM_METHOD_CDP) score = 3ull * (u64)b * n;
      else if (method == LLMEM_METHOD_ADP) score = 2ull * (u64)b * n;
      else if (method == LLMEM_METHOD_TP) score = 2ull * (u64)b;
      else if (method == LLMEM_METHOD_DPTP && t > 0) score = 2ull * (u64)b * (n / t);
      if (score > best_score) {  // strict: the first of equals stays
        best_score = score;
        best_item = i;
        best_method = (int)method;
        best_batch = b;
      }
    }
    item_out[o] = best_item;
    if (method_out) method_out[o] = best_method;
    if (batch_out) batch_out[o] = best_batch;
  }
}

// ---------------------------------------------------------------------------
// llmem_chunk_search: least-waste chunk size.  One warp per configuration; lanes take
// candidates cs_min + k cs_step round-robin (one 64-bit division each) and the warp
// reduces to the smallest waste, the smaller candidate index among equals.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
chunk_search_kernel(const llmem_config* __restrict__ cfg, i64 n, i64 cs_min, i64 cs_step, int n_candidates,
                    i64* __restrict__ chunk_out, i64* __restrict__ waste_out, uint8_t* __restrict__ status_out) {
  const int lane = threadIdx.x & 31;
  const i64 warps = ((i64)gridDim.x * blockDim.x) >> 5;
  for (i64 i = ((i64)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
    Cfg f = load_cfg(cfg + i);
    f.chunk_elems = 1;  // the record's own chunk size plays no part here
    const int st = check_fields(f, false, true);
    u64 best_waste = ~0ull;
    int best_k = 0x7fffffff;
    if (st == LLMEM_CFG_OK) {
      const u64 other_p = other_params(f);
      for (int k = lane; k < n_candidates; k += 32) {
        const u64 cs = (u64)cs_min + (u64)k * (u64)cs_step;
        const u64 waste = ceil_div(other_p, cs) * cs - other_p;  // < cs <= 2^40
        if (waste < best_waste) {  // k increases: the first of equals stays
          best_waste = waste;
          best_k = k;
        }
      }
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {
        const u64 ow = __shfl_xor_sync(0xffffffffu, best_waste, d);
        const int ok = __shfl_xor_sync(0xffffffffu, best_k, d);
        if (ow < best_waste || (ow == best_waste && ok < best_k)) {
          best_waste = ow;
          best_k = ok;
        }
      }
    }
    if (lane == 0) {
      const bool ok = st == LLMEM_CFG_OK;
      chunk_out[i] = ok ? (i64)((u64)cs_min + (u64)best_k * (u64)cs_step) : -1;
      if (waste_out) waste_out[i] = ok ? (i64)best_waste : -1;
      if (status_out) status_out[i] = (uint8_t)st;
    }
  }
}

static int grid_for(i64 threads_needed, int block, int ctas_per_sm) {
  i64 blocks = (threads_needed + block - 1) / block;
  i64 cap = (i64)sm_count() * ctas_per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_estimate_batch(const llmem_config* cfg, int64_t n, int64_t* peak_out,
                                             int64_t* peak_index_out, uint8_t* status_out,
                                             void* scratch, size_t scratch_bytes, uint32_t flags,
                                             void* cuda_stream) {
  (void)scratch; (void)scratch_bytes;
  clear_error();
  TraceRange trace("llmem_estimate_batch");
  if (n < 0) { set_error("llmem_estimate_batch: n < 0"); return LLMEM_ERR_ARG; }
  if (n == 0) return LLMEM_OK;
  if (!cfg || !peak_out) { set_error("llmem_estimate_batch: cfg and peak_out are required"); return LLMEM_ERR_ARG; }
  if (!aligned_to(cfg, 16) || !aligned_to(peak_out, 8) || !aligned_to(peak_index_out, 8)) {
    set_error("llmem_estimate_batch: cfg must be 16-byte and outputs 8-byte aligned");
    return LLMEM_ERR_ARG;
  }
  const int grid = grid_for(n, LLMEM_EST_THREADS, LLMEM_EST_GRID_CTAS);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (flags & LLMEM_ESTIMATOR_DNNMEM)
    estimate_kernel<true><<<grid, LLMEM_EST_THREADS, 0, s>>>(cfg, n, reinterpret_cast<i64*>(peak_out),
                                                             reinterpret_cast<i64*>(peak_index_out), status_out);
  else
    estimate_kernel<false><<<grid, LLMEM_EST_THREADS, 0, s>>>(cfg, n, reinterpret_cast<i64*>(peak_out),
                                                              reinterpret_cast<i64*>(peak_index_out), status_out);
  return check_launch("llmem_estimate_batch");
}

static llmem_status check_search_args(const char* who, const llmem_config* shape, int64_t n,
                                      const int64_t* caps, int32_t n_cap, int32_t bmax) {
  if (n < 0 || n_cap < 0) { set_error("%s: negative size", who); return LLMEM_ERR_ARG; }
  if (bmax < 1 || bmax > (1 << 26)) { set_error("%s: bmax must be in 1 .. 2^26", who); return LLMEM_ERR_ARG; }
  if (n == 0 || n_cap == 0) return LLMEM_OK;
  if (!shape || !caps) { set_error("%s: shape and capacity_bytes are required", who); return LLMEM_ERR_ARG; }
  if (!aligned_to(shape, 16) || !aligned_to(caps, 8)) { set_error("%s: misaligned input", who); return LLMEM_ERR_ARG; }
  return LLMEM_OK;
}

extern "C" llmem_status llmem_max_batch(const llmem_config* shape, int64_t n,
                                        const int64_t* capacity_bytes, int32_t n_cap, int32_t bmax,
                                        int32_t* bs_out, uint8_t* status_out, void* scratch,
                                        size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  (void)scratch; (void)scratch_bytes;
  clear_error();
  TraceRange trace("llmem_max_batch");
  if (flags & LLMEM_ESTIMATOR_DNNMEM) { set_error("llmem_max_batch: Algorithm 1 searches with the LLMem estimate only"); return LLMEM_ERR_ARG; }
  llmem_status st = check_search_args("llmem_max_batch", shape, n, capacity_bytes, n_cap, bmax);
  if (st != LLMEM_OK || n == 0 || n_cap == 0) return st;
  if (!bs_out || !aligned_to(bs_out, 4)) { set_error("llmem_max_batch: bs_out is required"); return LLMEM_ERR_ARG; }
  max_batch_kernel<<<grid_for(n, 256, LLMEM_SEARCH_GRID_CTAS), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      shape, n, reinterpret_cast<const i64*>(capacity_bytes), n_cap, bmax, (kSat - 1) / (u64)bmax, bs_out, status_out);
  return check_launch("llmem_max_batch");
}

extern "C" llmem_status llmem_select_method(const llmem_config* shape, int64_t n,
                                            const int64_t* capacity_bytes, int32_t n_cap,
                                            int32_t bmax, int32_t* method_out, int32_t* batch_out,
                                            int32_t* bs_list_out, uint8_t* status_out, void* scratch,
                                            size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  (void)scratch; (void)scratch_bytes;
  clear_error();
  TraceRange trace("llmem_select_method");
  if (flags & LLMEM_ESTIMATOR_DNNMEM) { set_error("llmem_select_method: Algorithm 1 selects with the LLMem estimate only"); return LLMEM_ERR_ARG; }
  llmem_status st = check_search_args("llmem_select_method", shape, n, capacity_bytes, n_cap, bmax);
  if (st != LLMEM_OK || n == 0 || n_cap == 0) return st;
  if (!method_out || !batch_out) { set_error("llmem_select_method: method_out and batch_out are required"); return LLMEM_ERR_ARG; }
  select_kernel<<<grid_for(4 * n, 256, LLMEM_SEARCH_GRID_CTAS), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      shape, n, reinterpret_cast<const i64*>(capacity_bytes), n_cap, bmax, (kSat - 1) / (u64)bmax, flags, method_out,
      batch_out, bs_list_out, status_out);
  return check_launch("llmem_select_method");
}

extern "C" llmem_status llmem_select_segmented(const llmem_config* item_cfg, const int32_t* bs,
                                               const int64_t* group_offsets, int64_t n_groups,
                                               int64_t n_items, int32_t n_cap, int64_t* item_out,
                                               int32_t* method_out, int32_t* batch_out, void* scratch,
                                               size_t scratch_bytes, uint32_t flags, void* cuda_stream) {
  (void)scratch; (void)scratch_bytes; (void)flags;
  clear_error();
  TraceRange trace("llmem_select_segmented");
  if (n_groups < 0 || n_items < 0 || n_cap < 0) { set_error("llmem_select_segmented: negative size"); return LLMEM_ERR_ARG; }
  if (n_groups == 0 || n_cap == 0) return LLMEM_OK;
  if (!group_offsets || !item_out || (n_items > 0 && (!item_cfg || !bs))) {
    set_error("llmem_select_segmented: item_cfg, bs, group_offsets and item_out are required");
    return LLMEM_ERR_ARG;
  }
  if (!aligned_to(item_cfg, 16) || !aligned_to(bs, 4) || !aligned_to(group_offsets, 8) || !aligned_to(item_out, 8)) {
    set_error("llmem_select_segmented: misaligned pointer");
    return LLMEM_ERR_ARG;
  }
  select_segmented_kernel<<<grid_for(n_groups * n_cap, 256, 8), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      item_cfg, bs, reinterpret_cast<const i64*>(group_offsets), n_groups, n_cap,
      reinterpret_cast<i64*>(item_out), method_out, batch_out);
  return check_launch("llmem_select_segmented");
}

extern "C" llmem_status llmem_chunk_search(const llmem_config* cfg, int64_t n, int64_t cs_min, int64_t cs_step,
                                           int32_t n_candidates, int64_t* chunk_out, int64_t* waste_out,
                                           uint8_t* status_out, void* scratch, size_t scratch_bytes,
                                           uint32_t flags, void* cuda_stream) {
  (void)scratch; (void)scratch_bytes; (void)flags;
  clear_error();
  TraceRange trace("llmem_chunk_search");
  if (n < 0) { set_error("llmem_chunk_search: n < 0"); return LLMEM_ERR_ARG; }
  if (cs_min < 1 || cs_step < 1 || n_candidates < 1 ||
      cs_min > (1ll << 40) || cs_step > (1ll << 40) ||
      (int64_t)(n_candidates - 1) > ((1ll << 40) - cs_min) / cs_step) {  // no product: it could wrap
    set_error("llmem_chunk_search: candidates must be cs_min + k cs_step in 1 .. 2^40, k < n_candidates");
    return LLMEM_ERR_ARG;
  }
  if (n == 0) return LLMEM_OK;
  if (!cfg || !chunk_out || !aligned_to(cfg, 16) || !aligned_to(chunk_out, 8) || !aligned_to(waste_out, 8)) {
    set_error("llmem_chunk_search: cfg (16-byte aligned) and chunk_out are required");
    return LLMEM_ERR_ARG;
  }
  chunk_search_kernel<<<grid_for(32 * n, 256, 8), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      cfg, n, cs_min, cs_step, n_candidates, reinterpret_cast<i64*>(chunk_out), reinterpret_cast<i64*>(waste_out),
      status_out);
  return check_launch("llmem_chunk_search");
}
