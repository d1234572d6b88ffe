// Event expansion shared by the kernels that materialise event lists: launch shape,
// the run-table description of one configuration's list (Sections 4.1 and 5 phase order),
// the per-lane run cursor, and the TMA bulk-store primitives.
#pragma once

#include "llmem_model.cuh"

namespace llmem {

// Launch shape (overridable at compile time for tuning sweeps).
#ifndef LLMEM_EXP_THREADS
#define LLMEM_EXP_THREADS 256
#endif
#ifndef LLMEM_EXP_PER_LANE
#define LLMEM_EXP_PER_LANE 18
#endif
#ifndef LLMEM_EXP_CTAS_PER_SM
#define LLMEM_EXP_CTAS_PER_SM 1
#endif
constexpr int kExpThreads = LLMEM_EXP_THREADS;
constexpr int kExpWarps = kExpThreads / 32;
// 18 events = 144 bytes = nine 16-byte words per lane: an odd word count makes
// the per-lane spans fall on distinct shared-memory banks.
constexpr int kExpPerLane = LLMEM_EXP_PER_LANE;
constexpr int kExpChunk = 32 * kExpPerLane;  // 576 events, 4608 bytes: one warp's unit of work
constexpr int kExpCtasPerSm = LLMEM_EXP_CTAS_PER_SM;
static_assert(kExpPerLane % 2 == 0 && (kExpPerLane / 2) % 2 == 1, "per-lane span: odd number of 16-byte words");
// What a segment boundary costs the expansion, in events (descriptor build, cursor seeks):
// the kappa of the cost-balanced work split.
#ifndef LLMEM_EXP_SEGMENT_COST
#define LLMEM_EXP_SEGMENT_COST 6144
#endif
constexpr i64 kExpSegmentCost = LLMEM_EXP_SEGMENT_COST;
constexpr int kRuns = 17;

// A run of events that repeat with a short period: the first `split` events of each
// period have value a, the others b.  Constant runs use period 1.
struct Run {
  int cnt, period, split, pad;
  i64 a, b;
};

// The event list of one configuration as runs.  Order: 0-1 initialisation,
// 2-13 one iteration (allocations, then frees mirrored), 14-16 optimizer states,
// which follow the first iteration only.
struct SegDesc {
  i64 gstart, gend;  // global event range of the segment
  u32 init_n, dyn_n, os_n;
  int invalid;
  Run run[kRuns];
};

__device__ __forceinline__ void set_run(Run& r, int cnt, int period, int split, i64 a, i64 b) {
  r.cnt = cnt; r.period = period; r.split = split; r.pad = 0; r.a = a; r.b = b;
}

__device__ inline void build_desc(SegDesc& d, const llmem_config* __restrict__ cfg, i64 gstart, i64 gend, bool round) {
  d.gstart = gstart;
  d.gend = gend;
  d.invalid = 1;
  d.init_n = d.dyn_n = d.os_n = 0;
  if (gend <= gstart) return;
  Cfg f = load_cfg(cfg);
  if (check_fields(f, true, true) != LLMEM_CFG_OK) return;
  Plan p = make_plan(f, f.method);
  if (p.status != LLMEM_CFG_OK) return;
  Dyn y = make_dyn(p, (u64)f.batch);
  if (y.out >= kSat || y.logit >= kSat || y.shift >= kSat) return;
  d.invalid = 0;
#define LLMEM_V(x) ((i64)(round ? page_round(x) : (x)))
  const int C = (int)p.C, L = p.L;
  const int G = p.gather ? 1 : 0, T = p.tpback ? 1 : 0;
  set_run(d.run[0], 2, 2, 1, LLMEM_V(p.p16_embed), LLMEM_V(p.p32_embed));
  set_run(d.run[1], 2 * C, 2, 1, LLMEM_V(p.p16_chunk), LLMEM_V(p.p32_chunk));
  const i64 ge = LLMEM_V(p.gat_embed), gc = LLMEM_V(p.gat_chunk), out = LLMEM_V(y.out);
  const i64 lg = LLMEM_V(y.logit), sh = LLMEM_V(y.shift), bk = LLMEM_V(y.back);
  set_run(d.run[2], G, 1, 1, ge, ge);
  set_run(d.run[3], G * C, 1, 1, gc, gc);
  set_run(d.run[4], p.e_n + L, 1, 1, out, out);
  set_run(d.run[5], 1, 1, 1, lg, lg);
  set_run(d.run[6], 2, 1, 1, sh, sh);
  set_run(d.run[7], T * L, 1, 1, bk, bk);
  set_run(d.run[8], T * L, 1, 1, -bk, -bk);
  set_run(d.run[9], 2, 1, 1, -sh, -sh);
  set_run(d.run[10], 1, 1, 1, -lg, -lg);
  set_run(d.run[11], p.e_n + L, 1, 1, -out, -out);
  set_run(d.run[12], G * C, 1, 1, -gc, -gc);
  set_run(d.run[13], G, 1, 1, -ge, -ge);
  const i64 ot = LLMEM_V(p.os_tok), op = LLMEM_V(p.os_pos);
  set_run(d.run[14], 1, 1, 1, ot, ot);
  set_run(d.run[15], f.pos_len > 0 ? 1 : 0, 1, 1, op, op);
  set_run(d.run[16], p.K * L, p.K, 4, LLMEM_V(p.os_hh), LLMEM_V(p.os_hf));
#undef LLMEM_V
  d.init_n = 2u + 2u * (u32)C;
  const u32 allocs = (u32)(G * (1 + C) + p.e_n + L + 3 + T * L);
  d.dyn_n = 2 * allocs;
  d.os_n = (u32)(p.e_n + p.K * L);
}

// Cursor of one thread inside a segment.
struct Cursor {
  int r, it, rem, phase, period, split;
  i64 a, b;
};

__device__ __forceinline__ void enter_run(Cursor& c, const SegDesc& d, int r, int o) {
  const Run& rn = d.run[r];
  c.r = r;
  c.rem = rn.cnt - o;
  c.period = rn.period;
  c.split = rn.split;
  c.a = rn.a;
  c.b = rn.b;
  c.phase = rn.period == 1 ? 0 : (rn.period == 2 ? (o & 1) : (int)((u32)o % (u32)rn.period));
}

// Position the cursor on event `pos` (0-based inside the segment).
__device__ __forceinline__ void seek(Cursor& c, const SegDesc& d, u32 pos) {
  c.it = 1;
  if (pos < d.init_n) {
    if (pos < 2) enter_run(c, d, 0, (int)pos);
    else enter_run(c, d, 1, (int)(pos - 2));
    return;
  }
  u32 q = pos - d.init_n;
  int r = 2;
  if (q >= d.dyn_n) {
    q -= d.dyn_n;
    if (q < d.os_n) {
      r = 14;
    } else {
      q -= d.os_n;
      c.it = 2 + (int)(q / d.dyn_n);
      q = q % d.dyn_n;
    }
  }
  while (r < kRuns - 1 && q >= (u32)d.run[r].cnt) {
    q -= (u32)d.run[r].cnt;
    ++r;
  }
  enter_run(c, d, r, (int)q);
}

// Move to the next non-empty run.  After the frees of iteration 1 come the optimizer
// states; after them, and after the frees of every later iteration, the next iteration.
__device__ __forceinline__ void next_run(Cursor& c, const SegDesc& d) {
  int r = c.r;
  for (int guard = 0; guard < 2 * kRuns; ++guard) {
    if (r == 13) {
      if (c.it == 1) r = 14;
      else { r = 2; ++c.it; }
    } else if (r == 16) {
      r = 2;
      c.it = 2;
    } else {
      ++r;
    }
    if (d.run[r].cnt > 0) break;
  }
  enter_run(c, d, r, 0);
}

__device__ __forceinline__ i64 emit(Cursor& c, const SegDesc& d) {
  const i64 v = c.phase < c.split ? c.a : c.b;
  if (++c.phase == c.period) c.phase = 0;
  if (--c.rem == 0) next_run(c, d);
  return v;
}

__device__ __forceinline__ u32 smem_addr(const void* p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, u32 bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(gdst),
               "r"(smem_addr(ssrc)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// One warp's private shared memory: two chunk buffers (filled, then handed to the
// TMA engine while the other one is being filled) and the descriptor of the
// segment the warp is currently inside.
struct ExpandWarpSmem {
  alignas(128) i64 buf[2][kExpChunk];
  SegDesc desc;
};

// Write `cnt` events starting at segment position `pos` to dst[0 .. cnt).  Spans that
// stay inside one run of period 1 or 2 (parameter chunks, gathers, outputs: almost
// all of a long list) are written as constants; anything else goes through the
// run cursor event by event.
__device__ __forceinline__ void fill_span(i64* __restrict__ dst, const SegDesc& d, u32 pos, int cnt) {
  Cursor c;
  seek(c, d, pos);
  if (c.rem >= cnt && c.period <= 2) {
    const i64 x0 = c.phase < c.split ? c.a : c.b;
    const i64 x1 = c.period == 1 ? x0 : (c.phase < c.split ? c.b : c.a);
    if (cnt == kExpPerLane && (smem_addr(dst) & 15u) == 0) {
      longlong2* v = reinterpret_cast<longlong2*>(dst);
#pragma unroll
      for (int j = 0; j < kExpPerLane / 2; ++j) v[j] = make_longlong2(x0, x1);
    } else {
      for (int j = 0; j < cnt; ++j) dst[j] = (j & 1) ? x1 : x0;
    }
    return;
  }
  for (int j = 0; j < cnt; ++j) dst[j] = emit(c, d);
}

}  // namespace llmem
