// Event expansion shared by the kernels that materialise event lists: launch shape,
// the run-table description of one configuration's list (Sections 4.1 and 5 phase order),
// the per-lane run cursor, and the TMA bulk-store primitives.
#pragma once

#include "llmem_model.cuh"

namespace llmem {

// Launch shape (overridable at compile time for tuning sweeps).
#ifndef LLMEM_EXP_THREADS
#define LLMEM_EXP_THREADS 384
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
// Blocks of work per resident warp of the expansion kernel and the fewest chunks a block
// is given (ranges.cuh).
#ifndef LLMEM_EXP_OVERSUB
#define LLMEM_EXP_OVERSUB 36
#endif
#ifndef LLMEM_EXP_MIN_CHUNKS
#define LLMEM_EXP_MIN_CHUNKS 128
#endif
// Bulk stores a warp may have in flight from buffers it is not rewriting.
#ifndef LLMEM_EXP_INFLIGHT
#define LLMEM_EXP_INFLIGHT 8
#endif
constexpr int kExpStoresInFlight = LLMEM_EXP_INFLIGHT;
constexpr int kRuns = 16;
constexpr int kDynFirst = 2, kDynLast = 13, kOsFirst = 14, kOsLast = 15;  // run indices, see SegDesc

// A run of events that repeat with a short period (at most 16): position j of a period
// has value v[(code >> 2j) & 3].  Constant runs use period 1 and code 0.
struct alignas(16) Run {
  int cnt, period;
  u32 code;
  int start;  // events of the same group (initialisation / one iteration / optimizer states) before this run
  i64 a, b, c;
  i64 links;  // byte 0: the next non-empty run during the first iteration, byte 1: during later ones
};

// The event list of one configuration as runs.  Order: 0-1 initialisation (embedding unit,
// chunks); 2-13 one iteration (gathered embedding unit, gathered chunks, embedding and layer
// outputs, per-layer operator outputs, logits with the two shifted copies, TP buffers, then
// the frees mirrored); 14-15 optimizer states (embedding tensors, layer tensors), which
// follow the first iteration only.  Neighbouring events of equal size share a run, and the
// logits and their two copies form one run of period 3, so that a list has few runs.
struct SegDesc {
  i64 first_part;  // where the parts of a long segment start in the list of parts (-1: not cut into parts)
  i64 reserved;
  u32 init_n, dyn_n, os_n;
  int invalid;
  Run run[kRuns];
};

__device__ __forceinline__ void set_run(Run& r, int cnt, int period, u32 code, i64 a, i64 b, i64 c) {
  r.cnt = cnt; r.period = period; r.code = code; r.start = 0; r.a = a; r.b = b; r.c = c; r.links = 0;
}
__device__ __forceinline__ void set_const_run(Run& r, int cnt, i64 a) { set_run(r, cnt, 1, 0u, a, a, a); }

// 2-bit value selectors of the operator outputs of one layer in forward order
// (0 hidden-sized, 1 attention-score sized, 2 feed-forward sized): norm, q, k, v, scores,
// softmax, context, o-proj, residual, norm, up [x2, product], activation, down, residual.
__device__ __forceinline__ u32 layer_code(bool gated, bool reversed, int* n_ops) {
  const int n = gated ? 16 : 14;
  *n_ops = n;
  u32 code = 0;
  for (int k = 0; k < n; ++k) {
    const int kind = (k == 4 || k == 5) ? 1 : ((k >= 10 && k < n - 2) ? 2 : 0);
    const int pos = reversed ? n - 1 - k : k;
    code |= (u32)kind << (2 * pos);
  }
  return code;
}

// Not inlined: the kernels reach it from two places, and the warps of an SM, each somewhere
// else in a long kernel, already miss the instruction cache more than anything else
// ("no instruction" is the top stall on lists of short segments).
// Fills in where each run starts inside its group and which run follows it.
__device__ __forceinline__ void link_runs(SegDesc& d) {
  d.run[1].start = 2;
  for (int r = kDynFirst + 1; r <= kDynLast; ++r) d.run[r].start = d.run[r - 1].start + d.run[r - 1].cnt;
  for (int r = kOsFirst + 1; r <= kOsLast; ++r) d.run[r].start = d.run[r - 1].start + d.run[r - 1].cnt;
  // in the first iteration the optimizer states follow the frees
  for (int r = 0; r < kRuns; ++r) {
    i64 links = 0;
    for (int later = 0; later < 2; ++later) {
      int nx = r;
      for (int guard = 0; guard < 2 * kRuns; ++guard) {
        if (nx == kDynLast) nx = later ? kDynFirst : kOsFirst;
        else if (nx == kOsLast) nx = kDynFirst;
        else ++nx;
        if (d.run[nx].cnt > 0) break;
      }
      links |= (i64)nx << (8 * later);
    }
    d.run[r].links = links;
  }
}

// The list of the DNNMem-style estimator (Section 3.1) in the same form: runs 0-1 the buffer
// with the token embedding, then the position embedding; the "iteration" group holds the
// Linear matrices, the vectors, the final norm, the lm_head and the forward outputs, and is
// passed once; there are no optimizer states and no frees.  `f` has passed check_fields.
__device__ __forceinline__ void build_dnn_runs(SegDesc& d, const Cfg& f, bool round) {
  const DnnPlan p = make_dnn_plan(f);
  if (p.status != LLMEM_CFG_OK) return;
  if (p.out >= kSat || p.logit >= kSat || p.shift >= kSat || p.attn >= kSat || p.ffn >= kSat) return;
  d.invalid = 0;
#define LLMEM_W(x) ((i64)(round ? align512(x) : (x)))
  const int L = p.L;
  set_run(d.run[0], 2, 2, 1u << 2, (i64)kDnnBuffer, LLMEM_W(p.tok), 0);
  set_const_run(d.run[1], p.has_pos, LLMEM_W(p.pos));
  set_run(d.run[2], p.K * L, p.K, p.K == 7 ? 0x1500u : 0x0500u, LLMEM_W(p.hh), LLMEM_W(p.hf), 0);
  if (p.wide > 0) {
    // per layer: `small` vectors of the hidden size, then `wide` of the feed-forward size
    u32 code = 0;
    for (int k = p.small; k < p.small + p.wide; ++k) code |= 1u << (2 * k);
    set_run(d.run[3], (p.small + p.wide) * L, p.small + p.wide, code, LLMEM_W(p.vec_h), LLMEM_W(p.vec_f), 0);
  } else {
    set_const_run(d.run[3], p.small * L, LLMEM_W(p.vec_h));
  }
  set_const_run(d.run[4], p.final_n, LLMEM_W(p.vec_h));
  set_const_run(d.run[5], 1, LLMEM_W(p.lm));
  int n_ops = 1;
  u32 fwd = 0;
  if (f.act_mode) fwd = layer_code(f.ffn_kind != 0, false, &n_ops);
  const i64 out = LLMEM_W(p.out);
  set_const_run(d.run[6], p.e_n + (f.act_mode ? 0 : L), out);
  set_run(d.run[7], f.act_mode ? L * n_ops : 0, n_ops, fwd, out, LLMEM_W(p.attn), LLMEM_W(p.ffn));
  set_run(d.run[8], 3, 3, 0x14u, LLMEM_W(p.logit), LLMEM_W(p.shift), 0);  // logits, shifted copy, shifted copy
  for (int r = 9; r < kRuns; ++r) set_const_run(d.run[r], 0, 0);
#undef LLMEM_W
  link_runs(d);
  d.init_n = 2u + (u32)p.has_pos;
  d.dyn_n = (u32)(p.count - d.init_n);
  d.os_n = 0;
}

static __device__ __noinline__ void build_desc(SegDesc& d, const llmem_config* __restrict__ cfg, i64 gstart, i64 gend,
                                               bool round, bool dnn = false) {
  d.first_part = -1;
  d.reserved = 0;
  d.invalid = 1;
  d.init_n = d.dyn_n = d.os_n = 0;
  if (gend <= gstart) return;
  Cfg f = load_cfg(cfg);
  if (check_fields(f, true, true) != LLMEM_CFG_OK) return;
  if (dnn) {
    build_dnn_runs(d, f, round);
    return;
  }
  Plan p = make_plan(f, f.method);
  if (p.status != LLMEM_CFG_OK) return;
  Dyn y = make_dyn(p, (u64)f.batch);
  if (y.out >= kSat || y.logit >= kSat || y.shift >= kSat || y.attn >= kSat || y.ffn >= kSat) return;
  d.invalid = 0;
#define LLMEM_V(x) ((i64)(round ? page_round(x) : (x)))
  const int C = (int)p.C, L = p.L;
  const int G = p.gather ? 1 : 0, T = p.tpback ? 1 : 0;
  set_run(d.run[0], 2, 2, 1u << 2, LLMEM_V(p.p16_embed), LLMEM_V(p.p32_embed), 0);
  set_run(d.run[1], 2 * C, 2, 1u << 2, LLMEM_V(p.p16_chunk), LLMEM_V(p.p32_chunk), 0);
  const i64 ge = LLMEM_V(p.gat_embed), gc = LLMEM_V(p.gat_chunk), out = LLMEM_V(y.out);
  const i64 lg = LLMEM_V(y.logit), sh = LLMEM_V(y.shift), bk = LLMEM_V(y.back);
  const i64 at = LLMEM_V(y.attn), ff = LLMEM_V(y.ffn);
  int n_ops = 1;
  u32 fwd = 0, bwd = 0;
  if (f.act_mode) {
    fwd = layer_code(f.ffn_kind != 0, false, &n_ops);
    bwd = layer_code(f.ffn_kind != 0, true, &n_ops);
  }
  // with gradient checkpointing a layer keeps one output of the size of an embedding output:
  // one run; otherwise the layers' operator outputs form a periodic run of their own
  const int plain_layers = f.act_mode ? 0 : L;
  set_const_run(d.run[2], G, ge);
  set_const_run(d.run[3], G * C, gc);
  set_const_run(d.run[4], p.e_n + plain_layers, out);
  set_run(d.run[5], f.act_mode ? L * n_ops : 0, n_ops, fwd, out, at, ff);
  set_run(d.run[6], 3, 3, 0x14u, lg, sh, 0);     // logits, shifted copy, shifted copy
  set_const_run(d.run[7], T * L, bk);
  set_const_run(d.run[8], T * L, -bk);
  set_run(d.run[9], 3, 3, 0x05u, -lg, -sh, 0);   // the copies, then the logits
  set_run(d.run[10], f.act_mode ? L * n_ops : 0, n_ops, bwd, -out, -at, -ff);
  set_const_run(d.run[11], p.e_n + plain_layers, -out);
  set_const_run(d.run[12], G * C, -gc);
  set_const_run(d.run[13], G, -ge);
  // token embedding states, then those of the position embedding if there is one
  set_run(d.run[14], f.pos_len > 0 ? 2 : 1, 2, 1u << 2, LLMEM_V(p.os_tok), LLMEM_V(p.os_pos), 0);
  // per layer: four H x H tensors, then the feed-forward ones
  set_run(d.run[15], p.K * L, p.K, p.K == 7 ? 0x1500u : 0x0500u, LLMEM_V(p.os_hh), LLMEM_V(p.os_hf), 0);
#undef LLMEM_V
  link_runs(d);
  d.init_n = 2u + 2u * (u32)C;
  const u32 allocs = (u32)(G * (1 + C) + p.e_n + L * n_ops + 3 + T * L);
  d.dyn_n = 2 * allocs;
  d.os_n = (u32)(p.e_n + p.K * L);
}

// Cursor of one thread inside a segment.
struct Cursor {
  int r, it, rem, phase, period;
  u32 code;
  i64 a, b, c;
  __device__ __forceinline__ i64 value(int ph) const {
    const u32 k = (code >> (2 * ph)) & 3u;
    return k == 0 ? a : (k == 1 ? b : c);
  }
};

__device__ __forceinline__ void enter_run(Cursor& c, const SegDesc& d, int r, int o) {
  const Run& rn = d.run[r];
  c.r = r;
  c.rem = rn.cnt - o;
  c.period = rn.period;
  c.code = rn.code;
  c.a = rn.a;
  c.b = rn.b;
  c.c = rn.c;
  c.phase = rn.period == 1 ? 0 : (rn.period == 2 ? (o & 1) : (int)((u32)o % (u32)rn.period));
}

// Run, offset inside it and iteration of event `pos` (0-based inside the segment).
__device__ __forceinline__ void locate(const SegDesc& d, u32 pos, int* r_out, int* o_out, int* it_out) {
  *it_out = 1;
  if (pos < d.init_n) {
    *r_out = pos < 2 ? 0 : 1;
    *o_out = pos < 2 ? (int)pos : (int)(pos - 2);
    return;
  }
  u32 q = pos - d.init_n;
  int r = kDynFirst;
  if (q >= d.dyn_n) {
    q -= d.dyn_n;
    if (q < d.os_n) {
      r = kOsFirst;
    } else {
      q -= d.os_n;
      *it_out = 2 + (int)(q / d.dyn_n);
      q = q % d.dyn_n;
    }
  }
  while (r < kRuns - 1 && q >= (u32)d.run[r].cnt) {
    q -= (u32)d.run[r].cnt;
    ++r;
  }
  *r_out = r;
  *o_out = (int)q;
}

// Position the cursor on event `pos`.
__device__ __forceinline__ void seek(Cursor& c, const SegDesc& d, u32 pos) {
  int r, o;
  locate(d, pos, &r, &o, &c.it);
  enter_run(c, d, r, o);
}

// Move to the next non-empty run.  After the frees of iteration 1 come the optimizer
// states; after them, and after the frees of every later iteration, the next iteration.
__device__ __forceinline__ void next_run(Cursor& c, const SegDesc& d) {
  int r = c.r;
  for (int guard = 0; guard < 2 * kRuns; ++guard) {
    if (r == kDynLast) {
      if (c.it == 1) r = kOsFirst;
      else { r = kDynFirst; ++c.it; }
    } else if (r == kOsLast) {
      r = kDynFirst;
      c.it = 2;
    } else {
      ++r;
    }
    if (d.run[r].cnt > 0) break;
  }
  enter_run(c, d, r, 0);
}

__device__ __forceinline__ i64 emit(Cursor& c, const SegDesc& d) {
  const i64 v = c.value(c.phase);
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
static_assert(sizeof(SegDesc) % 16 == 0, "descriptors are copied in 16-byte words");
struct ExpandWarpSmem {
  alignas(128) i64 buf[2][kExpChunk];
  SegDesc desc;
};

// ---- chunks that repeat -------------------------------------------------------------------
// A full chunk inside one run of equal events, or of two alternating ones, repeats the chunk
// issued from the same buffer two chunks earlier.  AlternatingRun remembers the run the last
// such chunk lay in; BufferKeys what pattern each of the warp's two chunk buffers holds.
struct AlternatingRun {
  i64 end = -1;  // chunks that end at or before this list index repeat the pattern
  i64 key = -1;  // (segment, run, phase): identifies the pattern
  i64 x0 = 0, x1 = 0;  // the value on even / odd positions of a chunk
};

struct BufferKeys {
  i64 key0 = -1, key1 = -1;
  __device__ __forceinline__ i64 get(int parity) const { return parity ? key1 : key0; }
  __device__ __forceinline__ void set(int parity, i64 k) {
    if (parity) key1 = k;
    else key0 = k;
  }
};

// Makes sure the warp's descriptor is that of segment `seg` (range [gs, ge)): built by lane 0
// when the warp enters the segment.
__device__ __forceinline__ void ensure_desc(ExpandWarpSmem& ws, i64& desc_seg, const llmem_config* __restrict__ cfg,
                                            i64 seg, i64 gs, i64 ge, int round /* bit 0: rounded values, bit 1: second estimator */,
                                            int lane, const Guard& g) {
  if (desc_seg != seg) {
    __syncwarp();  // every lane is done with the previous descriptor
    if (lane == 0) {
      if (in_bounds(seg >= 0 && seg < g.n, g, kSiteDescriptor)) build_desc(ws.desc, cfg + seg, gs, ge, (round & 1) != 0, (round & 2) != 0);
      else ws.desc.invalid = 1;  // the segment is written as zeros
    }
    __syncwarp();
    desc_seg = seg;
  }
}

// Does the full chunk [tb, tb + kExpChunk), which lies inside segment `seg`, consist of one
// run of period 1 or 2?  Updates `ar` when it enters a new such run.
__device__ __forceinline__ bool chunk_alternates(AlternatingRun& ar, ExpandWarpSmem& ws, i64& desc_seg,
                                                 const llmem_config* __restrict__ cfg, i64 seg, i64 gs, i64 ge, i64 tb,
                                                 int round, int lane, const Guard& g) {
  if (tb + kExpChunk <= ar.end) return true;
  ensure_desc(ws, desc_seg, cfg, seg, gs, ge, round, lane, g);
  if (ws.desc.invalid) return false;
  int r, o, it;
  locate(ws.desc, (u32)(tb - gs), &r, &o, &it);
  const Run& rn = ws.desc.run[r];
  if (rn.cnt - o < kExpChunk || rn.period > 2) return false;
  // period 1: a everywhere; period 2: a on even offsets of the run, b on odd ones
  const bool odd = rn.period == 2 && (o & 1);
  ar.x0 = odd ? rn.b : rn.a;
  ar.x1 = rn.period == 2 ? (odd ? rn.a : rn.b) : rn.a;
  ar.end = tb + (rn.cnt - o);
  ar.key = (seg << 8) | (i64)(r << 1) | (odd ? 1 : 0);
  return true;
}

// Gets buffer `parity` ready for an alternating chunk: nothing to do if it already holds the
// pattern (only the number of stores in flight is bounded); otherwise the bulk store issued
// from it two chunks ago must have read it, then every lane writes its span (an even offset:
// x0 comes first).
template <int kStoresInFlight>
__device__ __forceinline__ void prepare_alternating(const AlternatingRun& ar, BufferKeys& keys, int parity,
                                                    i64* __restrict__ buf, int lane) {
  if (keys.get(parity) != ar.key) {
    if (lane == 0) bulk_wait_read<1>();
    __syncwarp();
    longlong2* v = reinterpret_cast<longlong2*>(buf + lane * kExpPerLane);
#pragma unroll
    for (int j = 0; j < kExpPerLane / 2; ++j) v[j] = make_longlong2(ar.x0, ar.x1);
    keys.set(parity, ar.key);
    fence_async_shared();
    __syncwarp();
  } else if (lane == 0) {
    bulk_wait_read<kStoresInFlight>();
  }
}

// Hands chunk [tb, tb + cnt) to the TMA engine (or copies it with plain stores when the
// output is not 16-byte aligned).
__device__ __forceinline__ void store_chunk(i64* __restrict__ out, i64 tb, u32 cnt, const i64* __restrict__ buf,
                                            int bulk_ok, int lane, const Guard& g) {
  if (!in_bounds(tb >= 0 && cnt <= (u32)kExpChunk && tb + (i64)cnt <= g.total, g, kSiteStore)) return;
  if (bulk_ok) {
    if (lane == 0) {
      const u32 even = cnt & ~1u;
      if (even) bulk_store(out + tb, buf, even * 8u);
      bulk_commit();
      if (cnt & 1u) out[tb + cnt - 1] = buf[cnt - 1];
    }
  } else {
    for (u32 i = lane; i < cnt; i += 32) out[tb + i] = buf[i];
    __syncwarp();  // the buffer may be rewritten two chunks from now
  }
}

// Write `cnt` events starting at segment position `pos` to dst[0 .. cnt).  Spans that
// stay inside one run of period 1 or 2 (parameter chunks, gathers, outputs: almost
// all of a long list) are written as constants; anything else goes through the
// run cursor event by event.
__device__ __forceinline__ void fill_span(i64* __restrict__ dst, const SegDesc& d, u32 pos, int cnt) {
  int r, o, it;
  locate(d, pos, &r, &o, &it);
  const Run& rn = d.run[r];
  if (rn.cnt - o >= cnt && rn.period <= 2) {
    // period 1: a everywhere; period 2: a on even offsets of the run, b on odd ones
    const bool odd = rn.period == 2 && (o & 1);
    const i64 x0 = odd ? rn.b : rn.a;
    const i64 x1 = rn.period == 2 ? (odd ? rn.a : rn.b) : rn.a;
    if (cnt == kExpPerLane && (smem_addr(dst) & 15u) == 0) {
      longlong2* v = reinterpret_cast<longlong2*>(dst);
#pragma unroll
      for (int j = 0; j < kExpPerLane / 2; ++j) v[j] = make_longlong2(x0, x1);
    } else {
      for (int j = 0; j < cnt; ++j) dst[j] = (j & 1) ? x1 : x0;
    }
    return;
  }
  Cursor c;
  c.it = it;
  enter_run(c, d, r, o);
  for (int j = 0; j < cnt; ++j) dst[j] = emit(c, d);
}

}  // namespace llmem
