// Device-side memory model shared by every kernel of the library: configuration
// checks, parameter inventory (Table 1 of the paper), raw event sizes per method
// (Sections 4.1, 4.2 and 5) and the per-phase sums used by the fused kernels.
//
// All arithmetic is unsigned 64-bit and saturates at 2^62: every quantity is a
// sum or product of non-negative terms, so "the exact value is >= 2^62" and "the
// saturating value is 2^62" are the same statement, which is how the overflow
// status is decided without wider integers.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/llmem.h"

namespace llmem {

typedef unsigned long long u64;
typedef long long i64;
typedef unsigned int u32;

constexpr u64 kPage = 2ull * 1024ull * 1024ull;  // cu_p, Section 4.2
constexpr u64 kSat = 1ull << 62;                 // bytes limit (exclusive)
constexpr u64 kCountLimit = 1ull << 31;          // events limit (exclusive)

// Checked builds (-DLLMEM_DEBUG, csrc/libllmem_debug.so): the streaming kernels test every
// index they derive from offsets, block numbers and segment numbers before using it.  A
// failed test records 16 + its site number in the scratch status word (the largest one wins)
// and the access is skipped; nothing traps.  In normal builds in_bounds() is the constant
// true and the tests cost nothing.
#ifdef LLMEM_DEBUG
constexpr bool kChecked = true;
#else
constexpr bool kChecked = false;
#endif
constexpr u32 kCheckBase = 16;  // status words from here on name a failed check

struct Guard {
  u32* word;  // scratch status word, or null
  i64 n;      // configurations
  i64 total;  // events
};

enum CheckSite : u32 { kSiteStore = 1, kSiteDescriptor = 2, kSiteBlock = 3, kSiteResult = 4, kSiteLoad = 5, kSiteFill = 6 };

__device__ __forceinline__ bool in_bounds(bool ok, const Guard& g, u32 site) {
  if (kChecked && !ok) {
    if (g.word) atomicMax(g.word, kCheckBase + site);
    return false;
  }
  return true;
}

__host__ __device__ __forceinline__ u64 sat_add(u64 a, u64 b) {
  u64 s = a + b;  // a, b <= 2^62: no wrap
  return s > kSat ? kSat : s;
}

// Saturating a * b (b <= 2^62) for a 32-bit factor, which every product of the model has
// (a count, a batch, a sequence length): two widening multiplies instead of a 64 x 64 product.
__device__ __forceinline__ u64 sat_mul_u32(u32 a, u64 b) {
  const u64 lo = (u64)a * (u32)b;          // a * (low half of b)
  const u64 hi = (u64)a * (u32)(b >> 32);  // a * (high half of b), to be shifted by 32
  const u64 t = lo + (hi << 32);
  return (hi >= (1ull << 30) || t < lo || t >= kSat) ? kSat : t;
}

// The model's sums and products under two policies.  SatMath clamps every result at 2^62, so
// a value can be carried on and compared (the searches do).  StickyMath computes the plain
// 64-bit result and only remembers whether some result reached 2^62: every quantity is
// non-negative and enters the peak, so "some result reached 2^62" and "the peak reached 2^62"
// are the same statement, and where the peak is all that is asked for the clamps (two
// compares and two selects per operation) shrink to one OR.  Operands must be exact (below
// 2^62) or follow a result that has already been recorded as too large.
struct SatMath {
  __device__ __forceinline__ u64 add(u64 a, u64 b) { return sat_add(a, b); }
  __device__ __forceinline__ u64 mul(u32 a, u64 b) { return sat_mul_u32(a, b); }
  __device__ __forceinline__ bool too_large(u64 total) const { return total >= kSat; }
};

struct StickyMath {
  u32 top = 0;   // bits 64.. of some result
  u32 word = 0;  // bits 32..63 of some result: too large when bit 30 or 31 is set
  __device__ __forceinline__ u64 add(u64 a, u64 b) {
    const u64 s = a + b;  // a, b < 2^62: no wrap
    word |= (u32)(s >> 32);
    return s;
  }
  __device__ __forceinline__ u64 mul(u32 a, u64 b) {
    const u64 lo = (u64)a * (u32)b;
    const u64 upper = (u64)a * (u32)(b >> 32) + (lo >> 32);  // the product >> 32; b < 2^62: no wrap
    top |= (u32)(upper >> 32);
    word |= (u32)upper;
    return (upper << 32) | (u32)lo;
  }
  __device__ __forceinline__ bool too_large(u64) const { return (top | (word >> 30)) != 0; }
};

// zero-extension of a field that check_fields has shown to be non-negative: tells the
// compiler that the upper half is zero, so products of two such values are one widening multiply
__device__ __forceinline__ u64 zx(int v) { return (u64)(u32)v; }

// ceil(x / cu_p) * cu_p; x <= 2^62 keeps the result <= 2^62
__host__ __device__ __forceinline__ u64 page_round(u64 x) { return (x + (kPage - 1)) & ~(kPage - 1); }

// signed variant: the magnitude is rounded, the sign kept.  For d < 0 the result
// -ceil(|d| / cu_p) * cu_p equals floor(d / cu_p) * cu_p, i.e. clearing the low bits of
// the two's-complement value; for d >= 0 it is the usual add-and-mask.
__host__ __device__ __forceinline__ i64 page_round_signed(i64 d) {
  const i64 addend = ~(d >> 63) & (i64)(kPage - 1);
  return (i64)(((u64)d + (u64)addend) & ~(kPage - 1));
}

__device__ __forceinline__ u64 ceil_div(u64 a, u64 b) { return (a + b - 1) / b; }

// A configuration record loaded into registers (four 16-byte loads).
struct Cfg {
  int layers, hidden, heads, ffn, vocab, pos_len, seq, batch;
  i64 chunk_elems, base_bytes;
  u32 method, gpu_n, tp_n, lm_bytes, ffn_kind, has_bias, iters, act_mode;
  bool reserved_zero;
};

// The four 16-byte words of a record, unpacked.
__device__ __forceinline__ Cfg unpack_cfg(const int4& a, const int4& b, const int4& c, const int4& d) {
  Cfg f;
  f.layers = a.x; f.hidden = a.y; f.heads = a.z; f.ffn = a.w;
  f.vocab = b.x; f.pos_len = b.y; f.seq = b.z; f.batch = b.w;
  f.chunk_elems = (i64)(((u64)(u32)c.y << 32) | (u32)c.x);
  f.base_bytes = (i64)(((u64)(u32)c.w << 32) | (u32)c.z);
  u32 w0 = (u32)d.x, w1 = (u32)d.y;
  f.method = w0 & 0xff; f.gpu_n = (w0 >> 8) & 0xff; f.tp_n = (w0 >> 16) & 0xff; f.lm_bytes = w0 >> 24;
  f.ffn_kind = w1 & 0xff; f.has_bias = (w1 >> 8) & 0xff; f.iters = (w1 >> 16) & 0xff;
  f.act_mode = w1 >> 24;
  f.reserved_zero = d.z == 0 && d.w == 0;
  return f;
}

__device__ __forceinline__ Cfg load_cfg(const llmem_config* __restrict__ p) {
  const int4* q = reinterpret_cast<const int4*>(p);
  int4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2), d = __ldg(q + 3);
  return unpack_cfg(a, b, c, d);
}

// Whether d divides x, for 1 <= x <= 2^20 and d >= 1, without the integer division routine:
// both numbers are exact in single precision, the quotient of a fast division is within
// 2^20 * 3 * 2^-24 < 1/2 of the true one, so it rounds to the true quotient whenever that is an
// integer, and one exact multiplication tells.  (A d above x gives quotient 0 or 1 and fails.)
__device__ __forceinline__ bool divides(int d, int x) {
  const int dc = d < (1 << 21) ? d : (1 << 21);
  const float two23 = 8388608.0f;
  const float xf = __uint_as_float(0x4b000000u | (u32)x) - two23;
  const float df = __uint_as_float(0x4b000000u | (u32)dc) - two23;
  const u32 q = __float_as_uint(__fdividef(xf, df) + two23) & 0x007fffffu;  // nearest integer
  return q * (u32)dc == (u32)x;
}

// Field ranges (status 1).  `check_batch` is false for the search entry points,
// which choose the batch themselves; `check_method` is false for selection.
__device__ __forceinline__ int check_fields(const Cfg& f, bool check_batch, bool check_method) {
  bool ok = f.layers >= 1 && f.layers <= (1 << 16) && f.hidden >= 1 && f.hidden <= (1 << 20) &&
            f.heads >= 1 && f.ffn >= 1 && f.ffn <= (1 << 22) && f.vocab >= 1 &&
            f.vocab <= (1 << 26) && f.pos_len >= 0 && f.pos_len <= (1 << 26) && f.seq >= 1 &&
            f.seq <= (1 << 26) && f.chunk_elems >= 1 && f.chunk_elems <= (1ll << 40) &&
            f.base_bytes >= 0 && f.base_bytes <= (1ll << 60) && f.gpu_n >= 1 &&
            (f.lm_bytes == 2 || f.lm_bytes == 4) && f.ffn_kind <= 1 && f.has_bias <= 1 &&
            f.iters >= 1 && f.act_mode <= 1 && f.reserved_zero;
  if (ok) ok = divides(f.heads, f.hidden);
  if (ok && check_batch) ok = f.batch >= 1 && f.batch <= (1 << 26);
  if (ok && check_method) ok = f.method <= 3;
  return ok ? LLMEM_CFG_OK : LLMEM_CFG_FIELD;
}

// Section 5, DP+TP: needs both a DP and a TP dimension (status 2 otherwise).
__device__ __forceinline__ int check_combo(u32 method, u32 gpu_n, u32 tp_n) {
  if (method == LLMEM_METHOD_DPTP && (tp_n < 2 || 2 * tp_n > gpu_n || gpu_n % tp_n != 0))
    return LLMEM_CFG_COMBO;
  return LLMEM_CFG_OK;
}

// Everything that does not depend on the batch size.
struct Plan {
  int status;
  int e_n;        // Embedding operators: token, + learned position
  int K;          // Linear operators per layer (q,k,v,o + 2 or 3 feed-forward matrices)
  int gather;     // phase 2 present: ADP, DP+TP
  int tpback;     // phase 4 present: TP, DP+TP
  int L, iters;
  u32 tp;         // TP degree of the backward buffers: gpu_n for TP, tp_n for DP+TP
  u64 tp_recip;   // ceil(2^64 / tp), 0 for tp = 1
  u32 C;          // chunks = ceil(other_p / cs); < 2^31 when status == 0
  u64 count;      // number of events
  u64 offset;     // m_base + lm_p (added unrounded, Section 4.2)
  // raw byte sizes of the batch-independent event kinds
  u64 p16_embed, p32_embed, p16_chunk, p32_chunk, gat_embed, gat_chunk;
  u64 os_tok, os_pos, os_hh, os_hf;
  // per-sample factors of the batch-dependent kinds: out = batch * out1, ...
  u64 out1, logit1, shift1;
  // operator outputs kept per layer: n_x of the size of a layer output, n_attn attention-score
  // sized (attn1 per sample, saturating), n_ffn feed-forward sized (ffn1 per sample).  With
  // gradient checkpointing (act_mode 0) only the layer output itself: 1, 0, 0.
  int n_x, n_attn, n_ffn;
  u64 attn1, ffn1;
};

// Division by a partition degree (1 .. 255) without a hardware-emulated 64-bit divide:
// with m = ceil(2^64 / d), floor(x / d) = high 64 bits of x * m for every x < 2^56
// (Granlund and Montgomery, "Division by invariant integers using multiplication", 1994,
// N = 56 dividend bits, 8 divisor bits).  Every byte count divided here is below 2^56.
struct Recip {
  u64 m;
  u32 d;
};

// ceil(2^64 / d) for every degree a configuration record can hold, built at compile time.
struct RecipTable {
  u64 m[256];
};
constexpr RecipTable make_recip_table() {
  RecipTable t{};
  for (unsigned d = 2; d < 256; ++d) t.m[d] = ~0ull / d + 1;
  return t;
}
static __device__ const RecipTable kRecipTable = make_recip_table();

__device__ __forceinline__ Recip make_recip(u32 d) {  // d <= 255
  Recip r;
  r.d = d;
  r.m = __ldg(&kRecipTable.m[d & 255u]);
  return r;
}

__device__ __forceinline__ u64 floor_div(u64 x, const Recip& r) { return r.d <= 1 ? x : __umul64hi(x, r.m); }
__device__ __forceinline__ u64 ceil_div(u64 x, const Recip& r) { return floor_div(x + (r.d - 1), r); }

// min(ceil(a / b), 2^31) for a < 2^61, 1 <= b <= 2^40: the number of chunks, or the event
// limit if there would be that many.  ceil(a / b) >= 2^31 exactly when a > (2^31 - 1) b;
// below that the double-precision quotient is within one of the integer one (relative error
// 2^-52 on a value below 2^31) and one multiplication settles it.
__device__ __forceinline__ u64 chunk_count(u64 a, u64 b) {
  const u64 lim = kCountLimit - 1;
  const u64 hi = __umul64hi(b, lim), lo = b * lim;
  if (hi == 0 && a > lo) return kCountLimit;
  u64 q = (u64)__double2ull_rz(__ddiv_rn(__ull2double_rn(a), __ull2double_rn(b)));
  i64 r = (i64)(a - q * b);  // q b <= a + b: no wrap
  if (r < 0) {
    --q;
    r += (i64)b;
  } else if ((u64)r >= b) {
    ++q;
    r -= (i64)b;
  }
  return q + (r != 0 ? 1 : 0);
}

// Bytes of a tensor's shard on one device: the whole tensor for CDP (the caller passes the
// reciprocal of 1), ceil(bytes / gpu_n) otherwise.  No branch on the method: the lanes of a
// warp hold different methods, and a division skipped by some of them is not time saved.
__device__ __forceinline__ u64 shard_bytes(u64 bytes, const Recip& n) { return ceil_div(bytes, n); }

// fp16 bytes of a unit of x elements that exist only while computing:
// ADP holds the whole of param fp16 (m_p,16 undivided in m_peak^dp);
// DP+TP holds m_p,16 * (1 - tp_n/gpu_n) (m_peak^dp+tp).
// `kept` = ceil(2 x / gpu_n), the shard that stays; `n` the reciprocal of gpu_n.
__device__ __forceinline__ u64 gathered_bytes(u64 x, u32 method, const Recip& n, u32 t, u64 kept) {
  const u64 whole = 2 * x;
  const u64 tp_share = floor_div(whole * t, n);  // whole * t < 2^56
  u64 g = 0;
  if (method == LLMEM_METHOD_ADP) g = whole - kept;
  if (method == LLMEM_METHOD_DPTP) g = whole - tp_share - kept;
  return g;
}

// Table 1, other_p: every parameter outside the input embedding and lm_head of a standard
// decoder: per layer q, k, v, o (H x H) and 2 or 3 feed-forward matrices (H x F), their
// biases, two norm vectors; one final norm.  `f` has passed check_fields.
__device__ __forceinline__ u64 other_params(const Cfg& f) {
  const u64 H = zx(f.hidden), F = zx(f.ffn), bias = f.has_bias;
  const u64 nffn = f.ffn_kind ? 3 : 2;
  const u64 bias_p = bias * (4 * H + (nffn - 1) * F + H);
  const u64 norm_p = 2 * H * (1 + bias);
  return zx(f.layers) * (4 * H * H + nffn * H * F + bias_p + norm_p) + H * (1 + bias);  // < 2^61
}

// a1: parameter inventory and event sizes.  `f` has passed check_fields.
template <class Math>
__device__ __forceinline__ Plan make_plan(Math& m, const Cfg& f, u32 method) {
  Plan p;
  p.status = check_combo(method, f.gpu_n, f.tp_n);
  const u64 H = zx(f.hidden), F = zx(f.ffn), V = zx(f.vocab), P = zx(f.pos_len);
  const Recip rn = make_recip(method == LLMEM_METHOD_CDP ? 1u : f.gpu_n);
  p.e_n = 1 + (f.pos_len > 0);
  p.K = f.ffn_kind ? 7 : 6;
  p.gather = (method == LLMEM_METHOD_ADP || method == LLMEM_METHOD_DPTP);
  p.tpback = (method == LLMEM_METHOD_TP || method == LLMEM_METHOD_DPTP);
  p.tp = method == LLMEM_METHOD_TP ? f.gpu_n : f.tp_n;
  if (p.tp == 0) p.tp = 1;  // only reachable with status 2; keeps divisions defined
  p.tp_recip = make_recip(p.tp).m;
  p.L = f.layers;
  p.iters = (int)f.iters;
  const u64 tok_p = V * H, pos_p = P * H, hh_p = H * H, hf_p = H * F;
  const u64 embed_p = tok_p + pos_p;                       // <= 2^47
  const u64 other_p = other_params(f);                     // < 2^61
  const u64 cs = (u64)f.chunk_elems;
  const u64 chunks = chunk_count(other_p, cs);
  p.offset = (u64)f.base_bytes + tok_p * (u64)f.lm_bytes;  // < 2^60 + 2^49
  p.p16_embed = shard_bytes(2 * embed_p, rn);
  p.p32_embed = shard_bytes(4 * embed_p, rn);
  p.p16_chunk = shard_bytes(2 * cs, rn);
  p.p32_chunk = shard_bytes(4 * cs, rn);
  p.gat_embed = gathered_bytes(embed_p, method, rn, p.tp, p.p16_embed);
  p.gat_chunk = gathered_bytes(cs, method, rn, p.tp, p.p16_chunk);
  p.os_tok = shard_bytes(8 * tok_p, rn);
  p.os_pos = shard_bytes(8 * pos_p, rn);
  p.os_hh = shard_bytes(8 * hh_p, rn);
  p.os_hf = shard_bytes(8 * hf_p, rn);
  p.out1 = 2 * zx(f.seq) * H;                              // <= 2^47
  p.logit1 = (u64)f.lm_bytes * zx(f.seq) * V;              // <= 2^54
  p.shift1 = (u64)f.lm_bytes * zx(f.seq - 1) * V;
  // Without gradient checkpointing every operator of a pre-norm layer keeps its fp16 output:
  // norm, q, k, v, scores, softmax, context, o-proj, residual, norm, up (x2 + product when
  // gated), activation, down, residual: 10 hidden-sized, 2 score-sized, 2 or 4 ffn-sized.
  p.n_x = f.act_mode ? 10 : 1;
  p.n_attn = f.act_mode ? 2 : 0;
  p.n_ffn = f.act_mode ? (f.ffn_kind ? 4 : 2) : 0;
  p.attn1 = f.act_mode ? m.mul((u32)f.seq, m.mul((u32)f.seq, 2 * zx(f.heads))) : 0;
  p.ffn1 = 2 * zx(f.seq) * F;                              // <= 2^49
  if (chunks >= kCountLimit) {
    p.C = 0;
    p.count = kCountLimit;
    if (p.status == LLMEM_CFG_OK) p.status = LLMEM_CFG_OVERFLOW;
  } else {
    p.C = (u32)chunks;
    const u64 allocs = (p.gather ? 1 + chunks : 0) + (u64)p.e_n +
                       (u64)p.L * (u64)(p.n_x + p.n_attn + p.n_ffn) + 3 + (p.tpback ? (u64)p.L : 0);
    p.count = 2 + 2 * chunks + (u64)p.e_n + (u64)p.K * (u64)p.L + (u64)p.iters * 2 * allocs;
    if (p.count >= kCountLimit && p.status == LLMEM_CFG_OK) p.status = LLMEM_CFG_OVERFLOW;
  }
  return p;
}

__device__ __forceinline__ Plan make_plan(const Cfg& f, u32 method) {
  SatMath m;
  return make_plan(m, f, method);
}

// Batch-dependent raw sizes (saturating).
struct Dyn {
  u64 out, logit, shift, back, attn, ffn;
};

template <class Math>
__device__ __forceinline__ Dyn make_dyn(Math& m, const Plan& p, u64 batch) {
  Dyn d;
  const u32 b32 = (u32)batch;  // batch <= 2^26
  d.out = m.mul(b32, p.out1);
  d.logit = m.mul(b32, p.logit1);
  d.shift = m.mul(b32, p.shift1);
  // ceil(out * (tp-1) / tp) = out - floor(out / tp)   (m_back^tp, one layer's share); the
  // reciprocal is exact below 2^56, and a saturated output makes the whole peak overflow.
  // The quotient is formed in every lane (no branch on the method), the rare wide one apart.
  u64 share = floor_div(d.out, Recip{p.tp_recip, p.tp});
  if (p.tpback && d.out >= (1ull << 56)) share = d.out / p.tp;
  d.back = p.tpback ? d.out - share : 0;
  if (p.tpback && d.out >= kSat) d.back = kSat;
  d.attn = p.n_attn ? m.mul(b32, p.attn1) : 0;
  d.ffn = p.n_ffn ? m.mul(b32, p.ffn1) : 0;
  return d;
}

__device__ __forceinline__ Dyn make_dyn(const Plan& p, u64 batch) {
  SatMath m;
  return make_dyn(m, p, batch);
}

// Batch-independent sums of rounded events.
struct StaticSums {
  u64 init, gather, os;
};

template <class Math>
__device__ __forceinline__ StaticSums make_static_sums(Math& m, const Plan& p, bool has_pos) {
  StaticSums s;
  s.init = m.add(m.add(page_round(p.p16_embed), page_round(p.p32_embed)),
                 m.mul(p.C, page_round(p.p16_chunk) + page_round(p.p32_chunk)));
  s.gather = p.gather ? m.add(page_round(p.gat_embed), m.mul(p.C, page_round(p.gat_chunk))) : 0;
  const u64 per_layer = 4 * page_round(p.os_hh) + (u64)(p.K - 4) * page_round(p.os_hf);  // < 2^48
  s.os = m.add(page_round(p.os_tok) + (has_pos ? page_round(p.os_pos) : 0), m.mul((u32)p.L, per_layer));
  return s;
}

__device__ __forceinline__ StaticSums make_static_sums(const Plan& p, bool has_pos) {
  SatMath m;
  return make_static_sums(m, p, has_pos);
}

// Sum of the rounded batch-dependent allocations of one iteration (phases 3 and 4).
template <class Math>
__device__ __forceinline__ u64 dyn_sum(Math& m, const Plan& p, const Dyn& d) {
  u64 s = m.mul((u32)(p.e_n + p.L * p.n_x), page_round(d.out));
  if (p.n_attn) s = m.add(s, m.mul((u32)(p.L * p.n_attn), page_round(d.attn)));
  if (p.n_ffn) s = m.add(s, m.mul((u32)(p.L * p.n_ffn), page_round(d.ffn)));
  s = m.add(s, page_round(d.logit));
  s = m.add(s, m.mul(2u, page_round(d.shift)));
  if (p.tpback) s = m.add(s, m.mul((u32)p.L, page_round(d.back)));
  return s;
}

__device__ __forceinline__ u64 dyn_sum(const Plan& p, const Dyn& d) {
  SatMath m;
  return dyn_sum(m, p, d);
}

// Largest prefix sum (without the offset) given the phase sums.  Iteration 1
// peaks before the optimizer states exist; they are allocated after its frees and
// stay; every later iteration peaks on top of them.  Only sums that the result is at least
// as large as are formed, so that a sum which is too large makes the result too large.
template <class Math>
__device__ __forceinline__ u64 relative_peak(Math& m, const Plan& p, const StaticSums& s, u64 dyn_total,
                                             bool* first_iteration_wins) {
  const u64 after = m.add(s.init, s.os);
  if (p.iters >= 2) {
    *first_iteration_wins = false;
    return m.add(after, dyn_total);
  }
  const u64 first = m.add(s.init, dyn_total);
  *first_iteration_wins = first >= after;
  return first >= after ? first : after;
}

__device__ __forceinline__ u64 relative_peak(const Plan& p, const StaticSums& s, u64 dyn_total,
                                             bool* first_iteration_wins) {
  SatMath m;
  return relative_peak(m, p, s, dyn_total, first_iteration_wins);
}

// Complete admissibility check of a configuration for estimation: field ranges,
// method / degree combination, event-count limit and byte limit.  On LLMEM_CFG_OK
// *plan_out holds the plan and *peak_out the peak (offset included).
__device__ __forceinline__ int full_status(const Cfg& f, Plan* plan_out, u64* peak_out) {
  int st = check_fields(f, true, true);
  if (st != LLMEM_CFG_OK) return st;
  *plan_out = make_plan(f, f.method);
  if (plan_out->status != LLMEM_CFG_OK) return plan_out->status;
  StaticSums s = make_static_sums(*plan_out, f.pos_len > 0);
  Dyn d = make_dyn(*plan_out, (u64)f.batch);
  bool fw;
  u64 rel = relative_peak(*plan_out, s, sat_add(s.gather, dyn_sum(*plan_out, d)), &fw);
  u64 total = sat_add(plan_out->offset, rel);
  if (total >= kSat) return LLMEM_CFG_OVERFLOW;
  *peak_out = total;
  return LLMEM_CFG_OK;
}

// ---------------------------------------------------------------------------
// The DNNMem-style estimator of Section 3.1, which the paper implements for comparison: the
// weight tensors as loaded (fp16), a constant 64 MB buffer of the block manager, and the
// outputs of the forward pass accumulated operator by operator, every tensor aligned to 512
// bytes; one device, no mixed precision, no chunks, no optimizer states.  The allocations in
// order: buffer; token (and position) embedding; the Linear matrices layer by layer; the
// vectors layer by layer (two norm weights, with biases also two norm biases, four attention
// biases and the feed-forward output bias, then the feed-forward input biases); the final
// norm; the lm_head; then embedding outputs, layer outputs (or every operator output),
// logits and the two shifted copies as in the LLMem list.  Nothing is released during the
// forward pass, so the peak is the total.
// ---------------------------------------------------------------------------
constexpr u64 kDnnAlign = 512;
constexpr u64 kDnnBuffer = 64ull * 1024ull * 1024ull;

__host__ __device__ __forceinline__ u64 align512(u64 x) { return (x + (kDnnAlign - 1)) & ~(kDnnAlign - 1); }

struct DnnPlan {
  int status;
  int e_n, K, L, has_pos;
  int small, wide, final_n;  // vectors per layer of the hidden / of the feed-forward size; final norm vectors
  int n_x, n_attn, n_ffn;    // operator outputs kept per layer, by size
  u64 count;                 // number of events
  u64 tok, pos, hh, hf, vec_h, vec_f, lm;  // raw bytes of the weight tensors
  u64 out, attn, ffn, logit, shift;        // raw bytes of the forward outputs (saturating)
};

// `f` has passed check_fields(f, true, true).
__device__ __forceinline__ DnnPlan make_dnn_plan(const Cfg& f) {
  DnnPlan p;
  p.status = f.method == LLMEM_METHOD_CDP ? LLMEM_CFG_OK : LLMEM_CFG_COMBO;  // one device, no sharding
  const u64 H = zx(f.hidden), F = zx(f.ffn), V = zx(f.vocab), P = zx(f.pos_len);
  const int bias = (int)f.has_bias;
  p.e_n = 1 + (f.pos_len > 0);
  p.has_pos = f.pos_len > 0;
  p.K = f.ffn_kind ? 7 : 6;
  p.L = f.layers;
  p.small = 2 + 7 * bias;
  p.wide = bias * (p.K - 5);
  p.final_n = 1 + bias;
  p.n_x = f.act_mode ? 10 : 1;
  p.n_attn = f.act_mode ? 2 : 0;
  p.n_ffn = f.act_mode ? (f.ffn_kind ? 4 : 2) : 0;
  p.tok = 2 * V * H;
  p.pos = 2 * P * H;
  p.hh = 2 * H * H;
  p.hf = 2 * H * F;
  p.vec_h = 2 * H;
  p.vec_f = 2 * F;
  p.lm = V * H * (u64)f.lm_bytes;
  const u32 b = (u32)f.batch;
  p.out = sat_mul_u32(b, 2 * zx(f.seq) * H);
  p.logit = sat_mul_u32(b, (u64)f.lm_bytes * zx(f.seq) * V);
  p.shift = sat_mul_u32(b, (u64)f.lm_bytes * zx(f.seq - 1) * V);
  p.attn = p.n_attn ? sat_mul_u32(b, sat_mul_u32((u32)f.seq, sat_mul_u32((u32)f.seq, 2 * zx(f.heads)))) : 0;
  p.ffn = p.n_ffn ? sat_mul_u32(b, 2 * zx(f.seq) * F) : 0;
  p.count = 2 + (u64)p.has_pos + (u64)p.L * (u64)(p.K + p.small + p.wide) + (u64)p.final_n + 1 + (u64)p.e_n +
            (u64)p.L * (u64)(p.n_x + p.n_attn + p.n_ffn) + 3;
  return p;
}

// Sum of the aligned events (without m_base), saturating at 2^62.
__device__ __forceinline__ u64 dnn_total(const DnnPlan& p) {
  u64 s = kDnnBuffer + align512(p.tok) + (p.has_pos ? align512(p.pos) : 0) + align512(p.lm);
  s = sat_add(s, sat_mul_u32((u32)p.L, 4 * align512(p.hh) + (u64)(p.K - 4) * align512(p.hf) +
                                           (u64)p.small * align512(p.vec_h) + (u64)p.wide * align512(p.vec_f)));
  s += (u64)p.final_n * align512(p.vec_h);
  if (p.out >= kSat || p.logit >= kSat || p.shift >= kSat || p.attn >= kSat || p.ffn >= kSat) return kSat;
  s = sat_add(s, sat_mul_u32((u32)(p.e_n + p.L * p.n_x), align512(p.out)));
  if (p.n_attn) s = sat_add(s, sat_mul_u32((u32)(p.L * p.n_attn), align512(p.attn)));
  if (p.n_ffn) s = sat_add(s, sat_mul_u32((u32)(p.L * p.n_ffn), align512(p.ffn)));
  s = sat_add(s, align512(p.logit));
  s = sat_add(s, sat_mul_u32(2u, align512(p.shift)));
  return s;
}

// Status and peak of a configuration under the second estimator; on LLMEM_CFG_OK *plan_out
// holds the plan and *peak_out the peak (m_base included).
__device__ __forceinline__ int dnn_full_status(const Cfg& f, DnnPlan* plan_out, u64* peak_out) {
  int st = check_fields(f, true, true);
  if (st != LLMEM_CFG_OK) return st;
  *plan_out = make_dnn_plan(f);
  if (plan_out->status != LLMEM_CFG_OK) return plan_out->status;
  const u64 total = sat_add((u64)f.base_bytes, dnn_total(*plan_out));
  if (total >= kSat) return LLMEM_CFG_OVERFLOW;
  *peak_out = total;
  return LLMEM_CFG_OK;
}

}  // namespace llmem
