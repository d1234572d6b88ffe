/*
 * LLMem peak-memory oracle  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of what the estimator
 * computes, written from the paper (Kim et al., "LLMem: Estimating GPU Memory
 * Usage for Fine-Tuning Pre-Trained LLMs", arXiv 2404.10933).  It exists so
 * that tests can check the CUDA library against it and so that the benchmark
 * can time a CPU baseline.  Nothing in the product path may call it, and it
 * shares no code, header, table or helper with the CUDA library; the record
 * layout below is restated here because it is the input format.
 *
 * What is computed (level 1, "the definition"):
 *   1. the parameter inventory of a standard transformer decoder
 *      (Table 1 symbols embed_p, other_p, lm_p, t_p, e_n, l_n, o_n, dict_n);
 *   2. the explicit list of signed allocate/free byte counts in the phase
 *      order of Sections 4.1 and 5 (phases 1..5 of Figure 4): initialisation,
 *      ADP gather, output phase, TP backward buffers, frees, optimizer states
 *      in iteration 1;
 *   3. rounding of every magnitude up to the CUDA page size cu_p = 2*1024^2
 *      (Section 4.2, every ceil(./cu_p)*cu_p);
 *   4. a linear prefix sum and its maximum, plus m_base and lm_p which the
 *      equations of Section 4.2 add unrounded;
 *   5. Algorithm 1 (Section 6): per-method largest batch by literal
 *      increment, scores, tie order, CPU-offload sentinel.
 *
 * Level 2 (oracle_*_collapsed / *_bisect) is a second, independent-by-
 * construction evaluation inside the oracle: per-phase sums instead of an
 * explicit list, bisection instead of increment.  Tests show level 2 == level 1
 * before level 2 is used on grids too large for level 1.
 *
 * Pins (see tests/test_oracle_pins.py): closed forms of Sections 4.2 and 5 in
 * exact rational arithmetic on page-aligned shapes; two-sided bound between
 * per-event and per-term rounding; public parameter counts of two well known
 * decoders; interval-sweep allocator simulation; invariants; hand cases for
 * rounding and for Algorithm 1.  "parity unpinned": Table 2 and Figures 7-9
 * values (m_base, cs and batch sizes are not printed in the paper); and the
 * operator list of act_mode = 1 (Section 4.2 allows summing per-operator
 * outputs without gradient checkpointing but prints neither the operators nor a
 * number: the list here is a reading, pinned only to an independent
 * enumeration of the same reading and to its reduction to m_out).
 *
 * A second estimator (oracle_dnn_*) restates the DNNMem-style procedure that Section 3.1
 * describes and the paper compares with: weight tensors as loaded plus a constant 64 MB
 * buffer, then the outputs of the forward pass accumulated operator by operator, every
 * tensor aligned to 512 bytes; no mixed precision, no chunks, no optimizer states.  The paper
 * gives the procedure in words only: the tensor list is this file's standard-decoder
 * inventory and the event order a reading ("parity unpinned" with respect to the paper's
 * numbers, which need its models); pinned to an independent tensor enumeration and to the
 * facts that the list only grows and that it stays below the LLMem estimate.
 *
 * All arithmetic is integer.  Intermediate values use unsigned __int128 so
 * that the overflow guard (status 3) is decided exactly.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;
typedef __int128 i128;

/* ---- input record: 64 bytes, same layout as the library's llmem_config ---- */
typedef struct {
  int32_t layers;      /* l_n */
  int32_t hidden;      /* o_n */
  int32_t heads;       /* carried and validated only */
  int32_t ffn;
  int32_t vocab;       /* dict_n */
  int32_t pos_len;     /* learned position embedding rows, 0 = none */
  int32_t seq;         /* sl */
  int32_t batch;       /* bs */
  int64_t chunk_elems; /* cs */
  int64_t base_bytes;  /* m_base */
  uint8_t method;      /* 0 CDP, 1 ADP, 2 TP, 3 DP+TP */
  uint8_t gpu_n;
  uint8_t tp_n;
  uint8_t lm_bytes;    /* B of the m_lm equation */
  uint8_t ffn_kind;    /* 0: two FFN matrices, 1: three (gated) */
  uint8_t has_bias;
  uint8_t iters;
  uint8_t act_mode;    /* 0: gradient checkpointing (layer outputs kept), 1: every operator output kept */
  uint8_t reserved[8];
} oracle_config;

_Static_assert(sizeof(oracle_config) == 64, "record is 64 bytes");

enum { ST_OK = 0, ST_FIELD = 1, ST_COMBO = 2, ST_OVERFLOW = 3 };
enum { M_CDP = 0, M_ADP = 1, M_TP = 2, M_DPTP = 3 };

/* Table 1: B16 = 2, B32 = 4; Section 4.2: cu_p = 2 x 1024^2 bytes. */
#define B16 ((u128)2)
#define B32 ((u128)4)
#define CU_P ((u128)2 * 1024 * 1024)
#define BYTES_LIMIT (((u128)1) << 62) /* every event, prefix and peak must stay below */
#define COUNT_LIMIT (((u128)1) << 31) /* events per configuration must stay below */

/* supported input domain (documented in the library header as well) */
#define MAX_LAYERS (1 << 16)
#define MAX_HIDDEN (1 << 20)
#define MAX_FFN (1 << 22)
#define MAX_VOCAB (1 << 26)
#define MAX_POS (1 << 26)
#define MAX_SEQ (1 << 26)
#define MAX_BATCH (1 << 26)
#define MAX_CHUNK (((int64_t)1) << 40)
#define MAX_BASE (((int64_t)1) << 60)

static u128 ceil_div(u128 a, u128 b) { return (a + b - 1) / b; }

/* ceil(x / cu_p) * cu_p */
static u128 page_round(u128 x) { return ceil_div(x, CU_P) * CU_P; }

/* ------------------------------------------------------------------------ */
/* validation                                                               */
/* ------------------------------------------------------------------------ */
static int validate_fields(const oracle_config *c, int check_batch) {
  if (c->layers < 1 || c->layers > MAX_LAYERS) return ST_FIELD;
  if (c->hidden < 1 || c->hidden > MAX_HIDDEN) return ST_FIELD;
  if (c->heads < 1 || c->hidden % c->heads != 0) return ST_FIELD;
  if (c->ffn < 1 || c->ffn > MAX_FFN) return ST_FIELD;
  if (c->vocab < 1 || c->vocab > MAX_VOCAB) return ST_FIELD;
  if (c->pos_len < 0 || c->pos_len > MAX_POS) return ST_FIELD;
  if (c->seq < 1 || c->seq > MAX_SEQ) return ST_FIELD;
  if (check_batch && (c->batch < 1 || c->batch > MAX_BATCH)) return ST_FIELD;
  if (c->chunk_elems < 1 || c->chunk_elems > MAX_CHUNK) return ST_FIELD;
  if (c->base_bytes < 0 || c->base_bytes > MAX_BASE) return ST_FIELD;
  if (c->method > 3) return ST_FIELD;
  if (c->gpu_n < 1) return ST_FIELD;
  if (c->lm_bytes != 2 && c->lm_bytes != 4) return ST_FIELD;
  if (c->ffn_kind > 1 || c->has_bias > 1) return ST_FIELD;
  if (c->iters < 1) return ST_FIELD;
  if (c->act_mode > 1) return ST_FIELD;
  for (int i = 0; i < 8; ++i)
    if (c->reserved[i] != 0) return ST_FIELD;
  return ST_OK;
}

static int validate_combo(const oracle_config *c) {
  if (c->method == M_DPTP) {
    /* Section 5, "Combination of DP+TP": both a DP and a TP dimension exist */
    int n = c->gpu_n, t = c->tp_n;
    if (t < 2 || 2 * t > n || n % t != 0) return ST_COMBO;
  }
  return ST_OK;
}

int oracle_validate(const oracle_config *c) {
  int st = validate_fields(c, 1);
  if (st) return st;
  return validate_combo(c);
}

/* ------------------------------------------------------------------------ */
/* step 1: parameter inventory and event sizes                              */
/* ------------------------------------------------------------------------ */
typedef struct {
  int e_n;     /* number of Embedding operators (token, + learned position) */
  int K;       /* Linear operators per layer */
  int gather;  /* phase 2 present (ADP, DP+TP) */
  int tpback;  /* phase 4 present (TP, DP+TP) */
  int64_t L;
  u128 C;        /* ceil(other_p / cs) chunks */
  u128 embed_p;  /* elements */
  u128 other_p;  /* elements */
  u128 lm_p;     /* bytes */
  u128 tok_p, pos_p, hh_p, hf_p; /* elements of each Embedding / Linear tensor kind */
  /* raw (unrounded) byte sizes of each event kind */
  u128 p16_embed, p32_embed, p16_chunk, p32_chunk;
  u128 gat_embed, gat_chunk;
  u128 os_tok, os_pos, os_hh, os_hf;
  u128 out, logit, shift, back;
  /* without gradient checkpointing: attention-score and feed-forward sized outputs */
  u128 act_attn, act_ffn;
  int n_ops;         /* operator outputs kept per layer (1 with checkpointing) */
  int op_kind[16];   /* 0: hidden-sized (out), 1: attention scores, 2: feed-forward sized */
} sizes_t;

/* Persistent fp16 bytes of a unit of x elements.  CDP keeps all of it
 * (Section 5, CDP = single GPU); the other methods keep a 1/gpu_n shard
 * (Section 5: ZeRO-3 and TP split parameters evenly over the gpu_n devices). */
static u128 shard(u128 bytes, const oracle_config *c) {
  return c->method == M_CDP ? bytes : ceil_div(bytes, c->gpu_n);
}

/* Temporary fp16 bytes of a unit while computing.
 * ADP: the whole of param fp16 is resident (m_p,16 undivided in m_peak^dp).
 * DP+TP: m_peak^dp minus m_p,16 * tp_n / gpu_n. */
static u128 gathered(u128 x_elems, const oracle_config *c) {
  u128 whole = B16 * x_elems;
  u128 kept = ceil_div(whole, c->gpu_n);
  if (c->method == M_ADP) return whole - kept;
  if (c->method == M_DPTP) return whole - (whole * c->tp_n) / c->gpu_n - kept;
  return 0;
}

static void compute_sizes(const oracle_config *c, sizes_t *z) {
  memset(z, 0, sizeof *z);
  u128 H = (u128)c->hidden, F = (u128)c->ffn, V = (u128)c->vocab, P = (u128)c->pos_len;
  u128 bias = c->has_bias;
  z->L = c->layers;
  z->e_n = 1 + (c->pos_len > 0);
  z->K = c->ffn_kind ? 7 : 6;
  z->gather = (c->method == M_ADP || c->method == M_DPTP);
  z->tpback = (c->method == M_TP || c->method == M_DPTP);

  /* standard decoder: token (+ position) embedding; per layer q,k,v,o (H x H)
   * and K-4 FFN matrices (H x F); biases and norm vectors */
  z->tok_p = V * H;
  z->pos_p = P * H;
  z->hh_p = H * H;
  z->hf_p = H * F;
  z->embed_p = z->tok_p + z->pos_p;
  u128 nffn = (u128)(z->K - 4);
  u128 bias_p = bias * (4 * H + (nffn - 1) * F + H);
  u128 norm_p = 2 * H * (1 + bias);
  z->other_p = (u128)z->L * (4 * z->hh_p + nffn * z->hf_p + bias_p + norm_p) + H * (1 + bias);
  z->C = ceil_div(z->other_p, (u128)c->chunk_elems);
  z->lm_p = V * H * (u128)c->lm_bytes;

  /* phase 1: param fp16 and fp32 are allocated one chunk at a time (Section 4.1) */
  u128 cs = (u128)c->chunk_elems;
  z->p16_embed = shard(B16 * z->embed_p, c);
  z->p32_embed = shard(B32 * z->embed_p, c);
  z->p16_chunk = shard(B16 * cs, c);
  z->p32_chunk = shard(B32 * cs, c);
  /* phase 2 */
  z->gat_embed = gathered(z->embed_p, c);
  z->gat_chunk = gathered(cs, c);
  /* phase 5: momentum + variance, per Embedding / Linear tensor (m_os equation) */
  z->os_tok = shard((B32 + B32) * z->tok_p, c);
  z->os_pos = shard((B32 + B32) * z->pos_p, c);
  z->os_hh = shard((B32 + B32) * z->hh_p, c);
  z->os_hf = shard((B32 + B32) * z->hf_p, c);
  /* phase 3: one output per embedding and per layer (m_out), logits and the
   * two shifted temporaries (m_lm) */
  u128 bs = (u128)c->batch, sl = (u128)c->seq;
  z->out = bs * sl * H * B16;
  z->logit = bs * sl * V * (u128)c->lm_bytes;
  z->shift = bs * (sl - 1) * V * (u128)c->lm_bytes;
  /* Section 4.2 notes that estimation per operator output is supported when gradient
   * checkpointing is off, without printing an equation.  Reading: every operator of a layer
   * keeps its fp16 output until backward.  Forward order of a pre-norm decoder layer:
   * norm, q, k, v, attention scores, softmax, context, output projection, residual, norm,
   * feed-forward up (two of them plus their product when gated), activation, feed-forward
   * down, residual.  The last one is the layer output that checkpointing keeps. */
  z->act_attn = bs * (u128)c->heads * sl * sl * B16;
  z->act_ffn = bs * sl * F * B16;
  if (c->act_mode == 0) {
    z->n_ops = 1;
    z->op_kind[0] = 0;
  } else {
    static const int plain[14] = {0, 0, 0, 0, 1, 1, 0, 0, 0, 0, 2, 2, 0, 0};
    static const int gated[16] = {0, 0, 0, 0, 1, 1, 0, 0, 0, 0, 2, 2, 2, 2, 0, 0};
    z->n_ops = c->ffn_kind ? 16 : 14;
    for (int k = 0; k < z->n_ops; ++k) z->op_kind[k] = c->ffn_kind ? gated[k] : plain[k];
  }
  /* phase 4: per-layer share of m_back^tp; for plain TP tp_n = gpu_n */
  if (z->tpback) {
    u128 t = (c->method == M_TP) ? c->gpu_n : c->tp_n;
    z->back = ceil_div(z->out * (t - 1), t);
  }
}

/* number of events, by formula (used for the count guard before any walk) */
static u128 event_count_formula(const oracle_config *c, const sizes_t *z) {
  u128 init = 2 + 2 * z->C;
  u128 os = (u128)z->e_n + (u128)z->K * (u128)z->L;
  u128 allocs = (z->gather ? 1 + z->C : 0) + (u128)z->e_n + (u128)z->L * (u128)z->n_ops + 3 +
                (z->tpback ? (u128)z->L : 0);
  return init + os + (u128)c->iters * 2 * allocs;
}

/* ------------------------------------------------------------------------ */
/* step 2: the explicit event list, in phase order                          */
/* ------------------------------------------------------------------------ */
typedef struct {
  int64_t *dst;   /* NULL: count only */
  int64_t n;
  int overflow;   /* some rounded magnitude reaches BYTES_LIMIT */
} sink_t;

static void emit(sink_t *s, int sign, u128 bytes) {
  if (page_round(bytes) >= BYTES_LIMIT) s->overflow = 1;
  if (s->dst && !s->overflow) s->dst[s->n] = sign > 0 ? (int64_t)bytes : -(int64_t)bytes;
  s->n++;
}

static u128 op_size(const sizes_t *z, int k) {
  return z->op_kind[k] == 0 ? z->out : (z->op_kind[k] == 1 ? z->act_attn : z->act_ffn);
}

static void walk_events(const oracle_config *c, const sizes_t *z, sink_t *s) {
  int64_t C = (int64_t)z->C, L = z->L;
  /* phase 1: initialisation (Section 4.1) */
  emit(s, +1, z->p16_embed);
  emit(s, +1, z->p32_embed);
  for (int64_t j = 0; j < C; ++j) {
    emit(s, +1, z->p16_chunk);
    emit(s, +1, z->p32_chunk);
  }
  for (int it = 1; it <= c->iters; ++it) {
    /* phase 2: ADP / DP+TP gather the rest of param fp16 before computing */
    if (z->gather) {
      emit(s, +1, z->gat_embed);
      for (int64_t j = 0; j < C; ++j) emit(s, +1, z->gat_chunk);
    }
    /* phase 3: embedding and layer outputs kept for checkpointed backward,
     * then lm_head logits and the two shifted copies for the loss */
    for (int64_t i = 0; i < z->e_n; ++i) emit(s, +1, z->out);
    for (int64_t l = 0; l < L; ++l)
      for (int k = 0; k < z->n_ops; ++k) emit(s, +1, op_size(z, k));
    emit(s, +1, z->logit);
    emit(s, +1, z->shift);
    emit(s, +1, z->shift);
    /* phase 4: TP backward all-gather buffers, one per layer */
    if (z->tpback)
      for (int64_t l = 0; l < L; ++l) emit(s, +1, z->back);
    /* end of iteration: everything temporary is released, last allocated first */
    if (z->tpback)
      for (int64_t l = 0; l < L; ++l) emit(s, -1, z->back);
    emit(s, -1, z->shift);
    emit(s, -1, z->shift);
    emit(s, -1, z->logit);
    for (int64_t l = 0; l < L; ++l)
      for (int k = z->n_ops - 1; k >= 0; --k) emit(s, -1, op_size(z, k));
    for (int64_t i = 0; i < z->e_n; ++i) emit(s, -1, z->out);
    if (z->gather) {
      for (int64_t j = 0; j < C; ++j) emit(s, -1, z->gat_chunk);
      emit(s, -1, z->gat_embed);
    }
    /* phase 5: momentum and variance fp32 appear in the first iteration and
     * are retained (Section 4.1); one allocation per Embedding / Linear tensor */
    if (it == 1) {
      emit(s, +1, z->os_tok);
      if (c->pos_len > 0) emit(s, +1, z->os_pos);
      for (int64_t l = 0; l < L; ++l)
        for (int k = 0; k < z->K; ++k) emit(s, +1, k < 4 ? z->os_hh : z->os_hf);
    }
  }
}

/* Validate, apply the guards, and build the raw (unrounded) signed list.
 * On ST_OK *list_out is malloc'd (caller frees) and holds *n_out entries. */
static int build_events(const oracle_config *c, int64_t **list_out, int64_t *n_out) {
  *list_out = NULL;
  *n_out = 0;
  int st = oracle_validate(c);
  if (st) return st;
  sizes_t z;
  compute_sizes(c, &z);
  if (event_count_formula(c, &z) >= COUNT_LIMIT) return ST_OVERFLOW;
  sink_t counter = {NULL, 0, 0};
  walk_events(c, &z, &counter);
  if (counter.overflow) return ST_OVERFLOW;
  int64_t *d = (int64_t *)malloc((size_t)counter.n * sizeof(int64_t));
  if (!d) return -1;
  sink_t writer = {d, 0, 0};
  walk_events(c, &z, &writer);
  /* every prefix of the rounded list, on top of m_base + lm_p, stays in [0, 2^62) */
  u128 off = (u128)c->base_bytes + z.lm_p;
  i128 run = 0;
  int bad = off >= BYTES_LIMIT;
  for (int64_t k = 0; k < writer.n && !bad; ++k) {
    u128 mag = d[k] < 0 ? (u128)(-(i128)d[k]) : (u128)d[k];
    run += d[k] < 0 ? -(i128)page_round(mag) : (i128)page_round(mag);
    if (run < 0 || (u128)run + off >= BYTES_LIMIT) bad = 1;
  }
  if (bad) {
    free(d);
    return ST_OVERFLOW;
  }
  *list_out = d;
  *n_out = writer.n;
  return ST_OK;
}

/* status and number of events of a configuration (0 events unless status 0) */
int oracle_event_count(const oracle_config *c, int64_t *count_out) {
  int64_t *d;
  int st = build_events(c, &d, count_out);
  free(d);
  return st;
}

/* the same count by the closed formula, without walking (tests compare the two) */
int oracle_event_count_formula(const oracle_config *c, int64_t *count_out) {
  *count_out = 0;
  int st = oracle_validate(c);
  if (st) return st;
  sizes_t z;
  compute_sizes(c, &z);
  u128 e = event_count_formula(c, &z);
  if (e >= COUNT_LIMIT) return ST_OVERFLOW;
  *count_out = (int64_t)e;
  return ST_OK;
}

/* raw (unrounded) signed byte deltas; dst must hold oracle_event_count() entries */
int oracle_expand_events(const oracle_config *c, int64_t *dst, int64_t capacity) {
  int64_t *d, n;
  int st = build_events(c, &d, &n);
  if (st) return st;
  if (capacity < n) {
    free(d);
    return -1;
  }
  memcpy(dst, d, (size_t)n * sizeof(int64_t));
  free(d);
  return ST_OK;
}

/* ------------------------------------------------------------------------ */
/* step 3: granularity rounding                                             */
/* ------------------------------------------------------------------------ */
void oracle_round_events(int64_t *d, int64_t n) {
  for (int64_t k = 0; k < n; ++k) {
    if (d[k] >= 0)
      d[k] = (int64_t)page_round((u128)d[k]);
    else
      d[k] = -(int64_t)page_round((u128)(-(i128)d[k]));
  }
}

/* ------------------------------------------------------------------------ */
/* step 4: prefix sum and maximum                                           */
/* ------------------------------------------------------------------------ */
/* max over k of d[0]+..+d[k], and the first k that attains it; an empty list
 * gives 0 and -1 */
void oracle_scan_peak(const int64_t *d, int64_t n, int64_t *max_prefix, int64_t *first_index) {
  i128 run = 0, best = 0;
  int64_t arg = -1;
  for (int64_t k = 0; k < n; ++k) {
    run += d[k];
    if (arg < 0 || run > best) {
      best = run;
      arg = k;
    }
  }
  *max_prefix = (int64_t)best;
  *first_index = arg;
}

/* m_base + lm_p: the two terms the peak equations add without page rounding */
int oracle_peak_offset(const oracle_config *c, int64_t *offset_out) {
  *offset_out = -1;
  int st = oracle_validate(c);
  if (st) return st;
  sizes_t z;
  compute_sizes(c, &z);
  u128 off = (u128)c->base_bytes + z.lm_p;
  if (off >= BYTES_LIMIT) return ST_OVERFLOW;
  *offset_out = (int64_t)off;
  return ST_OK;
}

/* level 1 estimate: expand, round, scan */
int oracle_estimate(const oracle_config *c, int64_t *peak_out, int64_t *index_out,
                    int64_t *count_out) {
  *peak_out = -1;
  *index_out = -1;
  if (count_out) *count_out = 0;
  int64_t *d, n;
  int st = build_events(c, &d, &n);
  if (st) return st;
  oracle_round_events(d, n);
  int64_t best, arg, off;
  oracle_scan_peak(d, n, &best, &arg);
  free(d);
  oracle_peak_offset(c, &off);
  *peak_out = off + best;
  *index_out = arg;
  if (count_out) *count_out = n;
  return ST_OK;
}

/* Two position-weighted checksums (mod 2^64) of the page-rounded list of one configuration,
 * so that a test can compare a whole list held elsewhere with the explicit list built here
 * without moving it: with k the 0-based position inside the list,
 *   a = sum d[k] * (k + 1),   b = sum d[k] * (k + 1)^2.
 * A wrong, missing, shifted or swapped element changes at least one of them. */
int oracle_list_digest(const oracle_config *c, uint64_t *a_out, uint64_t *b_out) {
  *a_out = 0;
  *b_out = 0;
  int64_t *d, n;
  int st = build_events(c, &d, &n);
  if (st) return st;
  oracle_round_events(d, n);
  uint64_t a = 0, b = 0;
  for (int64_t k = 0; k < n; ++k) {
    const uint64_t w = (uint64_t)k + 1;
    a += (uint64_t)d[k] * w;
    b += (uint64_t)d[k] * w * w;
  }
  free(d);
  *a_out = a;
  *b_out = b;
  return ST_OK;
}

/* ------------------------------------------------------------------------ */
/* the DNNMem-style estimator of Section 3.1                                 */
/* ------------------------------------------------------------------------ */
#define DNN_ALIGN ((u128)512)                      /* PyTorch's tensor alignment (Section 3.1) */
#define DNN_BUFFER ((u128)64 * 1024 * 1024)        /* constant buffer of the block manager (Section 3.1) */

static u128 align512(u128 x) { return ceil_div(x, DNN_ALIGN) * DNN_ALIGN; }

/* The procedure models one device without sharding: only the conventional method is accepted. */
static int dnn_validate(const oracle_config *c) {
  int st = validate_fields(c, 1);
  if (st) return st;
  if (c->method != M_CDP) return ST_COMBO;
  return ST_OK;
}

/* Allocations in order (nothing is released during the forward pass of a fine-tuning
 * iteration: the outputs are kept for backward): the constant buffer; the weight tensors
 * as loaded, fp16, the embeddings first, then the Linear matrices layer by layer, then the
 * vectors (norm weights, and norm and Linear biases where the model has them) layer by
 * layer, the final norm, the lm_head; then the outputs of the forward pass as in phase 3
 * of the LLMem list. */
static void dnn_walk(const oracle_config *c, const sizes_t *z, sink_t *s) {
  u128 H = (u128)c->hidden, F = (u128)c->ffn, bias = c->has_bias;
  emit(s, +1, DNN_BUFFER);
  emit(s, +1, B16 * z->tok_p);
  if (c->pos_len > 0) emit(s, +1, B16 * z->pos_p);
  for (int64_t l = 0; l < z->L; ++l)
    for (int k = 0; k < z->K; ++k) emit(s, +1, B16 * (k < 4 ? z->hh_p : z->hf_p));
  for (int64_t l = 0; l < z->L; ++l) {
    /* two norm weights; with biases also two norm biases, the four attention biases and the
     * bias of the feed-forward output, all of the hidden size; then the biases of the
     * feed-forward inputs, of the feed-forward size */
    int small = 2 + (int)bias * 7, wide = (int)bias * (z->K - 5);
    for (int k = 0; k < small; ++k) emit(s, +1, B16 * H);
    for (int k = 0; k < wide; ++k) emit(s, +1, B16 * F);
  }
  for (int k = 0; k < 1 + (int)bias; ++k) emit(s, +1, B16 * H);
  emit(s, +1, z->lm_p);
  for (int k = 0; k < z->e_n; ++k) emit(s, +1, z->out);
  for (int64_t l = 0; l < z->L; ++l)
    for (int k = 0; k < z->n_ops; ++k) emit(s, +1, op_size(z, k));
  emit(s, +1, z->logit);
  emit(s, +1, z->shift);
  emit(s, +1, z->shift);
}

/* raw list of the second estimator (malloc'd, caller frees) with the byte guard */
static int dnn_build(const oracle_config *c, int64_t **list_out, int64_t *n_out) {
  *list_out = NULL;
  *n_out = 0;
  int st = dnn_validate(c);
  if (st) return st;
  sizes_t z;
  compute_sizes(c, &z);
  sink_t counter = {NULL, 0, 0};
  dnn_walk(c, &z, &counter);
  if (counter.overflow || (u128)counter.n >= COUNT_LIMIT) return ST_OVERFLOW;
  int64_t *d = (int64_t *)malloc((size_t)counter.n * sizeof(int64_t));
  if (!d) return -1;
  sink_t writer = {d, 0, 0};
  dnn_walk(c, &z, &writer);
  u128 run = (u128)c->base_bytes;
  int bad = 0;
  for (int64_t k = 0; k < writer.n && !bad; ++k) {
    run += align512((u128)d[k]);
    if (run >= BYTES_LIMIT) bad = 1;
  }
  if (bad) {
    free(d);
    return ST_OVERFLOW;
  }
  *list_out = d;
  *n_out = writer.n;
  return ST_OK;
}

int oracle_dnn_event_count(const oracle_config *c, int64_t *count_out) {
  int64_t *d;
  int st = dnn_build(c, &d, count_out);
  free(d);
  return st;
}

int oracle_dnn_expand_events(const oracle_config *c, int64_t *dst, int64_t capacity) {
  int64_t *d, n;
  int st = dnn_build(c, &d, &n);
  if (st) return st;
  if (capacity < n) {
    free(d);
    return -1;
  }
  memcpy(dst, d, (size_t)n * sizeof(int64_t));
  free(d);
  return ST_OK;
}

/* every magnitude up to a multiple of 512 bytes, the sign kept */
void oracle_dnn_round_events(int64_t *d, int64_t n) {
  for (int64_t k = 0; k < n; ++k) {
    if (d[k] >= 0)
      d[k] = (int64_t)align512((u128)d[k]);
    else
      d[k] = -(int64_t)align512((u128)(-(i128)d[k]));
  }
}

/* explicit list, alignment, linear scan; m_base is added as it is */
int oracle_dnn_estimate(const oracle_config *c, int64_t *peak_out, int64_t *index_out, int64_t *count_out) {
  *peak_out = -1;
  *index_out = -1;
  if (count_out) *count_out = 0;
  int64_t *d, n;
  int st = dnn_build(c, &d, &n);
  if (st) return st;
  oracle_dnn_round_events(d, n);
  int64_t best, arg;
  oracle_scan_peak(d, n, &best, &arg);
  free(d);
  *peak_out = c->base_bytes + best;
  *index_out = arg;
  if (count_out) *count_out = n;
  return ST_OK;
}

/* inventory, for the pins: e_n, K, C, embed_p, other_p, lm_p (bytes), tok_p, pos_p, hh_p, hf_p */
int oracle_inventory(const oracle_config *c, int64_t out[10]) {
  int st = oracle_validate(c);
  if (st) return st;
  sizes_t z;
  compute_sizes(c, &z);
  out[0] = z.e_n;
  out[1] = z.K;
  out[2] = (int64_t)z.C;
  out[3] = (int64_t)z.embed_p;
  out[4] = (int64_t)z.other_p;
  out[5] = (int64_t)z.lm_p;
  out[6] = (int64_t)z.tok_p;
  out[7] = (int64_t)z.pos_p;
  out[8] = (int64_t)z.hh_p;
  out[9] = (int64_t)z.hf_p;
  return ST_OK;
}

/* ------------------------------------------------------------------------ */
/* level 2: per-phase sums instead of an explicit list                      */
/* ------------------------------------------------------------------------ */
typedef struct {
  u128 init, gather, os, offset; /* batch-independent */
  u128 count;
  sizes_t z;
} phases_t;

static void static_phases(const oracle_config *c, phases_t *p) {
  compute_sizes(c, &p->z);
  const sizes_t *z = &p->z;
  p->init = page_round(z->p16_embed) + page_round(z->p32_embed) +
            z->C * (page_round(z->p16_chunk) + page_round(z->p32_chunk));
  p->gather = z->gather ? page_round(z->gat_embed) + z->C * page_round(z->gat_chunk) : 0;
  p->os = page_round(z->os_tok) + (c->pos_len > 0 ? page_round(z->os_pos) : 0) +
          (u128)z->L * (4 * page_round(z->os_hh) + (u128)(z->K - 4) * page_round(z->os_hf));
  p->offset = (u128)c->base_bytes + z->lm_p;
  p->count = event_count_formula(c, z);
}

static u128 dynamic_phase(const sizes_t *z) {
  u128 per_layer = 0;
  for (int k = 0; k < z->n_ops; ++k) per_layer += page_round(op_size(z, k));
  return (u128)z->e_n * page_round(z->out) + (u128)z->L * per_layer + page_round(z->logit) +
         2 * page_round(z->shift) + (z->tpback ? (u128)z->L * page_round(z->back) : 0);
}

int oracle_estimate_collapsed(const oracle_config *c, int64_t *peak_out) {
  *peak_out = -1;
  int st = oracle_validate(c);
  if (st) return st;
  phases_t p;
  static_phases(c, &p);
  if (p.count >= COUNT_LIMIT) return ST_OVERFLOW;
  u128 dyn = p.gather + dynamic_phase(&p.z);
  /* iteration 1 peaks before the optimizer states exist; they are allocated
   * after its frees; every later iteration peaks on top of them */
  u128 first = p.init + dyn;
  u128 after = p.init + p.os;
  u128 later = p.init + p.os + dyn;
  u128 rel = c->iters >= 2 ? later : (first > after ? first : after);
  if (p.offset + rel >= BYTES_LIMIT) return ST_OVERFLOW;
  *peak_out = (int64_t)(p.offset + rel);
  return ST_OK;
}

/* ------------------------------------------------------------------------ */
/* step 5: Algorithm 1                                                      */
/* ------------------------------------------------------------------------ */
/* Largest batch in 1..bmax whose peak does not exceed capacity, found by the
 * literal increment of Algorithm 1; 0 when batch 1 already exceeds it; -1 when
 * the shape itself is unusable (status returned through *status_out). */
int32_t oracle_max_batch(const oracle_config *shape, int64_t capacity, int32_t bmax,
                         int *status_out) {
  oracle_config c = *shape;
  c.batch = 1;
  int st = validate_fields(&c, 0);
  if (!st) st = validate_combo(&c);
  if (!st) {
    sizes_t z;
    compute_sizes(&c, &z);
    if (event_count_formula(&c, &z) >= COUNT_LIMIT) st = ST_OVERFLOW;
  }
  if (status_out) *status_out = st;
  if (st) return -1;
  int32_t bs = 1;
  for (;;) {
    if (bs > bmax) break;
    c.batch = bs;
    int64_t peak, idx;
    int e = oracle_estimate(&c, &peak, &idx, NULL);
    if (e != ST_OK || peak > capacity) break; /* m_peak > m_total */
    bs = bs + 1;
  }
  return bs - 1;
}

int32_t oracle_max_batch_bisect(const oracle_config *shape, int64_t capacity, int32_t bmax,
                                int *status_out) {
  oracle_config c = *shape;
  c.batch = 1;
  int st = validate_fields(&c, 0);
  if (!st) st = validate_combo(&c);
  if (!st) {
    sizes_t z;
    compute_sizes(&c, &z);
    if (event_count_formula(&c, &z) >= COUNT_LIMIT) st = ST_OVERFLOW;
  }
  if (status_out) *status_out = st;
  if (st) return -1;
  int32_t lo = 0, hi = bmax; /* fits(lo) (or lo == 0), answer in [lo, hi] */
  while (lo < hi) {
    int32_t mid = lo + (hi - lo + 1) / 2;
    c.batch = mid;
    int64_t peak;
    int e = oracle_estimate_collapsed(&c, &peak);
    if (e == ST_OK && peak <= capacity)
      lo = mid;
    else
      hi = mid - 1;
  }
  return lo;
}

#define SELECT_ALLZERO 1u /* offload only when every score is 0 (prose of Section 6) */

typedef int32_t (*max_batch_fn)(const oracle_config *, int64_t, int32_t, int *);

/* The decision of Algorithm 1 once the four largest batches are known:
 * scores, first maximum in the order CDP, ADP, TP, DP+TP, and the CPU-offload
 * sentinel (4, 0).  Scores are doubled so that CDP's factor 1.5 stays integral.
 * dp_n = gpu_n / tp_n; a DP+TP slot with batch 0 scores 0 whatever tp_n is. */
void oracle_decide(const int32_t bs_list[4], int32_t gpu_n, int32_t tp_n, uint32_t flags,
                   int32_t *method_out, int32_t *batch_out) {
  int64_t n = gpu_n;
  int64_t eval2[4];
  eval2[0] = (int64_t)bs_list[0] * n * 3;
  eval2[1] = (int64_t)bs_list[1] * n * 2;
  eval2[2] = (int64_t)bs_list[2] * 2;
  eval2[3] = bs_list[3] > 0 ? (int64_t)bs_list[3] * (n / tp_n) * 2 : 0;
  int idx = 0;
  for (int i = 1; i < 4; ++i)
    if (eval2[i] > eval2[idx]) idx = i; /* ties keep the earlier method */
  int any = eval2[0] || eval2[1] || eval2[2] || eval2[3];
  int keep = (flags & SELECT_ALLZERO) ? any : (eval2[2] != 0);
  if (keep) {
    *method_out = idx;
    *batch_out = bs_list[idx];
  } else {
    *method_out = 4; /* CPU offloading */
    *batch_out = 0;
  }
}

static int select_with(max_batch_fn mb, const oracle_config *shape, int64_t capacity,
                       int32_t bmax, uint32_t flags, int32_t *method_out, int32_t *batch_out,
                       int32_t bs_list[4]) {
  *method_out = -1;
  *batch_out = -1;
  for (int i = 0; i < 4; ++i) bs_list[i] = -1;
  oracle_config c = *shape;
  c.batch = 1;
  c.method = M_CDP;
  int st = validate_fields(&c, 0);
  if (st) return st;
  for (int i = 0; i < 4; ++i) {
    c.method = (uint8_t)i; /* configure method i */
    int mst;
    int32_t bs = mb(&c, capacity, bmax, &mst);
    if (bs < 0) bs = 0; /* a method that cannot be configured scores 0 */
    bs_list[i] = bs;
  }
  oracle_decide(bs_list, c.gpu_n, c.tp_n, flags, method_out, batch_out);
  return ST_OK;
}

int oracle_select_method(const oracle_config *shape, int64_t capacity, int32_t bmax,
                         uint32_t flags, int32_t *method_out, int32_t *batch_out,
                         int32_t bs_list[4]) {
  return select_with(oracle_max_batch, shape, capacity, bmax, flags, method_out, batch_out,
                     bs_list);
}

int oracle_select_method_bisect(const oracle_config *shape, int64_t capacity, int32_t bmax,
                                uint32_t flags, int32_t *method_out, int32_t *batch_out,
                                int32_t bs_list[4]) {
  return select_with(oracle_max_batch_bisect, shape, capacity, bmax, flags, method_out,
                     batch_out, bs_list);
}

/* ------------------------------------------------------------------------ */
/* batched drivers (plain loops; optional threads for the timed baseline)   */
/* ------------------------------------------------------------------------ */
typedef struct {
  int kind; /* 0 estimate (level 1), 1 collapsed, 2 max batch (linear), 3 max batch (bisect),
               4 select (linear), 5 select (bisect), 6 list checksums, 7 second estimator */
  const oracle_config *cfg;
  int64_t n;
  const int64_t *caps;
  int32_t n_cap, bmax;
  uint32_t flags;
  int64_t *peak, *index, *count;
  uint8_t *status;
  int32_t *bs, *method, *batch, *bs_list;
  uint64_t *digest_a, *digest_b;
  int64_t next; /* shared work counter */
  pthread_mutex_t lock;
} job_t;

#define JOB_BLOCK 16

static void run_one(job_t *j, int64_t i) {
  const oracle_config *c = j->cfg + i;
  if (j->kind == 0) {
    int64_t peak, idx, cnt;
    int st = oracle_estimate(c, &peak, &idx, &cnt);
    j->peak[i] = peak;
    if (j->index) j->index[i] = idx;
    if (j->count) j->count[i] = cnt;
    if (j->status) j->status[i] = (uint8_t)st;
  } else if (j->kind == 1) {
    int64_t peak;
    int st = oracle_estimate_collapsed(c, &peak);
    j->peak[i] = peak;
    if (j->status) j->status[i] = (uint8_t)st;
  } else if (j->kind == 7) {
    int64_t peak, idx, cnt;
    int st = oracle_dnn_estimate(c, &peak, &idx, &cnt);
    j->peak[i] = peak;
    if (j->index) j->index[i] = idx;
    if (j->count) j->count[i] = cnt;
    if (j->status) j->status[i] = (uint8_t)st;
  } else if (j->kind == 6) {
    int st = oracle_list_digest(c, &j->digest_a[i], &j->digest_b[i]);
    if (j->status) j->status[i] = (uint8_t)st;
  } else if (j->kind == 2 || j->kind == 3) {
    for (int32_t m = 0; m < j->n_cap; ++m) {
      int st;
      j->bs[i * j->n_cap + m] = (j->kind == 2 ? oracle_max_batch : oracle_max_batch_bisect)(
          c, j->caps[m], j->bmax, &st);
      if (j->status) j->status[i] = (uint8_t)st;
    }
  } else {
    for (int32_t m = 0; m < j->n_cap; ++m) {
      int64_t o = i * j->n_cap + m;
      int32_t bl[4];
      int st = (j->kind == 4 ? oracle_select_method : oracle_select_method_bisect)(
          c, j->caps[m], j->bmax, j->flags, &j->method[o], &j->batch[o], bl);
      if (j->bs_list) memcpy(j->bs_list + 4 * o, bl, sizeof bl);
      if (j->status) j->status[i] = (uint8_t)st;
    }
  }
}

static void *worker(void *arg) {
  job_t *j = (job_t *)arg;
  for (;;) {
    pthread_mutex_lock(&j->lock);
    int64_t lo = j->next;
    j->next += JOB_BLOCK;
    pthread_mutex_unlock(&j->lock);
    if (lo >= j->n) break;
    int64_t hi = lo + JOB_BLOCK < j->n ? lo + JOB_BLOCK : j->n;
    for (int64_t i = lo; i < hi; ++i) run_one(j, i);
  }
  return NULL;
}

static void run_job(job_t *j, int nthreads) {
  j->next = 0;
  if (nthreads <= 1) {
    for (int64_t i = 0; i < j->n; ++i) run_one(j, i);
    return;
  }
  if (nthreads > 256) nthreads = 256;
  pthread_t th[256];
  pthread_mutex_init(&j->lock, NULL);
  int started = 0;
  for (int t = 0; t < nthreads; ++t)
    if (pthread_create(&th[started], NULL, worker, j) == 0) started++;
  if (started == 0) worker(j);
  for (int t = 0; t < started; ++t) pthread_join(th[t], NULL);
  pthread_mutex_destroy(&j->lock);
}

void oracle_estimate_many(const oracle_config *cfg, int64_t n, int64_t *peak, int64_t *index,
                          uint8_t *status, int64_t *count, int level, int nthreads) {
  job_t j;
  memset(&j, 0, sizeof j);
  j.kind = level == 2 ? 1 : 0;
  j.cfg = cfg;
  j.n = n;
  j.peak = peak;
  j.index = index;
  j.status = status;
  j.count = count;
  run_job(&j, nthreads);
}

void oracle_dnn_estimate_many(const oracle_config *cfg, int64_t n, int64_t *peak, int64_t *index,
                              uint8_t *status, int64_t *count, int nthreads) {
  job_t j;
  memset(&j, 0, sizeof j);
  j.kind = 7;
  j.cfg = cfg;
  j.n = n;
  j.peak = peak;
  j.index = index;
  j.status = status;
  j.count = count;
  run_job(&j, nthreads);
}

void oracle_list_digest_many(const oracle_config *cfg, int64_t n, uint64_t *digest_a,
                             uint64_t *digest_b, uint8_t *status, int nthreads) {
  job_t j;
  memset(&j, 0, sizeof j);
  j.kind = 6;
  j.cfg = cfg;
  j.n = n;
  j.digest_a = digest_a;
  j.digest_b = digest_b;
  j.status = status;
  run_job(&j, nthreads);
}

void oracle_max_batch_many(const oracle_config *cfg, int64_t n, const int64_t *caps,
                           int32_t n_cap, int32_t bmax, int32_t *bs, uint8_t *status, int level,
                           int nthreads) {
  job_t j;
  memset(&j, 0, sizeof j);
  j.kind = level == 2 ? 3 : 2;
  j.cfg = cfg;
  j.n = n;
  j.caps = caps;
  j.n_cap = n_cap;
  j.bmax = bmax;
  j.bs = bs;
  j.status = status;
  run_job(&j, nthreads);
}

void oracle_select_many(const oracle_config *cfg, int64_t n, const int64_t *caps, int32_t n_cap,
                        int32_t bmax, uint32_t flags, int32_t *method, int32_t *batch,
                        int32_t *bs_list, uint8_t *status, int level, int nthreads) {
  job_t j;
  memset(&j, 0, sizeof j);
  j.kind = level == 2 ? 5 : 4;
  j.cfg = cfg;
  j.n = n;
  j.caps = caps;
  j.n_cap = n_cap;
  j.bmax = bmax;
  j.flags = flags;
  j.method = method;
  j.batch = batch;
  j.bs_list = bs_list;
  j.status = status;
  run_job(&j, nthreads);
}

/* ------------------------------------------------------------------------ */
/* extension: the decision of Algorithm 1 over an arbitrary candidate list  */
/* ------------------------------------------------------------------------ */
/* Section 6 scores a fixed list of four candidates.  Here a group holds any number
 * of candidates (method, gpu_n, tp_n), each with its largest batch per capacity, e.g.
 * every DP+TP split of every degree up to the number of devices at hand (Section 7.4
 * remarks that DP+TP admits several combinations).  Score of a candidate, as in
 * Algorithm 1: CDP 1.5 bs gpu_n, ADP bs gpu_n, TP bs, DP+TP bs gpu_n / tp_n; a
 * candidate with bs <= 0 (does not fit, or not admissible) scores 0.  The first
 * candidate with the largest score wins; if every score is 0 the answer is CPU
 * offloading: item -1, method 4, batch 0.
 *   item_cfg[n_items]        method, gpu_n, tp_n read
 *   bs[n_items][n_cap]
 *   group_offsets[n_groups+1] items of group g are [group_offsets[g], group_offsets[g+1])
 *   outputs [n_groups][n_cap] */
void oracle_select_segmented(const oracle_config *item_cfg, const int32_t *bs,
                             const int64_t *group_offsets, int64_t n_groups, int32_t n_cap,
                             int64_t *item_out, int32_t *method_out, int32_t *batch_out) {
  for (int64_t g = 0; g < n_groups; ++g) {
    for (int32_t m = 0; m < n_cap; ++m) {
      int64_t best_item = -1;
      i128 best_score = 0; /* doubled */
      for (int64_t i = group_offsets[g]; i < group_offsets[g + 1]; ++i) {
        const oracle_config *c = item_cfg + i;
        int64_t b = bs[i * n_cap + m];
        i128 score2 = 0;
        if (b > 0) {
          if (c->method == M_CDP) score2 = (i128)3 * b * c->gpu_n;
          else if (c->method == M_ADP) score2 = (i128)2 * b * c->gpu_n;
          else if (c->method == M_TP) score2 = (i128)2 * b;
          else if (c->method == M_DPTP && c->tp_n > 0) score2 = (i128)2 * b * (c->gpu_n / c->tp_n);
        }
        if (score2 > best_score) { /* strict: the first of equals stays */
          best_score = score2;
          best_item = i;
        }
      }
      int64_t o = g * n_cap + m;
      item_out[o] = best_item;
      method_out[o] = best_item >= 0 ? item_cfg[best_item].method : 4;
      batch_out[o] = best_item >= 0 ? bs[best_item * n_cap + m] : 0;
    }
  }
}

/* ------------------------------------------------------------------------ */
/* extension: chunk size search                                             */
/* ------------------------------------------------------------------------ */
/* Section 4.1 says only that the chunk manager picks the chunk size that wastes the least
 * memory for the given model.  Reading: the parameters outside the embedding occupy
 * ceil(other_p / cs) whole chunks (Section 4.2, m_p), so a candidate cs wastes
 * ceil(other_p / cs) * cs - other_p elements; among the candidates
 * cs_min, cs_min + cs_step, ... (n_candidates of them) the first one with the least waste
 * is chosen.  The record's own chunk_elems is ignored.  Returns the status; on status 0
 * *chunk_out and *waste_out (elements) are set, otherwise both are -1. */
int oracle_chunk_search(const oracle_config *cfg, int64_t cs_min, int64_t cs_step, int32_t n_candidates,
                        int64_t *chunk_out, int64_t *waste_out) {
  *chunk_out = -1;
  *waste_out = -1;
  oracle_config c = *cfg;
  c.chunk_elems = 1;
  int st = validate_fields(&c, 0);
  if (st) return st;
  if (c.method > 3) return ST_FIELD;
  sizes_t z;
  compute_sizes(&c, &z);
  u128 best_waste = 0;
  int64_t best_cs = -1;
  for (int32_t k = 0; k < n_candidates; ++k) {
    u128 cs = (u128)cs_min + (u128)k * (u128)cs_step;
    u128 waste = ceil_div(z.other_p, cs) * cs - z.other_p;
    if (best_cs < 0 || waste < best_waste) { /* strict: the first of equals stays */
      best_waste = waste;
      best_cs = (int64_t)cs;
    }
  }
  *chunk_out = best_cs;
  *waste_out = (int64_t)best_waste;
  return ST_OK;
}
