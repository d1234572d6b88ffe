/*
 * llmem.h -- C ABI of the batched LLMem peak-memory estimator for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for very many fine-tuning configurations at once, the
 * peak per-device memory model of Kim et al., "LLMem: Estimating GPU Memory
 * Usage for Fine-Tuning Pre-Trained LLMs" (arXiv 2404.10933):
 *
 *   Section 4.2   m_peak^s = m_base + m_p + m_os + m_out + m_lm        (single device / CDP)
 *   Section 5     m_peak^dp, m_peak^tp, m_peak^dp+tp and m_back^tp     (ZeRO-3, 1-D TP, DP+TP)
 *   Section 6     Algorithm 1: largest batch per method, scores, selection
 *
 * Every term is expanded into allocate/free events in the phase order of
 * Sections 4.1 and 5 (initialisation, gather, output phase, TP backward
 * buffers, frees, optimizer states in the first iteration); every event is
 * rounded up to the CUDA page size cu_p = 2 * 1024^2 bytes (Section 4.2); the
 * peak is m_base + lm_p + the largest prefix sum of the rounded list.
 *
 * Conventions
 *   - "DEV" pointers are device pointers owned by the caller; "HOST" are host
 *     pointers.  The library allocates no device memory and keeps no state
 *     between calls except the text returned by llmem_last_error().
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     default stream) and return without synchronising.  Outputs are valid once
 *     the stream has reached the end of the enqueued work.
 *   - The return code reports call-level problems (bad pointer, size, scratch,
 *     launch failure).  Problems of a single configuration are reported per
 *     element: status_out[i] != 0 and the element's outputs are -1.  Nothing
 *     traps, asserts or aborts on the device.
 *   - All byte quantities are int64.  Supported results are < 2^62 bytes and
 *     < 2^31 events per configuration; beyond that the element gets status 3.
 *   - `scratch` must be 256-byte aligned, at least llmem_scratch_bytes() long,
 *     and must not be shared by calls that may overlap on the device.
 */
#ifndef LLMEM_H_
#define LLMEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DEV
#define HOST

/* One fine-tuning configuration: the symbols of Table 1 that the equations use,
 * plus the method and its modelled partition degrees.  64 bytes, no padding. */
typedef struct __attribute__((aligned(16))) llmem_config {
  int32_t layers;      /* l_n, 1 .. 2^16 */
  int32_t hidden;      /* o_n, 1 .. 2^20 */
  int32_t heads;       /* >= 1 and a divisor of hidden; used only with act_mode = 1, where it sizes the
                          two attention-score outputs of a layer (2 * batch * heads * seq^2 bytes) */
  int32_t ffn;         /* inner width of the feed-forward block, 1 .. 2^22 */
  int32_t vocab;       /* dict_n, 1 .. 2^26 */
  int32_t pos_len;     /* rows of a learned position Embedding, 0 = none; 0 .. 2^26 (fixes e_n) */
  int32_t seq;         /* sl, 1 .. 2^26 */
  int32_t batch;       /* bs, 1 .. 2^26; ignored by llmem_max_batch / llmem_select_method */
  int64_t chunk_elems; /* cs in elements, 1 .. 2^40 */
  int64_t base_bytes;  /* m_base, 0 .. 2^60, added without rounding */
  uint8_t method;      /* LLMEM_METHOD_*; ignored by llmem_select_method */
  uint8_t gpu_n;       /* >= 1; a plain number, nothing runs across devices */
  uint8_t tp_n;        /* DP+TP only: 2 <= tp_n <= gpu_n/2 and tp_n | gpu_n */
  uint8_t lm_bytes;    /* B of the m_lm equation: 2 or 4 */
  uint8_t ffn_kind;    /* 0: two feed-forward matrices, 1: three (gated) */
  uint8_t has_bias;    /* 0 / 1: Linear biases and norm biases present */
  uint8_t iters;       /* fine-tuning iterations spanned by the event list, >= 1;
                          2 or more gives the paper's peak */
  uint8_t act_mode;    /* 0: gradient checkpointing, the layer and embedding outputs are kept (the
                          paper's m_out); 1: every operator output of every layer is kept */
  uint8_t reserved[8]; /* must be 0 */
} llmem_config;

enum { LLMEM_METHOD_CDP = 0, LLMEM_METHOD_ADP = 1, LLMEM_METHOD_TP = 2, LLMEM_METHOD_DPTP = 3,
       LLMEM_METHOD_OFFLOAD = 4 /* only ever an output of llmem_select_method */ };

typedef enum {
  LLMEM_OK = 0,
  LLMEM_ERR_ARG = 1,     /* null / misaligned pointer, negative size, bmax out of range */
  LLMEM_ERR_SCRATCH = 2, /* scratch missing, misaligned or too small */
  LLMEM_ERR_CUDA = 3,    /* a CUDA runtime call failed; text in llmem_last_error() */
  LLMEM_ERR_TIMEOUT = 4, /* a bounded device-side wait ran out (llmem_scratch_status only) */
  LLMEM_ERR_CHECK = 5    /* an index check of a checked build failed (llmem_scratch_status only) */
} llmem_status;

/* per-configuration status bytes */
enum { LLMEM_CFG_OK = 0, LLMEM_CFG_FIELD = 1 /* a field outside its range */,
       LLMEM_CFG_COMBO = 2 /* method / gpu_n / tp_n not admissible */,
       LLMEM_CFG_OVERFLOW = 3 /* >= 2^31 events or >= 2^62 bytes */ };

/* operations, for llmem_scratch_bytes */
enum { LLMEM_OP_ESTIMATE = 0, LLMEM_OP_EVENT_COUNTS = 1, LLMEM_OP_EXPAND = 2, LLMEM_OP_ROUND = 3,
       LLMEM_OP_SCAN_PEAK = 4, LLMEM_OP_MAX_BATCH = 5, LLMEM_OP_SELECT = 6, LLMEM_OP_EXPAND_SCAN = 7 };

/* call flags */
#define LLMEM_SELECT_ALLZERO 1u /* llmem_select_method: offload only if every score is 0 */
#define LLMEM_FUSE_ROUND 2u     /* llmem_expand_events: write page-rounded deltas;
                                   llmem_scan_peak: round each delta while reading */
/* Section 3.1: estimate as the DNNMem-style procedure does that the paper implements for
 * comparison, instead of LLMem: one device without sharding (method must be LLMEM_METHOD_CDP,
 * else LLMEM_CFG_COMBO; gpu_n, tp_n, chunk_elems and iters play no part), the weight tensors
 * as loaded (fp16, the lm_head in lm_bytes) and a constant 64 MB buffer, then the outputs of
 * the forward pass (embedding outputs, layer outputs or, with act_mode 1, every operator
 * output, logits, two shifted copies), every tensor aligned to 512 bytes instead of the 2 MiB
 * page.  The list has no frees: its peak is m_base + its total.  Event order: buffer, token
 * (position) embedding, the Linear matrices layer by layer, the vectors layer by layer (norm
 * weights, then norm / attention / feed-forward output biases, then feed-forward input
 * biases), final norm, lm_head, forward outputs.  Accepted by llmem_estimate_batch,
 * llmem_event_counts(_static), llmem_expand_events (LLMEM_FUSE_ROUND then aligns to 512 bytes),
 * llmem_expand_scan (only together with LLMEM_FUSE_ROUND) and llmem_scan_peak (then cfg adds
 * m_base alone; not together with LLMEM_FUSE_ROUND, which rounds to the 2 MiB page); refused
 * by llmem_max_batch and llmem_select_method (Algorithm 1 is LLMem's). */
#define LLMEM_ESTIMATOR_DNNMEM 4u

/* Bytes of scratch the operation needs for n configurations and total_events
 * events (0 where it needs none; such calls accept scratch = NULL).  For
 * LLMEM_OP_EXPAND the scratch is optional (see llmem_expand_events).  For
 * LLMEM_OP_EXPAND, LLMEM_OP_SCAN_PEAK and LLMEM_OP_EXPAND_SCAN the size depends on
 * total_events too (lists of short segments keep per-segment records there). */
size_t llmem_scratch_bytes(int op, int64_t n, int64_t total_events);

/* Sections 4.2 and 5, fused: peak of each configuration without materialising
 * its event list (identical runs of events are summed in registers).
 *   cfg            DEV [n]
 *   peak_out       DEV [n]   m_base + lm_p + largest prefix sum of the rounded events, -1 on status != 0
 *   peak_index_out DEV [n]   nullable; 0-based index of the first event whose prefix attains the peak
 *   status_out     DEV [n]   nullable; LLMEM_CFG_* */
llmem_status llmem_estimate_batch(const llmem_config* DEV cfg, int64_t n, int64_t* DEV peak_out,
                                  int64_t* DEV peak_index_out, uint8_t* DEV status_out,
                                  void* DEV scratch, size_t scratch_bytes, uint32_t flags,
                                  void* cuda_stream);

/* Sections 4.1 and 5: number of allocate/free events of each configuration
 * (0 on status != 0) as an exclusive prefix sum.
 *   offsets_out    DEV [n+1] offsets_out[0] = 0, offsets_out[n] = total number of events
 *   status_out     DEV [n]   nullable */
llmem_status llmem_event_counts(const llmem_config* DEV cfg, int64_t n, int64_t* DEV offsets_out,
                                uint8_t* DEV status_out, void* DEV scratch, size_t scratch_bytes,
                                uint32_t flags, void* cuda_stream);

/* Largest n accepted by llmem_event_counts_static. */
#define LLMEM_STATIC_MAX_CONFIGS 4194304

/* No counterpart in the paper: a convenience of this library.  Same results as
 * llmem_event_counts, bit for bit, for callers that are not in a position to
 * provide scratch because they cannot allocate device memory at the point of
 * the call: code running under a framework whose allocator they may not re-enter
 * (a callback, a custom-op hook), services that pre-size all device memory at
 * start-up and forbid cudaMalloc afterwards, and callers preparing a sequence of
 * work in which an allocation would force a device-wide synchronisation.  They
 * still pass the input and output buffers; only the scratch is supplied by the
 * library.
 *
 * The scratch (one partial sum per 1024 configurations) is a fixed array of about
 * 32 KiB in the library's device image; every GPU on which the library is used
 * holds it until the process exits.  Hence the limit: n <= LLMEM_STATIC_MAX_CONFIGS,
 * larger n returns LLMEM_ERR_ARG with an explanatory llmem_last_error() and does no
 * work.  The call itself performs no cudaMalloc, cudaFree or other allocation.
 *
 * The first call on each device looks up the array's device address (a query, not
 * an allocation) and caches it; make that first call in ordinary stream execution,
 * before any stream capture is begun on that device.  The cached address belongs to the
 * device's current context: do not call cudaDeviceReset() between uses of this entry point.
 *
 * All calls on one device share the one array, and it keeps what the previous call
 * left there.  That is harmless for calls that follow one another in one stream
 * (each call writes every entry before reading it), but two calls that may run on the
 * GPU at the same time -- different streams, different host threads -- race on it and
 * yield undefined offsets.  Serialise them, or use llmem_event_counts with separate
 * scratch buffers.
 *   cfg         DEV [n]
 *   offsets_out DEV [n+1]
 *   status_out  DEV [n], nullable */
llmem_status llmem_event_counts_static(const llmem_config* DEV cfg, int64_t n,
                                       int64_t* DEV offsets_out, uint8_t* DEV status_out,
                                       uint32_t flags, void* cuda_stream);

/* No counterpart in the paper: support for grids whose event lists do not fit in device
 * memory at once (Section 4.2's shapes times every batch, method and degree give lists of
 * hundreds of gigabytes).  Cuts configurations [first, n) into contiguous slabs of at most
 * max_events events each, greedily (every slab takes as many configurations as fit; a
 * configuration with more events than max_events is a slab of its own), so that each slab can
 * be expanded and scanned through one reusable list buffer.
 *   offsets     DEV [n+1]  as written by llmem_event_counts
 *   bounds_out  DEV [max_slabs+1]  slab k holds configurations bounds_out[k] .. bounds_out[k+1]-1;
 *                          bounds_out[0] = first, the last one written is n
 *   events_out  DEV [max_slabs+1]  offsets[bounds_out[k]]: slab k has events_out[k+1] - events_out[k] events
 *   count_out   DEV [1]    number of slabs, or -1 if max_slabs slabs do not reach n */
llmem_status llmem_slab_bounds(const int64_t* DEV offsets, int64_t n, int64_t max_events, int64_t first,
                               int64_t* DEV bounds_out, int64_t* DEV events_out, int64_t max_slabs,
                               int64_t* DEV count_out, void* cuda_stream);

/* Sections 4.1 and 5: the signed byte count of every event, allocations
 * positive and frees negative, configuration i occupying
 * delta_out[offsets[i] .. offsets[i+1]).  Order: initialisation (embedding unit,
 * then each chunk: fp16, fp32); per iteration gather, embedding and layer
 * outputs, logits, two shifted copies, TP backward buffers, then the frees in
 * reverse; optimizer states (per Embedding / Linear tensor) after the first
 * iteration.  With LLMEM_FUSE_ROUND the magnitudes are page-rounded.
 *   offsets        DEV [n+1] as written by llmem_event_counts for the same cfg
 *   total_events   HOST value of offsets[n]
 *   delta_out      DEV [total_events], 8-byte aligned (16-byte alignment enables bulk stores)
 *   scratch        DEV, optional: llmem_scratch_bytes(LLMEM_OP_EXPAND, n, total_events) bytes,
 *                  256-byte aligned.  For lists of long segments it holds the counter from which
 *                  the warps of a persistent grid claim blocks of the list; for lists whose
 *                  segments are short on average (about 1 KB per configuration then) the table of
 *                  segment descriptors from which every segment is written by one lane or warp.
 *                  With scratch = NULL (or too small) the list is cut into blocks handed out by
 *                  the hardware block scheduler, one warp per block.  The list written is the
 *                  same either way. */
llmem_status llmem_expand_events(const llmem_config* DEV cfg, int64_t n, const int64_t* DEV offsets,
                                 int64_t total_events, int64_t* DEV delta_out, void* DEV scratch,
                                 size_t scratch_bytes, uint32_t flags, void* cuda_stream);

/* Section 4.2, every ceil(x / cu_p) * cu_p: round each magnitude up to a
 * multiple of 2 MiB in place, keeping the sign. */
llmem_status llmem_round_events(int64_t* DEV delta, int64_t total_events, void* DEV scratch,
                                size_t scratch_bytes, uint32_t flags, void* cuda_stream);

/* Sections 4.2 and 5 (the peaks are these sums): per segment, the largest
 * prefix sum of delta[offsets[i] .. offsets[i+1]) and the first index attaining
 * it, plus m_base + lm_p of cfg[i] when cfg is given.  An empty segment yields
 * offset + 0 and index -1; with cfg, an inadmissible cfg[i] yields -1 / -1.
 *   delta          DEV [total_events]; any signed values whose prefix sums stay within int64
 *   cfg            DEV [n], nullable (then the offset is 0)
 *   scratch        required, llmem_scratch_bytes(LLMEM_OP_SCAN_PEAK, n, total_events) bytes;
 *                  holds a device status word readable with llmem_scratch_status */
llmem_status llmem_scan_peak(const int64_t* DEV delta, const int64_t* DEV offsets, int64_t n,
                             int64_t total_events, const llmem_config* DEV cfg,
                             int64_t* DEV peak_out, int64_t* DEV peak_index_out, void* DEV scratch,
                             size_t scratch_bytes, uint32_t flags, void* cuda_stream);

/* llmem_expand_events and llmem_scan_peak in one pass (Sections 4.1, 4.2 and 5): the list
 * is written exactly as llmem_expand_events writes it (raw sizes, or page-rounded with
 * LLMEM_FUSE_ROUND) and, while each piece of it is still in shared memory, folded into the
 * per-configuration peak of the page-rounded list (a piece that is one run of equal or of
 * two alternating events is folded in closed form: its prefix sums are arithmetic
 * progressions).  Outputs are those of llmem_scan_peak(..., cfg, ...) on the rounded list:
 * m_base + lm_p + largest prefix sum, first index attaining it, -1 / -1 for an
 * inadmissible cfg[i].  The list is written to device memory once and not read back.
 *   offsets        DEV [n+1]  as written by llmem_event_counts for the same cfg
 *   total_events   HOST value of offsets[n]
 *   delta_out      DEV [total_events]
 *   peak_out       DEV [n]
 *   peak_index_out DEV [n], nullable
 *   scratch        required, llmem_scratch_bytes(LLMEM_OP_EXPAND_SCAN, n, total_events) bytes
 *                  (for the same n and total_events: lists whose segments are short on average
 *                  need about 1 KB per configuration more, for a table of segment descriptors),
 *                  256-byte aligned; the call clears its header (status word, work counter)
 *                  and rewrites what it reads, so the buffer may be reused by later calls in
 *                  the same stream, but not by calls that may run at the same time */
llmem_status llmem_expand_scan(const llmem_config* DEV cfg, int64_t n, const int64_t* DEV offsets,
                               int64_t total_events, int64_t* DEV delta_out, int64_t* DEV peak_out,
                               int64_t* DEV peak_index_out, void* DEV scratch, size_t scratch_bytes,
                               uint32_t flags, void* cuda_stream);

/* Algorithm 1, the inner loop of every method: the largest batch b in 1..bmax
 * whose peak does not exceed the capacity (0 if even b = 1 does not fit, -1 on
 * status != 0).  The paper increments b; the peak is non-decreasing in b, so the
 * library bisects.
 *   shape          DEV [n]      method, gpu_n, tp_n used; batch ignored
 *   capacity_bytes DEV [n_cap]  m_total values
 *   bmax           1 .. 2^26
 *   bs_out         DEV [n][n_cap] */
llmem_status llmem_max_batch(const llmem_config* DEV shape, int64_t n,
                             const int64_t* DEV capacity_bytes, int32_t n_cap, int32_t bmax,
                             int32_t* DEV bs_out, uint8_t* DEV status_out, void* DEV scratch,
                             size_t scratch_bytes, uint32_t flags, void* cuda_stream);

/* Algorithm 1 in full: the four largest batches, the scores
 * [1.5 bs gpu_n, bs gpu_n, bs, bs gpu_n/tp_n], the first maximum in the order
 * CDP, ADP, TP, DP+TP, and (LLMEM_METHOD_OFFLOAD, 0) when the TP score is 0
 * (with LLMEM_SELECT_ALLZERO: when all four are 0).  A method that is not
 * admissible for (gpu_n, tp_n) scores 0.
 *   method_out, batch_out DEV [n][n_cap]
 *   bs_list_out           DEV [n][n_cap][4], nullable */
llmem_status llmem_select_method(const llmem_config* DEV shape, int64_t n,
                                 const int64_t* DEV capacity_bytes, int32_t n_cap, int32_t bmax,
                                 int32_t* DEV method_out, int32_t* DEV batch_out,
                                 int32_t* DEV bs_list_out, uint8_t* DEV status_out,
                                 void* DEV scratch, size_t scratch_bytes, uint32_t flags,
                                 void* cuda_stream);

/* Section 6 (scores and tie order of Algorithm 1) applied to candidate lists of any
 * length; Section 7.4 notes that DP+TP admits several splits once more devices are at
 * hand.  A group is a run of consecutive candidates, each a (method, gpu_n, tp_n) with its
 * largest batch per capacity as written by llmem_max_batch: for instance every method,
 * every degree up to the devices available and every admissible DP+TP split of one
 * decoder shape.  Scores as in Algorithm 1 (CDP 1.5 bs gpu_n, ADP bs gpu_n, TP bs, DP+TP
 * bs gpu_n/tp_n); a candidate with bs <= 0 scores 0; the first candidate with the largest
 * score wins; if all scores are 0 (or the group is empty) the result is CPU offloading.
 * The candidates are not checked for out-of-bounds group_offsets: these must be
 * non-decreasing and end at n_items.
 *   item_cfg      DEV [n_items]      method, gpu_n, tp_n read
 *   bs            DEV [n_items][n_cap]
 *   group_offsets DEV [n_groups+1]
 *   item_out      DEV [n_groups][n_cap]  index of the winning candidate, -1 = offloading
 *   method_out    DEV [n_groups][n_cap]  nullable; its method, LLMEM_METHOD_OFFLOAD if none
 *   batch_out     DEV [n_groups][n_cap]  nullable; its batch, 0 if none */
llmem_status llmem_select_segmented(const llmem_config* DEV item_cfg, const int32_t* DEV bs,
                                    const int64_t* DEV group_offsets, int64_t n_groups,
                                    int64_t n_items, int32_t n_cap, int64_t* DEV item_out,
                                    int32_t* DEV method_out, int32_t* DEV batch_out,
                                    void* DEV scratch, size_t scratch_bytes, uint32_t flags,
                                    void* cuda_stream);

/* Section 4.1: the chunk manager picks the chunk size that wastes the least memory for the
 * given model.  The parameters outside the embedding occupy ceil(other_p / cs) whole chunks
 * (Section 4.2, m_p), so a candidate cs wastes ceil(other_p / cs) * cs - other_p elements.
 * Among the candidates cs_min, cs_min + cs_step, ..., n_candidates of them, all within
 * 1 .. 2^40, the first with the least waste is returned.  The record's chunk_elems and
 * batch are ignored.
 *   chunk_out  DEV [n]  chosen cs in elements, -1 on status != 0
 *   waste_out  DEV [n]  nullable; wasted elements of the choice
 *   status_out DEV [n]  nullable */
llmem_status llmem_chunk_search(const llmem_config* DEV cfg, int64_t n, int64_t cs_min,
                                int64_t cs_step, int32_t n_candidates, int64_t* DEV chunk_out,
                                int64_t* DEV waste_out, uint8_t* DEV status_out, void* DEV scratch,
                                size_t scratch_bytes, uint32_t flags, void* cuda_stream);

/* Synchronises cuda_stream and returns the device status word that
 * llmem_scan_peak keeps at the start of its scratch: LLMEM_OK, or
 * LLMEM_ERR_TIMEOUT if a bounded wait inside a kernel gave up (outputs are then
 * undefined), LLMEM_ERR_CHECK if an index check of a checked build failed.  The scratch
 * may be that of llmem_scan_peak, llmem_expand_scan or llmem_expand_events. */
llmem_status llmem_scratch_status(const void* DEV scratch, void* cuda_stream);

/* No counterpart in the paper: a check of this library's own failure handling.  The scan
 * kernels wait on copy-completion barriers with a time limit; when a wait runs out they
 * record LLMEM_ERR_TIMEOUT in the scratch status word and return instead of hanging.  This
 * call exercises exactly that path without touching any data: one warp waits, for at most
 * limit_ms (1 .. 2000) milliseconds, on a barrier that nothing completes, gives up and
 * records the status.  Afterwards llmem_scratch_status(scratch, stream) must return
 * LLMEM_ERR_TIMEOUT and the CUDA context must be as usable as before.
 *   scratch  DEV, at least 256 bytes, 256-byte aligned */
llmem_status llmem_selftest_wait_limit(void* DEV scratch, size_t scratch_bytes, uint32_t limit_ms,
                                       void* cuda_stream);

/* No counterpart in the paper: a probe for the roofline of the kernels that generate events
 * in registers.  Launches 8 CTAs of 256 threads per SM in which every thread advances eight
 * independent 32-bit chains for `iters` iterations of 64 counted instructions: kind 0 add
 * and xor (the integer ALU pipe), 1 multiply-add (the pipe 32-bit multiplies share with
 * floating point), 2 the two alternating.  The caller times the launch with CUDA events;
 * *warp_instructions_out receives the number of counted warp instructions it executes
 * (loop counters and branches excluded), so rate = that / time.
 *   sink                   DEV, nullable; 8 bytes that the kernel may add to (never in practice)
 *   warp_instructions_out  HOST, nullable */
llmem_status llmem_selftest_int_rate(int kind, uint32_t iters, uint64_t* DEV sink,
                                     int64_t* warp_instructions_out, void* cuda_stream);

/* 1 if the library was compiled with -DLLMEM_DEBUG (csrc/libllmem_debug.so), else 0.  A
 * checked build tests every index its streaming kernels derive from offsets, block and
 * segment numbers before using it; a failed test skips the access and leaves its number in
 * the scratch status word, which llmem_scratch_status reports as LLMEM_ERR_CHECK.  No
 * counterpart in the paper: it stands in for a memory checker while kernels are changed. */
int llmem_checked_build(void);

/* Text of the last error on the calling thread ("" if none). */
const char* llmem_last_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int llmem_version(void);

#undef DEV
#undef HOST

#ifdef __cplusplus
}
#endif
#endif /* LLMEM_H_ */
