/*
 * heatkv.h -- C ABI of the B200 (sm_100a) HeatKV hot path.
 *
 * HeatKV (head-tuned KV-cache compression for visual autoregressive, next-scale
 * models) prunes the KV cache per attention head and per source scale with a static
 * schedule derived from calibrated attention statistics.  This library holds the
 * data-parallel part: the calibration reduction (Sec. 3.1), the schedule builder
 * (Sec. 3.2, 3.3, Appendix A), the per-head cache with append / eviction, and the
 * per-scale-step attention over the retained keys.
 *
 * Conventions
 *  - Scales ("steps"), layers and heads are 0-based here: step = k-1 for the paper's
 *    scale k, so t[step] tokens are generated at `step` and c[step] = t[0]+..+t[step].
 *  - Activations are bf16, shaped [n_seq, H, t_step, d] with d contiguous; the other
 *    three strides are given in elements by heatkv_strides (NULL = densely packed).
 *    Base pointers must be 16-byte aligned and strides multiples of 8 elements.
 *  - Every pointer is marked HOST or DEVICE.  Device buffers belong to the caller (the
 *    library never allocates or frees device memory); the library owns only the host
 *    objects behind heatkv_ctx / heatkv_schedule.  Kernels are enqueued on the given
 *    CUDA stream (a cudaStream_t passed as void*, NULL = default stream) and calls return
 *    without waiting, except the calls documented as synchronising.
 *  - Every function returns HEATKV_OK (0) or a negative heatkv_status.  Nothing throws or
 *    aborts across this boundary; a call that fails leaves cache and context unchanged.
 *  - A context is not thread-safe; use one context per thread or lock around it.
 *  - The kernels of one context share work counters and scratch inside its arena, so they must
 *    not overlap on the GPU: enqueue a context's calls on one stream, or order the streams
 *    with events.  After HEATKV_ERR_DEVICE_TIMEOUT (heatkv_device_status) a context stays in
 *    that state; destroy it and create a new one.
 */
#ifndef HEATKV_H_
#define HEATKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HEATKV_MAX_K 16          /* at most 16 scales (mask words are 16 bit)        */
#define HEATKV_MAX_BATCH 128     /* sequences per attention / append call            */
#define HEATKV_PAGE_TOKENS 64    /* rows per cache page and per key half-tile        */

typedef enum {
  HEATKV_OK = 0,
  HEATKV_ERR_INVALID_ARG = -1,
  HEATKV_ERR_SHAPE_MISMATCH = -2,
  HEATKV_ERR_BUDGET_INFEASIBLE = -3,   /* b*c_{K-1} < c_s, or the removal list ran out */
  HEATKV_ERR_OUT_OF_PAGES = -4,        /* pool or metadata region exhausted            */
  HEATKV_ERR_BAD_STEP_ORDER = -5,
  HEATKV_ERR_NAN_SCORE = -6,
  HEATKV_ERR_DEVICE_TIMEOUT = -7,      /* a bounded device-side wait gave up           */
  HEATKV_ERR_CUDA = -8,
  HEATKV_ERR_HOST_MEMORY = -9,
  HEATKV_ERR_TOO_LARGE = -10           /* the call needs more built-in scratch than the library holds */
} heatkv_status;

typedef enum { HEATKV_LAYOUT_RAGGED = 0, HEATKV_LAYOUT_PAGED = 1 } heatkv_layout;

typedef enum {
  HEATKV_POLICY_HEATKV = 0,   /* Algorithm 1, head-scale units, orders O_i from S-CAS      */
  HEATKV_POLICY_BINARY = 1,   /* Algorithm 1, head units, one order O from CAS            */
  HEATKV_POLICY_NAIVE = 2,    /* Sec. 3.3 boundary policy: prune before a scale, not after */
  HEATKV_POLICY_EXPLICIT = 3  /* per-head token fraction (no counterpart in the paper)     */
} heatkv_policy;

typedef enum {
  HEATKV_ACCOUNT_PHYSICAL = 0, /* layers not yet run hold what they held at scale start   */
  HEATKV_ACCOUNT_LITERAL = 1   /* Algorithm 2 exactly as printed                          */
} heatkv_accounting;

typedef enum {
  HEATKV_KERNEL_AUTO = 0,      /* tensor-memory kernel for steps of >= 256 queries (>= 128 once a call holds
                                  64 (sequence, head) units), generic otherwise */
  HEATKV_KERNEL_GENERIC = 1,   /* warp-level MMA kernel for every step                    */
  HEATKV_KERNEL_TCGEN05 = 2    /* tcgen05 / TMEM / TMA kernel wherever its shape rules allow */
} heatkv_kernel_choice;

typedef enum {
  HEATKV_CACHE_BF16 = 0,       /* rows stored verbatim                                            */
  HEATKV_CACHE_FP8_E4M3 = 1    /* rows stored as 8-bit codes plus one exponent byte (see below)    */
} heatkv_cache_dtype;

typedef struct heatkv_ctx heatkv_ctx;
typedef struct heatkv_schedule heatkv_schedule;

typedef struct {
  int32_t L, H, d, K;            /* layers, heads per layer, head dim (64 or 128), scales  */
  int32_t t[HEATKV_MAX_K];       /* tokens per scale, t_k = w_k * h_k (Sec. 3.1)           */
  int32_t s;                     /* sink scales always kept (Sec. 3.2); 0 allowed          */
  int32_t layout;                /* heatkv_layout                                           */
  int32_t kernel;                /* heatkv_kernel_choice                                    */
  float sm_scale;                /* logit scale; <= 0 selects 1/sqrt(d)                    */
  void* arena;                   /* DEVICE, caller-owned, 1024-byte aligned                */
  uint64_t arena_bytes;          /* metadata region + scratch region + K pool + V pool     */
  uint64_t meta_bytes;           /* bytes of the arena set aside for plans; 0 = default    */
  uint64_t scratch_bytes;        /* bytes of the arena for partial results of heads whose key range is
                                    split over several CTAs; 0 = default (1/8 of the arena, at most
                                    128 MiB); too little only disables splitting                    */
  int32_t cache_dtype;           /* heatkv_cache_dtype; FP8_E4M3 needs the paged layout                    */
  int32_t reserved0;
  uint64_t stage_bytes;          /* FP8_E4M3 only: bytes of the arena for the bf16 staging rows one attention
                                    call expands its visible keys into; 0 = default (1/8 of the arena)     */
} heatkv_config;

typedef struct {                 /* element strides of the [n_seq, H, t, d] activations    */
  int64_t q_seq, q_head, q_tok;
  int64_t kv_seq, kv_head, kv_tok;   /* shared by k and v                                  */
  int64_t o_seq, o_head, o_tok;
} heatkv_strides;

typedef struct {                 /* which kernels a context has launched so far             */
  uint32_t tcgen05_attention_ready;    /* 1: the tensor-memory attention kernel is set up on this device */
  uint32_t tcgen05_calibration_ready;  /* 1: the tensor-memory calibration kernel is set up               */
  uint64_t attention_tcgen05;    /* launches of the tcgen05 / TMEM / TMA attention kernel (carries the cache
                                    update of heatkv_attention_append in the paged layout)               */
  uint64_t attention_generic;    /* launches of the warp-level attention kernel                          */
  uint64_t calibration_tcgen05, calibration_generic;
  uint64_t append, compact;      /* stand-alone cache-update kernels                                     */
  uint64_t other;                /* small helper kernels (fixed-order reduction of the static-scratch call) */
} heatkv_kernel_stats;

typedef struct {
  uint64_t pool_rows;            /* rows (tokens) the K pool and the V pool can hold        */
  uint64_t reserved_rows;        /* rows reserved by open sequences                         */
  uint64_t used_tokens;          /* tokens held right now by open sequences                 */
  uint64_t peak_reserved_rows;   /* high-water mark of reserved_rows                        */
  uint64_t meta_bytes_used;
  uint32_t open_seqs;
  uint32_t plans;                /* schedules whose plan is resident                        */
} heatkv_alloc_stats;

/* fp8 cache (cache_dtype = HEATKV_CACHE_FP8_E4M3).  The paper names quantisation of the cache only as an
 * orthogonal direction (Sec. 5 and the conclusion) and defines no format; this one is the library's own.
 * A cached row (the d values of one token of one head, K or V) is stored as d codes of the OCP 8-bit
 * floating-point format E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, subnormals, no
 * infinities, largest finite value 448) plus one signed exponent byte e:
 *     code_j = round-to-nearest-even on the E4M3 grid of x_j * 2^-e,
 *     e = the smallest integer >= -120 with max_j |x_j| * 2^-e <= 448   (all-zero row: e = -120),
 * so a row costs d + 1 bytes instead of 2 d.  Reading gives x^_j = value(code_j) * 2^e, which a bf16 holds
 * exactly.  Attention in such a context is attention over x^ for the cached scales (the step's own K/V come
 * from k_new / v_new unquantised, as always): before the attention kernel runs, the call expands the visible
 * head-scales of its (layer, step) into bf16 staging rows inside the arena (stage_bytes), and the attention
 * kernels read those; the update after the layer quantises the new rows on their way into the pool.  Inputs
 * must be finite.  Only the paged layout is supported; heatkv_attention_append runs the expansion as a kernel of its
 * own, and the update inside the attention launch only on the generic kernel (small steps).  A call whose sequences need more staging rows than stage_bytes holds returns
 * HEATKV_ERR_OUT_OF_PAGES (rows needed per sequence: the largest number of visible 64-row half-tiles of any
 * (layer, step) of its schedule, times 64).
 *
 * Context: validates the shape, splits the arena into a metadata region and the K / V
 * pools, zero-fills the pools (enqueued on `stream`).  The arena must outlive the context.
 * With kernel = HEATKV_KERNEL_AUTO or HEATKV_KERNEL_TCGEN05 the tensor-memory kernels are set up here; if that
 * fails on a device of compute capability 10.x (or on any device under HEATKV_KERNEL_TCGEN05) the call returns
 * HEATKV_ERR_CUDA: a context never falls back to the warp-level kernel behind the caller's back.  Which kernel
 * ran is reported by heatkv_kernel_launches. */
int heatkv_create(const heatkv_config* cfg /*HOST*/, void* stream, heatkv_ctx** out /*HOST*/);
int heatkv_destroy(heatkv_ctx* ctx);

/* Sec. 3.1, Eq. 2 -- scale attention mass.  For one (layer, step) and n_seq calibration
 * sequences: attention of the t[step] queries over ALL c[step] keys (no pruning), fused
 * with the per-row probability mass on each source scale; the mean over rows is added to
 * beta_accum[layer][h][step][0..step] for every head (sum over the n_seq sequences; every
 * sequence counts as one data point d).  The attention matrix is never written out.
 *   q       DEVICE bf16 [n_seq,H,t[step],d]   strides q_*
 *   k_full  DEVICE bf16 [n_seq,H,c[step],d]   strides kv_*  (all scales up to `step`)
 *   v_full  DEVICE bf16 like k_full, or NULL when `out` is NULL
 *   seg_bias DEVICE fp32 [H][K] additive logit bias per source scale, or NULL
 *   beta_accum DEVICE fp32 [L][H][K][K], zero-initialised by the caller before the first call
 *   out     DEVICE bf16 [n_seq,H,t[step],d] strides o_*: the attention output, or NULL
 * Without an output the o_* strides are not read (they may be left zero).                */
int heatkv_calibrate_scores(heatkv_ctx* ctx, int layer, int step, int n_seq, const void* q,
                            const void* k_full, const void* v_full, const heatkv_strides* st,
                            const float* seg_bias, float* beta_accum, void* out, void* stream);

/* Sec. 3.1, Eq. 2 for the steps step_begin .. step_end - 1 of one layer in one call: offline calibration from
 * recorded activations, where the queries and keys of every scale of a sample are at hand (the beta rows of different
 * steps are independent of one another).  The steps the tensor-memory kernel takes run as ONE launch whose CTAs are
 * dispatched longest first, which evens out the rounds that a launch per step leaves partly filled; the small steps
 * share one launch of the generic kernel.  Results agree with step-by-step heatkv_calibrate_scores calls up to the
 * order of the fp32 sums.
 *   q_all   DEVICE bf16 [n_seq,H,c[step_end-1],d]  the queries of all scales, token axis = the scales one after the
 *           other, strides q_*
 *   k_all   DEVICE bf16 [n_seq,H,c[step_end-1],d]  the keys, same layout, strides kv_*
 *   seg_bias DEVICE fp32 [step_end][H][K]: the bias of step k at seg_bias + k*H*K, or NULL
 *   beta_accum as in heatkv_calibrate_scores.  The o_* strides are not read. */
int heatkv_calibrate_scores_steps(heatkv_ctx* ctx, int layer, int step_begin, int step_end, int n_seq, const void* q_all,
                                  const void* k_all, const heatkv_strides* st, const float* seg_bias, float* beta_accum,
                                  void* stream);

/* No counterpart in the paper: heatkv_calibrate_scores for callers that must not allocate device
 * memory while they run -- code inside a serving loop whose memory pool is fixed at start-up, a plug-in
 * of a host application that owns the allocator, a caller between stream-ordered allocator
 * checkpoints.  It computes the same beta update (no attention output, so no v_full / out), but every
 * CTA writes its partial masses into a 4 MiB array that is part of the library image (held by every GPU
 * that loads the library until the process exits) and a second small kernel adds them to beta_accum in a
 * fixed order; the call itself makes no cudaMalloc / cudaFree and uses no allocating library routine.
 *   Limit: ceil(t[step] / 64) * H * n_seq * 64 partial slots must fit in 2^20 floats, i.e. at most
 *   16 384 (query tile, head, sequence) CTAs; larger calls return HEATKV_ERR_TOO_LARGE and launch nothing.
 *   The first call on a device looks up the array's device address (once per device, on the device that
 *   is current); make that first call before any stream capture.
 *   All calls share the one array and it keeps the last call's contents: every slot a call reads is
 *   written by that call first, so nothing needs clearing, but two calls whose kernels overlap on the
 *   GPU (different streams) race on it -- keep them on one stream or order them yourself.
 * Arguments as in heatkv_calibrate_scores (the o_* strides are not read).  Results agree with it up to the
 * order of the fp32 sums. */
int heatkv_calibrate_scores_static(heatkv_ctx* ctx, int layer, int step, int n_seq, const void* q,
                                   const void* k_full, const heatkv_strides* st, const float* seg_bias,
                                   float* beta_accum, void* stream);

/* Text after Eq. 2, Eq. 3 and Eq. 4 -- copies beta_accum to the host (synchronises
 * `stream`), divides by n_samples = |D| and reduces in fp64:
 *   beta HOST [L][H][K][K], scas HOST [L][H][K] (0 outside s < k < K), cas HOST [L][H].
 * Any of the three outputs may be NULL.  HEATKV_ERR_NAN_SCORE if a value is not finite. */
int heatkv_finalize_scores(heatkv_ctx* ctx, const float* beta_accum /*DEVICE*/, int n_samples,
                           double* beta, double* scas, double* cas, void* stream);

/* Sec. 3.2 (Eq. 5), Sec. 3.3 (Algorithm 1), Appendix A (Algorithm 2) -- pure host code.
 * Ranks heads per source scale by ascending S-CAS (ties: ascending l*H+h), computes N_k,
 * the sets G_k, E_k (GreedyEarlyPruning) and A_k = G_{k-1} u E_k for every scale.
 *   scas HOST [L][H][K]  (HEATKV, NAIVE)      cas HOST [L][H]  (BINARY)
 *   fraction HOST [L][H] (EXPLICIT: the head stores scales 1..j, the largest prefix with
 *            c_j <= ceil(fraction * c_{K-1}), at least the sinks, and never evicts)
 *   b in (0,1]: the budget is B = floor(b * L*H * c_{K-1}) tokens (ignored by EXPLICIT).
 * Only L, H, K, t, s of cfg are read.                                                    */
int heatkv_build_schedule(const heatkv_config* cfg, const double* scas, const double* cas,
                          int policy, int accounting, double b, const double* fraction,
                          heatkv_schedule** out);
int heatkv_schedule_free(heatkv_schedule* sch);

/* Schedule as bit masks, HOST arrays of K*L*H uint16 indexed [step][layer][head]:
 *   attn_mask bit i (i < step): source scale i is in the cache and visible at `step`,
 *             i.e. i is a sink or (i,l,h) is not in A_step;
 *   keep_mask bit i (i <= step): source scale i is stored once the layer ran at `step`,
 *             i.e. i is a sink or (i,l,h) is not in G_step (last step: unchanged, nothing
 *             is appended because the last scale is never cached).
 *   n_k HOST [K] (N_k, 0 for the last step), budget_tokens = B (-1 for EXPLICIT).
 * Any output may be NULL.                                                                */
int heatkv_schedule_masks(const heatkv_schedule* sch, uint16_t* attn_mask, uint16_t* keep_mask,
                          int32_t* n_k, int64_t* budget_tokens);

/* Peak number of cached tokens over all checkpoints (scale start and after every layer)
 * and the pool rows one sequence reserves under `layout`.                                */
int heatkv_schedule_footprint(const heatkv_schedule* sch, int layout, int64_t* peak_tokens,
                              int64_t* reserved_rows);

/* The plan a sequence of this schedule runs under `layout`, as the flat int32 table the
 * kernels read (HOST copy, for inspection and tests): a 20-word header {L, H, K, n_desc,
 * word offsets of: desc, attn_begin, attn_cnt, app_begin, app_cnt, order, move, pre_begin,
 * pre_cnt, post_begin, post_cnt, then n_move, total_words, 3 spare} followed by the tables.
 * desc = {row relative to the reservation, n_valid | source_scale << 8}; move = {src, dst, n, 0};
 * the per-(step, layer, head) tables are indexed (step*L + layer)*H + head.
 * Call with words == NULL to get *n_words, then with a buffer of that many int32.        */
int heatkv_schedule_plan(const heatkv_schedule* sch, int layout, int32_t* words, int64_t* n_words);
/* The same for a context with the fp8 cache (paged layout): the attention descriptors of every (step, layer) carry
 * staging rows -- consecutive 64-row slots in descriptor order across the layer's heads -- and header word 17 is the
 * word offset of an extra table int32[n_desc] with the pool row behind every descriptor (append descriptors keep
 * pool rows).  *stage_rows (optional) = staging rows one sequence needs in an attention call: 64 per visible
 * half-tile of its busiest (step, layer).  Pure host code. */
int heatkv_schedule_plan_fp8(const heatkv_schedule* sch, int32_t* words, int64_t* n_words, int64_t* stage_rows);

/* Admit / retire one image.  Opening reserves the sequence's rows for its whole life (the
 * schedule is static, so the reservation and every page table are known up front) and, on
 * first use of a schedule, uploads its plan on `stream`.  HEATKV_ERR_OUT_OF_PAGES if the
 * pool or the metadata region cannot hold it.                                            */
int heatkv_seq_open(heatkv_ctx* ctx, const heatkv_schedule* sch, void* stream, int* seq_id);
int heatkv_seq_close(heatkv_ctx* ctx, int seq_id);

/* Sec. 3.3 -- cache update for one layer.
 *   k_new != NULL: after layer `layer` ran at `step`: store the step's K/V for every head
 *     whose (step,l,h) is not in G_step and drop the head-scales of G_step \ A_step of this
 *     layer (Sec. 3.3: these leave right after their own layer has run).  The last step stores
 *     nothing.  k_new, v_new DEVICE bf16 [n_seq,H,t[step],d], strides kv_*.
 *   k_new == NULL: before `step` starts: drop the head-scales of E_step (Sec. 3.3, Algorithm 1:
 *     the early-pruned set, gone before the scale begins) in `layer`, or in all layers when layer < 0.
 * Survivors keep their order.  In the paged layout eviction moves no data.               */
int heatkv_append_compact(heatkv_ctx* ctx, const int* seq_ids /*HOST*/, int n_seq, int layer,
                          int step, const void* k_new, const void* v_new,
                          const heatkv_strides* st, void* stream);

/* Attention of one layer at one step (Sec. 3.1 notation; Sec. 3.3 for the visible set):
 * out = softmax(sm_scale * q K^T + bias) V over the retained prior head-scales (ascending
 * scale, raster order inside) followed by the step's own t[step] keys, which always come
 * from k_new / v_new and are all visible.  bf16 operands, fp32 accumulation, probabilities
 * rounded to bf16 before the PV product.
 *   q, k_new, v_new DEVICE bf16 [n_seq,H,t[step],d]; seg_bias DEVICE fp32 [H][K] or NULL;
 *   out DEVICE bf16 [n_seq,H,t[step],d].                                                 */
int heatkv_scale_attention(heatkv_ctx* ctx, const int* seq_ids /*HOST*/, int n_seq, int layer,
                           int step, const void* q, const void* k_new, const void* v_new,
                           const heatkv_strides* st, const float* seg_bias, void* out,
                           void* stream);

/* heatkv_scale_attention followed by heatkv_append_compact(k_new != NULL) for the same (layer, step), as one
 * call: the order a model issues them in (Sec. 3.3: G_step \ A_step is evicted as soon as its layer has run).
 * In the paged layout both run in ONE kernel launch (the plan releases the pages of G_step \ A_step only
 * after the layer's append, so the new scale never lands on a page this step's attention still reads): on
 * the tensor-memory kernel two spare warps per SM copy the new rows beside the attention work, whatever the
 * update's size; on the generic kernel the copies are extra CTAs of the attention launch while the update
 * is small (up to 8 MiB of K/V, a launch-bound copy), and a larger update keeps its own bandwidth-bound
 * kernel.  In the ragged layout the in-place compaction must follow the attention, so
 * there the separate kernels run.  Arguments as in heatkv_scale_attention. */
int heatkv_attention_append(heatkv_ctx* ctx, const int* seq_ids /*HOST*/, int n_seq, int layer, int step,
                            const void* q, const void* k_new, const void* v_new, const heatkv_strides* st,
                            const float* seg_bias, void* out, void* stream);

/* How the tensor-memory attention kernel would cut the work of heatkv_scale_attention(seq_ids, layer,
 * step): *split_tiles = longest piece, in 128-key tiles, among the heads whose key range is cut (0: every
 * work item takes a whole head's key range), *items = work items of the launch (an upper bound when the
 * call mixes schedules).  A cut head's pieces leave partial results in the arena's scratch region, where
 * the last to arrive merges them.  The choice (a piece count per head) minimises an estimate of the launch's
 * makespan over the SMs and is cached per (schedule, step, layer, batch size).  Host only. */
int heatkv_attention_split(heatkv_ctx* ctx, const int* seq_ids /*HOST*/, int n_seq, int layer, int step,
                           int32_t* split_tiles, int32_t* items);

/* The search behind heatkv_attention_split, on its own (pure host code, needs no context and no GPU): given
 * the key tiles (128 keys each) of the heads of one launch in dispatch order (descending), the query tile
 * pairs per head (ceil(t_step / 256)), the sequences of the call and the SMs of the device, writes to
 * pieces[0..n_heads) into how many equal pieces every head's key range is cut (1 = whole head).  per_head = 0
 * restricts the choice to "no piece longer than some run", the rule a call that mixes schedules uses.
 * max_slots / max_ctrs bound the partial-result slots and arrival counters the cut may use (what the
 * context's scratch region holds).  The two optional outputs are the estimated makespans, in key tiles,
 * of the launch with whole heads and with the chosen cut.  Errors: INVALID_ARG for non-positive sizes or
 * tiles that are not sorted in descending order. */
int heatkv_split_plan(const int32_t* tiles /*HOST*/, int n_heads, int n_qp, int n_seq, int n_sm, int per_head,
                      uint64_t max_slots, uint64_t max_ctrs, int32_t* pieces /*HOST*/, double* makespan_whole,
                      double* makespan_cut);

/* Introspection (host state only unless noted). */
/* (With the fp8 cache a row counts d + 1 bytes instead of 2 d in both figures.)
 * Bytes of K and V the sequence holds right now, two ways: *actual = the pool rows its plan has placed for the
 * head-scales it stores (valid rows of their destination half-tiles) x d x 2 (K and V) x 2 bytes; *closed_form =
 * sum over (layer, head) of kept_tokens x d x 2 x 2 from the schedule's masks (Sec. 3.2: the cache size in
 * tokens).  The two agree unless the plan and the schedule have come apart.  Either may be NULL. */
int heatkv_cache_bytes(heatkv_ctx* ctx, int seq_id, uint64_t* actual, uint64_t* closed_form);
/* The pool rows reserved for the sequence: first row and row count (x d x 2 x 2 bytes of K and V). */
int heatkv_seq_reservation(heatkv_ctx* ctx, int seq_id, uint64_t* first_row, uint64_t* rows);
/* Global token indices c_{i-1}+j of the tokens head (layer, head) holds now; idx HOST with
 * room for c_{K-1} entries. */
int heatkv_retained_indices(heatkv_ctx* ctx, int seq_id, int layer, int head, int32_t* idx, int* n);
/* Gathers the head's cached K and V rows in logical order into DEVICE buffers of
 * n*d bf16 each (enqueued on `stream`). */
int heatkv_export_head(heatkv_ctx* ctx, int seq_id, int layer, int head, void* k_out, void* v_out,
                       void* stream);
/* The same for a context with the fp8 cache (heatkv_export_head answers HEATKV_ERR_INVALID_ARG there, and this
 * call in a bf16 context): the head's n cached rows in logical order as stored, k_codes / v_codes DEVICE
 * uint8 [n][d] (E4M3 codes) and k_exps / v_exps DEVICE int8 [n] (the rows' exponent bytes). */
int heatkv_export_head_fp8(heatkv_ctx* ctx, int seq_id, int layer, int head, void* k_codes, void* v_codes,
                           void* k_exps, void* v_exps, void* stream);
int heatkv_allocator_stats(heatkv_ctx* ctx, heatkv_alloc_stats* out);
/* Kernels launched by this context so far. */
int heatkv_launch_count(heatkv_ctx* ctx, uint64_t* n);
/* The same per kernel, with the state of the tensor-memory kernels' set-up. */
int heatkv_kernel_launches(heatkv_ctx* ctx, heatkv_kernel_stats* out);
/* Appendix on S-CAS stability -- how much the head ordering moves between calibration sets.  scas_runs HOST
 * [n_runs][L][H][K]: S-CAS of n_runs independent calibration sets (heatkv_finalize_scores).  For every prunable
 * source scale k (s <= k <= K-2, 0-based) each run ranks the L*H heads by ascending S-CAS (ties by ascending
 * l*H+h, as heatkv_build_schedule does); out[k] = mean over heads of the standard deviation (population form)
 * of the head's rank position over the runs; 0 for the other k.  out HOST [K].  Pure host code.
 * HEATKV_ERR_NAN_SCORE if a score is not finite. */
int heatkv_rank_dispersion(const double* scas_runs, int n_runs, int L, int H, int K, int s, double* out);
/* Exercises the bounded wait every tensor-memory kernel uses for its hand-overs: a one-thread kernel waits,
 * with a short limit, on a barrier that nothing will ever signal.  Synchronises `stream`.  Returns
 * HEATKV_ERR_DEVICE_TIMEOUT when the wait gave up and set the device status word as designed (the expected
 * outcome; the context is then in the timed-out state described above and should be destroyed), HEATKV_OK if
 * the wait claimed success, HEATKV_ERR_CUDA on any other outcome.  Nothing faults, traps or hangs. */
int heatkv_selftest_wait_expiry(heatkv_ctx* ctx, void* stream);
/* Reads the device-side status word (synchronises `stream`): HEATKV_OK or
 * HEATKV_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel ran out. */
int heatkv_device_status(heatkv_ctx* ctx, void* stream);
const char* heatkv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* HEATKV_H_ */
