/*
 * libcake -- CAKE prefill-time KV-cache eviction for NVIDIA B200 (sm_100a).
 *
 * Cascading and adaptive KV-cache eviction with layer preferences
 * (arXiv 2503.12491).  For every layer the library scores the observation-window
 * queries against all prompt keys, turns the window attention into the layer's
 * preference score and the per-token eviction indicator, re-splits the total
 * cache budget over the layers seen so far, shrinks every seen layer to its
 * budget with a per-head top-k on the stored indicators, and finally gathers
 * the retained K/V rows into a packed variable-length cache.
 *
 * Conventions
 *   - Every function returns an int32_t status: CAKE_OK (0) or a negative
 *     CAKE_ERR_* code.  Nothing throws, exits or prints.
 *   - Unless a parameter says "host", tensor pointers are DEVICE pointers that
 *     the caller owns and keeps alive until the stream has consumed them.  The
 *     context owns only its own state and scratch (allocated in cake_create).
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work;
 *     none synchronises the host with the device except cake_status,
 *     cake_profile_read and cake_destroy, which say so.
 *   - Stream order.  cake_score_layer runs on the caller's stream.  Everything
 *     that follows a layer's scoring (pooling, preference, cake_allocate,
 *     cake_evict) is enqueued on streams the context owns, ordered after that
 *     layer's score kernel by events, so that it runs beside the scoring of the
 *     following layers.  cake_compact, every cake_get_* / cake_set_* call, cake_begin
 *     and cake_status first make the stream they are given wait for that
 *     internal work.  Hence: results are ordered into the caller's stream by
 *     the call that hands them out, not by cake_allocate / cake_evict
 *     themselves, and the stream arguments of those two calls are unused.
 *     Q and K of a layer are read only by cake_score_layer's kernels (caller's
 *     stream); K and V are read again by cake_compact.
 *   - A context serves one batch of requests at a time and is not thread-safe.
 *
 * Shapes: L layers, H_q query heads, H_kv KV heads, G = H_q/H_kv, d = head_dim,
 * request r has N_r prompt tokens, S_w window queries, n_r = N_r - S_w
 * non-window tokens, T = sum_r N_r.
 *
 * Packed varlen layout of K and V of one layer: [H_kv][T][d], request r owns
 * token rows cu_seqlens[r] .. cu_seqlens[r+1]-1 of every head.
 */
#ifndef CAKE_H_
#define CAKE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CAKE_OK               0
#define CAKE_ERR_ARG        (-1)  /* null pointer, bad shape, unsupported size           */
#define CAKE_ERR_BUDGET     (-2)  /* total_budget < n_layers * window                    */
#define CAKE_ERR_CAPACITY   (-3)  /* batch exceeds max_requests / max_total_tokens       */
#define CAKE_ERR_NONFINITE  (-4)  /* a preference is NaN, infinite or negative (device)  */
#define CAKE_ERR_TIMEOUT    (-5)  /* a bounded device-side wait ran out (device)         */
#define CAKE_ERR_CUDA       (-6)  /* a CUDA runtime call failed                          */
#define CAKE_ERR_STATE      (-7)  /* call out of order (layer / stage sequence)          */

#define CAKE_DTYPE_FP32 0
#define CAKE_DTYPE_BF16 1
#define CAKE_POOL_MAX   0
#define CAKE_POOL_AVG   1
/* What the eviction indicator combines (Section 4.3; the alternatives are the
 * rows of the paper's indicator ablation, Table "indicator_abl"). */
#define CAKE_IND_MEAN_PLUS_VAR  0   /* Mean + gamma * Var, Eq. 11 (default) */
#define CAKE_IND_MEAN           1   /* Mean only                            */
#define CAKE_IND_VAR            2   /* Var only                             */
#define CAKE_IND_MEAN_TIMES_VAR 3   /* Mean * Var                           */
#define CAKE_IND_WINDOW_SUM     4   /* sum over the window queries (S_w * Mean): the SnapKV
                                       indicator of the paper's compatibility study,
                                       Section 5.3, here under the preference allocation */
/* How cake_allocate weighs the layers (Section 5.3, allocation ablation). */
#define CAKE_ALLOC_PREFERENCE 0     /* P_l of Eq. 6 (the paper's method, default)          */
#define CAKE_ALLOC_UNIFORM    1     /* every layer the same weight                         */
#define CAKE_ALLOC_PYRAMID    2     /* weights falling linearly with the layer index:
                                       w_l = 1 + s (L-1-2l)/(L-1), s = pyramid_slope        */

/* How cake_decode_step combines a new token's pooled attention with a stored score (the
 * appendix listing calls it "update_score" without defining it). */
#define CAKE_DECODE_ADD      0   /* stored + pooled (default reading)  */
#define CAKE_DECODE_MAX      1   /* max(stored, pooled)                */
#define CAKE_DECODE_REPLACE  2   /* pooled                             */

#define CAKE_MAX_LAYERS 128

typedef struct cake_ctx cake_ctx;

typedef struct cake_config {
  int32_t n_layers;         /* L, 1..CAKE_MAX_LAYERS                                      */
  int32_t n_q_heads;        /* H_q                                                        */
  int32_t n_kv_heads;       /* H_kv, divides H_q                                          */
  int32_t head_dim;         /* d: 64 or 128                                               */
  int32_t window;           /* S_w >= 1; G * S_w <= 128                                   */
  int32_t pool_kernel;      /* odd, >= 1 (1 = no pooling)                                 */
  int32_t pool_mode;        /* CAKE_POOL_MAX (window clipped at the ends) or CAKE_POOL_AVG
                               (zero padding, divisor pool_kernel)                        */
  int32_t var_ddof;         /* 0 = population variance (default), 1 = unbiased            */
  int32_t dtype;            /* CAKE_DTYPE_FP32 or CAKE_DTYPE_BF16: element type of Q/K/V  */
  float   gamma;            /* weight of the variance term in the indicator (Eq. 11)      */
  float   tau1, tau2;       /* temperatures of the preference score (Eq. 6), > 0          */
  int64_t total_budget;     /* B_total per request: tokens per KV head summed over layers,
                               window included; must be >= n_layers * window              */
  int32_t max_requests;     /* capacity: requests per batch                               */
  int64_t max_total_tokens; /* capacity: T = sum of prompt lengths per batch              */
  int32_t indicator_mode;   /* CAKE_IND_*: which combination of the window mean and
                               variance scores a key; gamma is used by mode 0 only        */
  int32_t alloc_mode;       /* CAKE_ALLOC_*: what the budget split is proportional to; the
                               rounding, the cap and the cascade are the same in every mode */
  float   pyramid_slope;    /* s in [0, 1] for CAKE_ALLOC_PYRAMID (0 = uniform; 1 = the last
                               layer gets no selectable budget)                            */
} cake_config;

/* Allocates a context (device state and scratch sized from the capacities) on
 * the current device.  The only entry point that allocates device memory. */
int32_t cake_create(const cake_config* cfg, cake_ctx** out);
/* Synchronises the device and frees everything the context owns. */
int32_t cake_destroy(cake_ctx* ctx);

/* Starts a new batch and resets the cascade (Algorithm 1, line 1).
 * cu_seqlens_host: HOST array [n_req+1], exclusive prefix sums of the prompt
 * lengths, cu[0] = 0; copied before the call returns.  Every N_r >= window.
 * n_req = 0 is a valid empty batch. */
int32_t cake_begin(cake_ctx* ctx, int32_t n_req, const int64_t* cu_seqlens_host, void* stream);

/* Layer `layer` arrives (Algorithm 1, lines 3-6; Section 2 Eq. 2, Section 3
 * Eq. 4-5, Section 4.1 Eq. 6, Section 4.3 Eq. 11).  Layers come in order 0..L-1,
 * each after the previous layer's cake_evict.
 *   q_win [n_req][H_q][S_w][d]  the last S_w queries of every request
 *   k     [H_kv][T][d]          packed varlen keys of this layer
 *   lse   optional [n_req][H_q][S_w] fp32: natural-log sum-exp of each window
 *         row's scaled logits over its visible keys (as a fused attention
 *         forward produces); NULL = computed here.
 * Computes A = softmax(q k^T / sqrt(d)) for the window rows with the causal
 * mask inside the window, keeps the columns of the n_r non-window keys without
 * renormalising, and stores in the context
 *   - the pooled indicator pool1d(Mean_i + gamma Var_i) of the attention
 *     averaged over each KV head's G query heads,
 *   - H_l, V_l (means over query heads of the row-entropy sum and of the
 *     column-variance sum) and P_l = H_l^(1/tau1) V_l^(1/tau2).
 * Non-finite or negative P_l sets the sticky device status CAKE_ERR_NONFINITE. */
int32_t cake_score_layer(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                         const float* lse, void* stream);

/* Budgets of layers 0..stage from the preferences known so far (Section 4.1
 * Eq. 7, Section 4.2 Eq. 9; Algorithm 1 line 7), entirely on the device.
 * Each layer owns S_w window slots; the remaining B' = B_total - L*S_w slots
 * are split in proportion to P_l and integerised by Webster / Sainte-Lague
 * highest averages (priorities P_l/(s+1/2), IEEE double; ties to the lower
 * layer, then the lower s), then capped at n_r.  A request with
 * N_r <= floor(B_total/L) keeps every token.  All-zero preferences count as
 * all-equal. */
int32_t cake_allocate(cake_ctx* ctx, int32_t stage, void* stream);

/* Shrinks every layer 0..stage to its current budget (Algorithm 1, lines 9-13;
 * Section 4.2 EVICT; Section 4.3 Eq. 12): per KV head keeps the entries that
 * come first in the order (indicator descending, token position ascending)
 * among the stored (indicator, position) pairs; survivors keep their stored
 * indicator.  The window tokens are always kept.  Needs cake_allocate(stage)
 * and stages in order.
 * The stored pairs of a layer are kept sorted by the leading bits of the
 * indicator (written once, when the layer arrives); a later, smaller budget
 * only moves the list's threshold, which selects the same set as a TopK on the
 * surviving pairs would. */
int32_t cake_evict(cake_ctx* ctx, int32_t stage, void* stream);

/* Gathers the retained rows of layers [layer_lo, layer_hi) (Eq. 12: K^ = K[D,:],
 * V^ = V[D,:]) into the packed cache.  All of those layers must have been
 * evicted.
 *   k_layers, v_layers  HOST arrays [n_layers] of device pointers, each
 *                       [H_kv][T][d]; entries outside [layer_lo, layer_hi) are ignored.
 *                       A pointer may also be page-locked host memory that the device can
 *                       address (cudaHostAlloc under unified addressing): the gather then reads
 *                       only the retained rows over the bus, so values that the scoring never
 *                       touches need not be copied to the device at all
 *   k_out, v_out        device, capacity >= cake_packed_rows_bound() rows of d elements
 *   row_offsets_out     device int64 [n_req*L + 1]: block (r,l) = index r*L+l occupies
 *                       rows row_offsets[r*L+l] .. row_offsets[r*L+l+1]-1 and is laid
 *                       out [H_kv][len][d], len = its retained length; rows are in
 *                       ascending token position, the window last
 *   positions_out       device int32, one token position per packed row (may be NULL) */
int32_t cake_compact(cake_ctx* ctx, int32_t layer_lo, int32_t layer_hi,
                     const void* const* k_layers, const void* const* v_layers,
                     void* k_out, void* v_out, int64_t* row_offsets_out,
                     int32_t* positions_out, void* stream);

/* cake_compact with 4-bit output: the retained rows written as asymmetric INT4 codes, keys
 * quantised per channel and values per token -- the combination of eviction and KIVI-style
 * quantisation the paper evaluates (Appendix "Comparison and Compatibility with Quantization
 * Methods").  Same packed row order, row offsets and positions as cake_compact.
 *   A group of `group` (32, 64 or 128, at most d) values shares zero = min and
 *   scale = (max - min) / 15 (1 when max = min); code = clamp(rint((x - zero) / scale), 0, 15)
 *   in IEEE fp32; x is recovered as zero + code * scale.
 *   values: groups of `group` consecutive channels of a row.
 *           v_codes uint8 [rows][d/2] (even channel in the low nibble),
 *           v_scale, v_zero fp32 [rows][d/group]
 *   keys:   one group per channel over `group` consecutive packed rows of a (request, layer,
 *           head); the last group of a head may be shorter.
 *           k_codes uint8 [rows][d/2]; k_scale, k_zero fp32 [key groups][d], where block
 *           (r,l) owns the key groups kgroup_offsets[r*L+l] .. kgroup_offsets[r*L+l+1]-1,
 *           laid out [H_kv][ceil(len/group)]
 *   kgroup_offsets_out: device int64 [n_req*L + 1].
 * Capacities: rows <= cake_packed_rows_bound(); key groups <= rows / group + n_req*L*H_kv. */
int32_t cake_compact_int4(cake_ctx* ctx, int32_t layer_lo, int32_t layer_hi,
                          const void* const* k_layers, const void* const* v_layers, int32_t group,
                          uint8_t* k_codes, float* k_scale, float* k_zero,
                          uint8_t* v_codes, float* v_scale, float* v_zero,
                          int64_t* row_offsets_out, int64_t* kgroup_offsets_out,
                          int32_t* positions_out, void* stream);

/* Upper bound on the rows cake_compact writes for the current batch:
 * H_kv * sum_r min(B_total, L*N_r).  Returns the bound or a negative error. */
int64_t cake_packed_rows_bound(const cake_ctx* ctx);

/* ---- getters (results stay on the device) and test hooks ---------------- */

/* Pooled indicators of the most recently scored (or set) layer, valid until
 * the next cake_score_layer: out is device fp32 [H_kv][T]; window positions
 * hold +inf (the paper's "arbitrarily large" value, Section 4.3). */
int32_t cake_get_indicators(cake_ctx* ctx, int32_t layer, float* out, void* stream);
/* H, V, P: device double [n_req][L] each (any may be NULL). */
int32_t cake_get_preferences(cake_ctx* ctx, double* H, double* V, double* P, void* stream);
/* Retained length of every layer including the window: device int32 [n_req][L];
 * layers beyond the last allocated stage read 0. */
int32_t cake_get_budgets(cake_ctx* ctx, int32_t* out, void* stream);
/* Retained positions of one (request, layer): device int32 [H_kv][len], len as
 * cake_get_budgets reports; `capacity` = elements available in out. */
int32_t cake_get_positions(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* out,
                           int64_t capacity, void* stream);
/* Replaces cake_score_layer's indicator output for `layer`: in is device fp32
 * [H_kv][T] (window positions ignored).  Lets a test run the cascade on
 * indicators computed elsewhere. */
int32_t cake_set_indicators(cake_ctx* ctx, int32_t layer, const float* in, void* stream);
/* Sets P for layers 0..n_layers_set-1: device double [n_req][n_layers_set]. */
int32_t cake_set_preferences(cake_ctx* ctx, int32_t n_layers_set, const double* P, void* stream);
/* Synchronises `stream`, then returns the sticky device status word through
 * device_status_out (CAKE_OK or the first CAKE_ERR_* a kernel raised). */
int32_t cake_status(cake_ctx* ctx, int32_t* device_status_out, void* stream);

/* ---- tracing ------------------------------------------------------------ */
#define CAKE_PROF_SCORE       0  /* window scores: softmax denominators and column statistics   */
#define CAKE_PROF_FINALIZE    1  /* preference + pooling                                         */
#define CAKE_PROF_ALLOCATE    2
#define CAKE_PROF_EVICT       3
#define CAKE_PROF_COMPACT     4
#define CAKE_PROF_KINDS       5
/* While enabled, every stage of the path brackets its kernels with CUDA events
 * on the stream the stage runs on: the caller's stream for the score kernel and
 * the compaction, the context's own streams for pooling/preference, budgets and
 * eviction (this perturbs back-to-back launches slightly). */
int32_t cake_profile_enable(cake_ctx* ctx, int32_t on);
/* Synchronises `stream`; returns, per CAKE_PROF_* kind, the milliseconds and
 * the number of bracketed spans accumulated since the last read (HOST arrays
 * of CAKE_PROF_KINDS entries), then clears them. */
int32_t cake_profile_read(cake_ctx* ctx, double* ms_out, int64_t* spans_out, void* stream);

/* 1 if cake_score_layer runs the tcgen05 tensor-core kernels for this context
 * (bf16, G*S_w a multiple of 32 up to 128, G in {1,2,4,8}), 0 if it runs the fp32
 * SIMT kernels, negative on error. */
int32_t cake_uses_tensor_cores(const cake_ctx* ctx);

/* ---- decode-time eviction ------------------------------------------------------------
 * Section 5.1 ("tokens are evicted during both prefilling and decoding"), Appendix "More
 * Implementation Details" (every layer's budget is frozen at the prefill's final allocation)
 * and the decode branches of the appendix listing.  After the last cake_evict of a batch:
 *
 *   cake_decode_begin   builds the decode cache: block (r,l) = rows row_offsets[r*L+l] ..
 *                       row_offsets[r*L+l+1]-1 of k_cache / v_cache, laid out [H_kv][cap][d] with
 *                       cap = len + 1 slots per head (len = the layer's retained length, window
 *                       included); slots 0..len-1 receive the retained rows in ascending token
 *                       position, slot len is free.  The stored indicators of the survivors
 *                       become their decode scores.  k_cache and v_cache: device, caller-owned,
 *                       at least cake_decode_rows_bound() rows of d elements; row_offsets_out:
 *                       device int64 [n_req*L+1] (may be NULL).  This call synchronises
 *                       `stream` once (it reads the final budgets back to size its kernels).
 *   cake_decode_step    one generated token, one layer: q_new [n_req][H_q][d], k_new and v_new
 *                       [n_req][H_kv][d].  Per KV head the new K/V row goes into the free slot;
 *                       the new query's attention over the head's cap cached keys (softmax over
 *                       all of them, the S_w most recent columns dropped, mean over the group's
 *                       query heads) is pooled along ascending token position with the
 *                       context's pooling mode and kernel; the pooled value is added to the
 *                       stored score of every token outside the recent window (a token that has
 *                       just left the window starts from its pooled value; CAKE_DECODE_* selects
 *                       other readings); then the entry that comes last in the order (score
 *                       descending, position ascending) among those tokens is evicted and its
 *                       slot becomes the free one, so the head is back at its frozen budget.
 *                       Rows never move; layers may be stepped in any order, each once per token.
 *   cake_decode_get_state  entries of one (request, layer) in ascending token position:
 *                       positions_out int32 [H_kv][len], scores_out fp32 [H_kv][len] (0 for the
 *                       window entries), slots_out int32 [H_kv][len] (slot of each entry inside
 *                       its head's cap slots); any may be NULL.
 * A head with more than 200 KB / (4 * (G + 1)) slots (10239 at G = 4) does not fit the step
 * kernel's shared memory and works in a global-memory area of the context instead (same
 * results, a slower step for that head). */
int64_t cake_decode_rows_bound(const cake_ctx* ctx);
int32_t cake_decode_begin(cake_ctx* ctx, const void* const* k_layers, const void* const* v_layers,
                          void* k_cache, void* v_cache, int64_t* row_offsets_out, int32_t update_mode,
                          void* stream);
int32_t cake_decode_step(cake_ctx* ctx, int32_t layer, const void* q_new, const void* k_new,
                         const void* v_new, void* k_cache, void* v_cache, void* stream);
int32_t cake_decode_get_state(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* positions_out,
                              float* scores_out, int32_t* slots_out, void* stream);

/* Bound, in SM clock cycles, of every wait inside the kernels (a CTA waiting for another CTA's
 * partial results, or for one of its own barriers).  A wait that runs out sets the sticky device
 * status CAKE_ERR_TIMEOUT; the kernel then drains and returns, and the context stays usable (the
 * results of that batch are not).  0 restores the default of 4e9 cycles (about two seconds).
 *
 * The score kernel's CTAs wait for one another, so all of them must be resident at once: it is
 * launched with at most one CTA per SM of the device.  Score launches of two contexts must
 * therefore not overlap on one device (two streams, or two host threads): each would hold SMs
 * the other waits for, and both would end with CAKE_ERR_TIMEOUT after the wait limit instead of
 * a result.  Serialise them with stream order or events. */
int32_t cake_set_wait_limit(cake_ctx* ctx, int64_t cycles);
/* Test hook for the bounded waits: adds `delta` to the launch count that the cross-CTA waits of
 * the following cake_score_layer calls expect, until the next cake_begin.  With delta != 0 no
 * count ever matches, so every such wait runs out after the wait limit (set a short one first)
 * and the launch ends with the device status CAKE_ERR_TIMEOUT. */
int32_t cake_debug_skew_sync(cake_ctx* ctx, int32_t delta);

/* Launch plan of cake_score_layer for the current batch, for tests and diagnostics (the plan is
 * built on the host in cake_begin; nothing here touches the device).  out8 is a HOST array of 8
 * int32: [0] 1 if the tensor-core kernels are used, [1] CTAs of the score kernel, [2] waves (groups
 * of (request, KV head) pairs whose keys pass A and pass B share through L2), [3] rows the merger
 * warps combine side by side (a power of two, 1 to 32), [4] pass-A segments, [5] pass-B segments, [6] ops in the
 * CTAs' programs, [7] SMs left to the cascade kernels.  Entries [1]..[6] are 0 on the SIMT path. */
int32_t cake_plan_info(const cake_ctx* ctx, int32_t* out8);

/* Builds the score kernel's launch plan for a batch on the HOST alone (no device, no context: it
 * runs without a GPU) and checks what the kernel relies on: every key tile covered exactly once
 * per pass, every CTA's program ordered so that a wave's column pass can only wait for row-pass
 * ops that wait for nothing, merge groups within two adjacent waves, table sizes.  n_sm = SMs of
 * the device to plan for, reserved_sms as CAKE_RESERVED_SMS.  info8 (HOST, 8 int32): CTAs,
 * waves, merge ways, pass-A segments, pass-B segments, ops of the two-pass programs, ops of the
 * column-pass-only programs, and the number of the violated property (0 = none).  Returns
 * CAKE_OK, CAKE_ERR_ARG (also when the shape takes the SIMT path), an error of the plan builder,
 * or CAKE_ERR_STATE when a property is violated. */
int32_t cake_plan_check(const cake_config* cfg, int32_t n_sm, int32_t reserved_sms, int32_t n_req,
                        const int64_t* cu_seqlens_host, int32_t* info8);

/* ---- selection without any allocation ------------------------------------- */
/* The paper has no counterpart for this entry point; it exists for callers that are not
 * allowed to allocate device memory when they call in: code running inside another
 * framework's memory pool or a fixed memory plan, a real-time or serving loop where
 * cudaMalloc / cudaFree would stall the device, or a process whose allocator is already
 * exhausted on purpose.  Such callers cannot use a context (cake_create allocates).
 *
 * Per head, keeps the `keep` entries of values[head][0..n) that come first in the order
 * (value descending, position ascending) -- the TopK of Eq. 12 with the same tie rule as
 * cake_evict -- and writes their positions in ascending order.
 *   values        device fp32 [n_heads][n]
 *   positions_out device int32 [n_heads][keep]
 * It calls no cudaMalloc, cudaFree or other allocating routine.  Its working memory (two
 * bitmaps per head) is a fixed 256 KB array inside the library, present on every GPU that
 * loads the library until the process exits, which bounds the problem size:
 *   n_heads * ceil(n / 32) <= 32768      (about one million values per call);
 * anything larger returns CAKE_ERR_CAPACITY and does nothing.  0 <= keep <= n, else
 * CAKE_ERR_ARG.  All calls share that array and the array keeps the previous call's
 * contents; the kernel clears what it needs first, but two calls that overlap on the GPU
 * (different streams, or different host threads without ordering) race on it: serialise them.
 * The first call on each device looks up the array's device address (once per device, with
 * that device current); make that first call outside any stream capture. */
int32_t cake_select_positions_static(const float* values, int32_t n_heads, int32_t n, int32_t keep,
                                     int32_t* positions_out, void* stream);

const char* cake_strerror(int32_t code);
/* Number of kernels this library has launched in the calling process. */
int64_t cake_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CAKE_H_ */
