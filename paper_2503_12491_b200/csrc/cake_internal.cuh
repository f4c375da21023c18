// Internal declarations shared by the translation units of libcake.
#pragma once

#include <cuda_runtime.h>
#include <cstdio>
#include <cstdlib>
#include <cuda_bf16.h>
#include <stdint.h>

#include "cake.h"

namespace cake {

constexpr int kMaxRows = 128;        // G * S_w rows handled per KV head
constexpr int kSimtTileKeys = 64;    // keys per tile of the SIMT score kernels
constexpr int kSimtThreads = 256;
constexpr int kBinBits = 12;         // survivor lists are sorted by the top bits of the indicator
constexpr int kBins = 1 << kBinBits;
constexpr int kChunkKeys = 4096;     // granularity of the token ranges of the pooling / scatter CTAs
constexpr int kBitmapSmemWords = 48 * 1024;   // positions of up to 1.5 M tokens are ordered in shared memory
constexpr int kScoreGroups = 3;      // statistics warp groups per CTA of the tensor-core score kernel
constexpr int kScoreWarps = 4 * kScoreGroups;   // statistics warps: one column-pass partial each

// One request of the current batch (device copy in ctx->d_req).
struct ReqInfo {
  int64_t cu;        // first token row of the request inside the packed K/V
  int32_t N;         // prompt length
  int32_t n;         // N - S_w non-window tokens
  int32_t keep_all;  // 1: N <= floor(B_total/L), nothing is evicted
  int32_t nsplit;    // CTAs of the pooling / scatter kernels that share the prompt's tokens
  int32_t span;      // tokens per such CTA (a multiple of kChunkKeys)
  int64_t list_off;  // first entry of this request's lists; list (layer, head) holds n entries
  int32_t unit0;     // first score unit of the request
  int32_t nunits;    // number of score units of the request
};

// A run of consecutive keys of one request handled by one CTA of a score kernel.
struct ScoreUnit {
  int32_t req;
  int32_t key0;
  int32_t nkeys;
  int32_t pad;
};

// One step of a CTA's program in the tensor-core score kernel: a run of consecutive
// keys of one (request, KV head) in pass A (phase 0, row statistics) or pass B (phase 1,
// column statistics).  `seg` numbers the partial results the step writes (one per
// statistics warp group).
struct ScoreOp {
  int64_t base;    // row of the pair's first key in the packed K: g * T + cu[req]
  int32_t req;
  int32_t g;
  int32_t key0;
  int32_t nkeys;
  int32_t phase;
  int32_t seg;
  int32_t n;       // non-window keys of the request
  int32_t pad;
};

// Retained set of one (request, layer, head) list, whose entries (ordered key, position) are
// stored by bucket.
struct ListState {
  int32_t bucket;        // threshold bucket d; all buckets before it are kept; -1: nothing kept
  uint32_t thr_key;      // inside bucket d an entry is kept if key > thr_key,
  int32_t pos_cut;       //   or key == thr_key and position <= pos_cut
  int32_t kept;          // number of retained non-window tokens
};

struct LayerPtrs {
  const void* k[CAKE_MAX_LAYERS];
  const void* v[CAKE_MAX_LAYERS];
};

}  // namespace cake

namespace cake {
struct ProfSpan { int kind; cudaEvent_t a, b; };
struct Profiler {
  bool on;
  int used, cap;
  ProfSpan* spans;
};
}  // namespace cake

struct cake_ctx {
  cake_config cfg;
  cake::Profiler prof;
  int device;
  int n_sm;
  int n_sm_score;          // SMs the persistent score kernel occupies; the rest stay free for the
                           // cascade kernels of the previous layer, which run beside it
  // The cascade of layer l (pooling, preference, budgets, eviction) runs on an internal side
  // stream while the caller's stream already scores layer l+1; events order the two.
  cudaStream_t side;
  cudaStream_t side2;               // older layers' thresholds of a stage, beside the newest layer's scatter
  cudaStream_t pool_st;             // pooling + preference of layer l+1, beside the budgets and eviction of layer l
  cudaStream_t alloc_st;            // budgets of stage m, beside the eviction of stage m-1
  cudaEvent_t ev_alloc[2];          // budgets of a stage of that parity are written
  cudaEvent_t ev_alloc_main;        // scratch event: budget stream -> caller's
  cudaEvent_t ev_main, ev_side;     // scratch events: caller's stream -> side, side -> caller's
  cudaEvent_t ev_fork, ev_join;     // side -> side2 and back
  cudaEvent_t ev_pool_side;         // scratch event: pooling stream -> caller's
  cudaEvent_t ev_evict[2];          // eviction stage of that parity has finished (it reads d_fresh of that parity)
  bool evict_recorded[2];
  cudaEvent_t ev_score[2];          // score kernel of a layer of that parity has finished
  cudaEvent_t ev_pool[2];           // pooling (the last reader of the score outputs) of that parity has finished
  bool pool_recorded[2];
  int32_t rows;            // R = G * S_w
  int64_t sel_budget;      // B' = B_total - L * S_w
  // ---- batch state (host) ----
  int32_t n_req;
  int64_t total_tokens;    // T
  int32_t n_units;         // score units for all N keys (phase A)
  int32_t n_ind;           // layers whose indicators have arrived
  int32_t n_pref;          // layers whose preference is known
  int32_t n_evicted;       // stages completed
  int32_t alloc_of_buf[2]; // stage whose budgets live in budget buffer 0/1 (-1 none)
  int32_t last_alloc;      // most recent stage passed to cake_allocate
  int64_t packed_rows_bound;
  int64_t* h_cu;           // host copy of cu_seqlens [max_requests+1]
  // ---- pinned staging ----
  cake::ReqInfo* h_req;    // [max_requests]
  cake::ScoreUnit* h_units;
  cudaEvent_t upload_done;
  bool upload_pending;
  // ---- device state ----
  cake::ReqInfo* d_req;
  cake::ScoreUnit* d_units;
  int32_t max_units;
  double* d_H;             // [max_requests][L]
  double* d_V;
  double* d_P;
  int32_t* d_budget[2];    // [max_requests][L] selectable budgets, double-buffered by stage parity
  int32_t* d_status;       // sticky device status word
  float* d_raw[2];         // [H_kv][max_total_tokens] un-pooled indicator, by layer parity
  float* d_fresh[2];       // [H_kv][max_total_tokens] pooled indicator of the newest layer, by layer parity
  uint2* d_lists;          // per (req, layer, head): n entries (ordered indicator key, position)
  int64_t list_elems;
  int32_t* d_prefix;       // [max_lists][kBins+1] bucket offsets of every list
  cake::ListState* d_lstate;   // [max_lists]
  int64_t max_lists;
  uint32_t* d_hist;        // [max_pairs][kBins] bucket histogram of the arriving layer (zero at rest)
  uint32_t* d_fill;        // [max_pairs][kBins] scatter cursors (zero at rest)
  uint32_t* d_arrivals;    // zero at rest: [max_pairs] split counters of the scatter, [max_requests] head
                           // counters of the preference, [max_pairs] split counters of the pooling (the
                           // pooling of layer l+1 runs beside the scatter of layer l: separate counters)
  double* d_headsum;       // [max_requests][H_q][2] per-head entropy / variance sums of the layer
  int32_t n_split;         // largest nsplit of the batch
  int32_t* d_pos_packed;   // [packed rows bound] positions in packed row order
  int64_t pos_packed_cap;
  uint32_t* d_bitmap;      // global bitmaps for requests too long for shared memory (or null)
  int64_t bitmap_words;
  float* d_lse2;           // [max_requests][H_q][S_w] base-2 log-sum-exp of window rows
  float2* d_rowpart;       // [max_units][H_kv][R] (max, sum) partials of phase A
  float* d_colpart[2];     // partial (sum p*log2 p, sum var) of the column pass, by layer parity
  // ---- tensor-core score path ----
  bool use_tc;
  bool hhead_from_rows;    // entropy came from pass A (d_hrow) rather than from pass B partials
  int32_t n_tc_ctas, max_tc_segs, max_pairs;
  int32_t n_tc_waves;             // waves of the current plan
  // ---- decode-time eviction (frozen budgets) ----
  bool dec_ready;                 // cake_decode_begin has built the decode state of this batch
  int32_t dec_update_mode;        // CAKE_DECODE_*
  int64_t dec_max_cap;            // slots of the largest head of the batch (len + 1)
  int64_t dec_rows_cap;           // capacity of the three arrays below
  int64_t* d_dec_off;             // [max_requests*L + 1] decode row offsets
  int64_t* d_dec_packed_off;      // [max_requests*L + 1] packed row offsets (set-up scratch)
  float* d_dec_score;             // stored eviction score of every slot
  float* d_dec_tmp;               // [H_kv][tokens + requests][G + 1]: work area of decode heads too large for shared memory
  int32_t* d_dec_pos;             // token position of every slot (-1: free)
  int32_t* d_dec_order;           // per head: rank in ascending position -> slot
  int4* d_dec_meta;               // [max_lists] (len, free slot, next position, frozen budget)
  int32_t* h_budget_stage;        // pinned [max_requests*L] read-back of the final budgets
  int64_t wait_limit_cycles;      // bound of every device-side wait (0 = the default, about 2 s)
  int32_t debug_epoch_skew;       // test hook: added to the launch count the cross-CTA waits expect
  int32_t n_tc_asegs, n_tc_bsegs;          // pass-A / pass-B segments per layer
  int32_t n_tc_ops_full, n_tc_ops_b, max_tc_ops;
  uint32_t tc_epoch;              // both-pass launches since cake_begin
  cake::ScoreOp* h_tc_ops;        // pinned: [both-pass programs][pass-B-only programs]
  cake::ScoreOp* d_tc_ops;
  // pinned / device index block of the current batch, P = n_req * H_kv pairs:
  //   pair_aseg [P+1] | pair_bseg [P+1] | cta_op of the both-pass programs [n_sm+1]
  //   | cta_op of the pass-B-only programs [n_sm+1]
  int32_t* h_tc_index;
  int32_t* d_tc_index;
  uint32_t* d_tc_sync;            // [max_pairs] delivered partial rows, then [max_pairs] merged rows
  int tc_merge_ways;              // rows the merger warp handles side by side (a power of two up to 32), chosen with the plan
  float4* d_tc_rowpart;           // [max_tc_segs][kScoreGroups][128]
  float* d_lse2_tc;               // [max_requests][H_kv][128], rows in tile order i*G + h
  float* d_hrow[2];               // [max_pairs][128] sum_j p log2 p per window row, by layer parity
};

namespace cake {

void count_launch(int64_t n = 1);

// score_simt.cu
int32_t launch_score_simt(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                          const float* lse, cudaStream_t st);
// score_tc.cu
bool tc_path_supported(const cake_config& c);
int64_t tc_max_segments(const cake_config& c, int n_sm);
int32_t tc_build_plan(cake_ctx* ctx, int32_t n_req);
int32_t tc_plan_check(const cake_config& c, int n_sm, int reserved, int32_t n_req, const int64_t* cu,
                      int32_t* info8);
int32_t launch_score_tc(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                        const float* lse, cudaStream_t st);
// cascade.cu
int32_t launch_pool(cake_ctx* ctx, int32_t layer, bool do_pool, bool finalize, cudaStream_t st);
int32_t launch_allocate(cake_ctx* ctx, int32_t stage, cudaStream_t st);
int32_t launch_evict(cake_ctx* ctx, int32_t stage, cudaStream_t st);
// decode.cu
int32_t launch_decode_begin(cake_ctx* ctx, const LayerPtrs& ptrs, void* k_cache, void* v_cache,
                            int64_t* row_offsets, cudaStream_t st);
int32_t launch_decode_step(cake_ctx* ctx, int32_t layer, const void* q_new, const void* k_new,
                           const void* v_new, void* k_cache, void* v_cache, cudaStream_t st);
int32_t launch_decode_read(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* positions, float* scores,
                           int32_t* slots, cudaStream_t st);
// quant.cu
int32_t launch_compact_int4(cake_ctx* ctx, int32_t lo, int32_t hi, const LayerPtrs& ptrs, int32_t group,
                            uint8_t* k_codes, float* k_scale, float* k_zero, uint8_t* v_codes,
                            float* v_scale, float* v_zero, int64_t* row_offsets, int64_t* kgroup_offsets,
                            int32_t* positions, cudaStream_t st);
// compact.cu
int32_t launch_compact(cake_ctx* ctx, int32_t lo, int32_t hi, const LayerPtrs& ptrs, void* k_out,
                       void* v_out, int64_t* row_offsets, int32_t* positions, cudaStream_t st);
int32_t launch_get_positions(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* out,
                             int64_t capacity, cudaStream_t st);

// The eviction indicator of one key from the mean and variance of its window attention
// (Section 4.3, Eq. 11, and the combinations of the paper's indicator ablation).
__device__ __forceinline__ float combine_indicator(int mode, float gamma, float mean, float var,
                                                   float sw) {
  return mode == CAKE_IND_MEAN_PLUS_VAR ? fmaf(gamma, var, mean)
         : mode == CAKE_IND_MEAN        ? mean
         : mode == CAKE_IND_VAR         ? var
         : mode == CAKE_IND_WINDOW_SUM  ? mean * sw
                                        : mean * var;
}

// Function attributes (the dynamic shared-memory limit) belong to a device: a flag per device,
// so that a context on a second GPU sets them there too.
constexpr int kOnceDevices = 64;
struct PerDeviceOnce {
  bool done[kOnceDevices] = {};
  bool need(int device) const { return device < 0 || device >= kOnceDevices || !done[device]; }
  void mark(int device) { if (device >= 0 && device < kOnceDevices) done[device] = true; }
};

// Tracing spans (no-ops unless cake_profile_enable was called).
int prof_begin(cake_ctx* ctx, int kind, cudaStream_t st);
void prof_end(cake_ctx* ctx, int span, cudaStream_t st);

// Maps a CUDA runtime result to a library status; with CAKE_VERBOSE set in the environment the
// runtime's own message goes to stderr, since the status code alone does not say which error it was.
inline int32_t cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return CAKE_OK;
  if (getenv("CAKE_VERBOSE")) fprintf(stderr, "libcake: CUDA error %d: %s\n", (int)e, cudaGetErrorString(e));
  return CAKE_ERR_CUDA;
}

#define CAKE_CUDA_TRY(expr)                         \
  do {                                              \
    cudaError_t _e = (expr);                        \
    if (_e != cudaSuccess) return cuda_status(_e);  \
  } while (0)

}  // namespace cake
