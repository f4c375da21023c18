// C-ABI of libcake: context life cycle, the call-order state machine, getters
// and test hooks.  Every step of the path runs in the kernels of the other
// translation units; this file only validates arguments and enqueues work.
#include "cake_internal.cuh"

#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

namespace cake {

static std::atomic<int64_t> g_launches{0};
void count_launch(int64_t n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int prof_begin(cake_ctx* ctx, int kind, cudaStream_t st) {
  Profiler& p = ctx->prof;
  if (!p.on || p.used >= p.cap) return -1;
  ProfSpan& s = p.spans[p.used];
  if (!s.a) {
    if (cudaEventCreate(&s.a) != cudaSuccess || cudaEventCreate(&s.b) != cudaSuccess) return -1;
  }
  s.kind = kind;
  cudaEventRecord(s.a, st);
  return p.used++;
}

void prof_end(cake_ctx* ctx, int span, cudaStream_t st) {
  if (span >= 0) cudaEventRecord(ctx->prof.spans[span].b, st);
}

namespace {

template <typename T>
cudaError_t dev_alloc(T** p, size_t count) {
  *p = nullptr;
  if (count == 0) count = 1;
  return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
}

int32_t choose_unit_keys(int64_t total_tokens, int n_kv_heads, int n_sm) {
  // Aim for about four CTAs per SM across the (unit, KV head) grid, units of 64..1024 keys.
  int64_t per = total_tokens * n_kv_heads / ((int64_t)4 * n_sm);
  per = per / kSimtTileKeys * kSimtTileKeys;
  if (per < kSimtTileKeys) per = kSimtTileKeys;
  if (per > 1024) per = 1024;
  return (int32_t)per;
}

__global__ void budgets_with_window(const int32_t* __restrict__ b, int32_t* __restrict__ out,
                                    int n_req, int L, int n_alloc, int Sw) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_req * L) return;
  const int l = i % L;
  out[i] = l < n_alloc ? b[i] + Sw : 0;
}

void free_ctx(cake_ctx* c) {
  if (!c) return;
  cudaFree(c->d_req); cudaFree(c->d_units); cudaFree(c->d_H); cudaFree(c->d_V); cudaFree(c->d_P);
  cudaFree(c->d_budget[0]); cudaFree(c->d_budget[1]); cudaFree(c->d_status);
  cudaFree(c->d_raw[0]); cudaFree(c->d_raw[1]);
  cudaFree(c->d_fresh[0]); cudaFree(c->d_fresh[1]); cudaFree(c->d_lists); cudaFree(c->d_prefix); cudaFree(c->d_lstate);
  cudaFree(c->d_hist); cudaFree(c->d_fill); cudaFree(c->d_arrivals); cudaFree(c->d_headsum);
  cudaFree(c->d_pos_packed); cudaFree(c->d_bitmap); cudaFree(c->d_lse2);
  cudaFree(c->d_rowpart); cudaFree(c->d_colpart[0]); cudaFree(c->d_colpart[1]);
  cudaFree(c->d_tc_ops); cudaFree(c->d_tc_index); cudaFree(c->d_tc_sync);
  cudaFree(c->d_tc_rowpart); cudaFree(c->d_lse2_tc); cudaFree(c->d_hrow[0]); cudaFree(c->d_hrow[1]);
  cudaFree(c->d_dec_off); cudaFree(c->d_dec_packed_off); cudaFree(c->d_dec_score); cudaFree(c->d_dec_tmp); cudaFree(c->d_dec_pos);
  cudaFree(c->d_dec_order); cudaFree(c->d_dec_meta);
  if (c->h_budget_stage) cudaFreeHost(c->h_budget_stage);
  if (c->h_tc_ops) cudaFreeHost(c->h_tc_ops);
  if (c->h_tc_index) cudaFreeHost(c->h_tc_index);
  if (c->h_req) cudaFreeHost(c->h_req);
  if (c->h_units) cudaFreeHost(c->h_units);
  if (c->upload_done) cudaEventDestroy(c->upload_done);
  if (c->ev_main) cudaEventDestroy(c->ev_main);
  if (c->ev_side) cudaEventDestroy(c->ev_side);
  for (int i = 0; i < 2; ++i) {
    if (c->ev_score[i]) cudaEventDestroy(c->ev_score[i]);
    if (c->ev_pool[i]) cudaEventDestroy(c->ev_pool[i]);
  }
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->ev_pool_side) cudaEventDestroy(c->ev_pool_side);
  for (int i = 0; i < 2; ++i) if (c->ev_evict[i]) cudaEventDestroy(c->ev_evict[i]);
  for (int i = 0; i < 2; ++i) if (c->ev_alloc[i]) cudaEventDestroy(c->ev_alloc[i]);
  if (c->ev_alloc_main) cudaEventDestroy(c->ev_alloc_main);
  if (c->alloc_st) cudaStreamDestroy(c->alloc_st);
  if (c->pool_st) cudaStreamDestroy(c->pool_st);
  if (c->side2) cudaStreamDestroy(c->side2);
  if (c->side) cudaStreamDestroy(c->side);
  if (c->prof.spans) {
    for (int i = 0; i < c->prof.cap; ++i) {
      if (c->prof.spans[i].a) cudaEventDestroy(c->prof.spans[i].a);
      if (c->prof.spans[i].b) cudaEventDestroy(c->prof.spans[i].b);
    }
    free(c->prof.spans);
  }
  free(c->h_cu);
  delete c;
}

// Orders the internal streams after everything enqueued so far on the caller's stream.
cudaError_t side_after(cake_ctx* c, cudaStream_t st) {
  cudaError_t e = cudaEventRecord(c->ev_main, st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(c->side, c->ev_main, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(c->pool_st, c->ev_main, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(c->alloc_st, c->ev_main, 0);
  return e;
}
// Orders the caller's stream after everything enqueued so far on the internal streams.
cudaError_t main_after_side(cake_ctx* c, cudaStream_t st) {
  cudaError_t e = cudaEventRecord(c->ev_side, c->side);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_side, 0);
  if (e == cudaSuccess) e = cudaEventRecord(c->ev_pool_side, c->pool_st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_pool_side, 0);
  if (e == cudaSuccess) e = cudaEventRecord(c->ev_alloc_main, c->alloc_st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_alloc_main, 0);
  return e;
}

}  // namespace
}  // namespace cake

using namespace cake;

extern "C" {

int32_t cake_create(const cake_config* cfg, cake_ctx** out) {
  if (!cfg || !out) return CAKE_ERR_ARG;
  *out = nullptr;
  const cake_config& c = *cfg;
  if (c.n_layers < 1 || c.n_layers > CAKE_MAX_LAYERS) return CAKE_ERR_ARG;
  if (c.n_kv_heads < 1 || c.n_q_heads < c.n_kv_heads || c.n_q_heads % c.n_kv_heads) return CAKE_ERR_ARG;
  if (c.head_dim != 64 && c.head_dim != 128) return CAKE_ERR_ARG;
  const int G = c.n_q_heads / c.n_kv_heads;
  if (c.window < 1 || G > 8 || (int64_t)G * c.window > kMaxRows) return CAKE_ERR_ARG;
  if (c.pool_kernel < 1 || c.pool_kernel % 2 == 0) return CAKE_ERR_ARG;
  if (c.pool_mode != CAKE_POOL_MAX && c.pool_mode != CAKE_POOL_AVG) return CAKE_ERR_ARG;
  if (c.var_ddof != 0 && !(c.var_ddof == 1 && c.window >= 2)) return CAKE_ERR_ARG;
  if (c.dtype != CAKE_DTYPE_FP32 && c.dtype != CAKE_DTYPE_BF16) return CAKE_ERR_ARG;
  if (!(c.tau1 > 0.f) || !(c.tau2 > 0.f) || !std::isfinite(c.gamma)) return CAKE_ERR_ARG;
  if (c.indicator_mode < CAKE_IND_MEAN_PLUS_VAR || c.indicator_mode > CAKE_IND_WINDOW_SUM) return CAKE_ERR_ARG;
  if (c.alloc_mode < CAKE_ALLOC_PREFERENCE || c.alloc_mode > CAKE_ALLOC_PYRAMID) return CAKE_ERR_ARG;
  if (c.alloc_mode == CAKE_ALLOC_PYRAMID && !(c.pyramid_slope >= 0.f && c.pyramid_slope <= 1.f)) return CAKE_ERR_ARG;
  if (c.max_requests < 1 || c.max_total_tokens < 1) return CAKE_ERR_ARG;
  if (c.max_total_tokens > ((int64_t)1 << 31) - 1024) return CAKE_ERR_ARG;
  if (c.total_budget < (int64_t)c.n_layers * c.window) return CAKE_ERR_BUDGET;
  if (c.total_budget > ((int64_t)1 << 31) - 1024) return CAKE_ERR_ARG;

  cake_ctx* x = new (std::nothrow) cake_ctx();
  if (!x) return CAKE_ERR_CUDA;
  memset(x, 0, sizeof(*x));
  x->cfg = c;
  x->rows = G * c.window;
  x->sel_budget = c.total_budget - (int64_t)c.n_layers * c.window;
  x->alloc_of_buf[0] = x->alloc_of_buf[1] = -1;
  x->last_alloc = -1;
  cudaError_t e = cudaGetDevice(&x->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&x->n_sm, cudaDevAttrMultiProcessorCount, x->device);
  if (e != cudaSuccess) { free_ctx(x); return CAKE_ERR_CUDA; }
  {
    // SMs left to the cascade kernels while a score kernel runs (CAKE_RESERVED_SMS, default 16).
    // The cascade kernels' CTAs are too large to share an SM with a score CTA, so they run on
    // exactly these SMs and cannot slow a score CTA down: the score kernel's CTAs advance wave
    // by wave together, and one delayed CTA delays all of them.
    int reserve = 16;
    if (const char* env = getenv("CAKE_RESERVED_SMS")) reserve = atoi(env);
    if (reserve < 0) reserve = 0;
    if (reserve > x->n_sm / 2) reserve = x->n_sm / 2;
    x->n_sm_score = x->n_sm - reserve;
  }

  const int64_t T = c.max_total_tokens;
  const int64_t R = c.max_requests;
  // a unit never spans requests: at most T/64 + R units
  x->max_units = (int32_t)(T / kSimtTileKeys + R + 1);
  x->list_elems = T * c.n_layers * c.n_kv_heads;
  x->max_lists = R * c.n_layers * c.n_kv_heads;
  {
    // packed rows: H_kv * sum_r min(B_total, L * N_r) <= H_kv * min(R * B_total, L * T)
    const int64_t a = R * c.total_budget, b = (int64_t)c.n_layers * T;
    x->pos_packed_cap = (int64_t)c.n_kv_heads * (a < b ? a : b);
    // a request longer than the shared-memory bitmap orders its positions in global scratch:
    // one bitmap of ceil(n/32) words per (request, layer, head) list
    x->bitmap_words = T > (int64_t)kBitmapSmemWords * 32
                          ? (int64_t)c.n_layers * c.n_kv_heads * (T / 32 + R + 1) : 0;
  }
  x->h_cu = (int64_t*)calloc((size_t)R + 1, sizeof(int64_t));
  bool ok = x->h_cu != nullptr;
  ok = ok && cudaMallocHost((void**)&x->h_req, sizeof(ReqInfo) * R) == cudaSuccess;
  ok = ok && cudaMallocHost((void**)&x->h_units, sizeof(ScoreUnit) * x->max_units) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->upload_done, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&x->side, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&x->side2, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&x->pool_st, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_pool_side, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&x->alloc_st, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_alloc_main, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 2; ++i)
    ok = ok && cudaEventCreateWithFlags(&x->ev_alloc[i], cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 2; ++i)
    ok = ok && cudaEventCreateWithFlags(&x->ev_evict[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_fork, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_join, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_main, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&x->ev_side, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 2; ++i) {
    ok = ok && cudaEventCreateWithFlags(&x->ev_score[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&x->ev_pool[i], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && dev_alloc(&x->d_req, R) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_units, x->max_units) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_H, R * c.n_layers) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_V, R * c.n_layers) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_P, R * c.n_layers) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_budget[0], R * c.n_layers) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_budget[1], R * c.n_layers) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_status, 1) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_raw[0], (size_t)c.n_kv_heads * T) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_raw[1], (size_t)c.n_kv_heads * T) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_fresh[0], (size_t)c.n_kv_heads * T) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_fresh[1], (size_t)c.n_kv_heads * T) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_lists, (size_t)x->list_elems) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_prefix, (size_t)x->max_lists * (kBins + 1)) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_lstate, (size_t)x->max_lists) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_hist, (size_t)R * c.n_kv_heads * kBins) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_fill, (size_t)R * c.n_kv_heads * kBins) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_arrivals, 2 * (size_t)R * c.n_kv_heads + R) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_headsum, (size_t)R * c.n_q_heads * 2) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_pos_packed, (size_t)x->pos_packed_cap) == cudaSuccess;
  if (x->bitmap_words > 0) ok = ok && dev_alloc(&x->d_bitmap, (size_t)x->bitmap_words) == cudaSuccess;
  ok = ok && cudaMemset(x->d_hist, 0, sizeof(uint32_t) * R * c.n_kv_heads * kBins) == cudaSuccess;
  ok = ok && cudaMemset(x->d_fill, 0, sizeof(uint32_t) * R * c.n_kv_heads * kBins) == cudaSuccess;
  ok = ok && cudaMemset(x->d_arrivals, 0, sizeof(uint32_t) * (2 * R * c.n_kv_heads + R)) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_lse2, (size_t)R * c.n_q_heads * c.window) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_rowpart, (size_t)x->max_units * c.n_kv_heads * x->rows) == cudaSuccess;
  {
    const char* force = getenv("CAKE_SCORE_PATH");       // "simt" forces the SIMT kernels
    x->use_tc = tc_path_supported(c) && !(force && strcmp(force, "simt") == 0);
  }
  const int64_t max_pairs = R * c.n_kv_heads;
  x->max_pairs = (int32_t)max_pairs;
  {
    const int64_t segs = tc_max_segments(c, x->n_sm);
    if (x->use_tc && segs > ((int64_t)1 << 24)) { free_ctx(x); return CAKE_ERR_ARG; }
    x->max_tc_segs = (int32_t)segs;
    x->max_tc_ops = (int32_t)(3 * segs + 8);
  }
  {
    const size_t a = (size_t)x->max_units * c.n_kv_heads, b = (size_t)x->max_tc_segs * kScoreWarps;
    ok = ok && dev_alloc(&x->d_colpart[0], (a > b ? a : b) * G * 2) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_colpart[1], (a > b ? a : b) * G * 2) == cudaSuccess;
  }
  if (x->use_tc) {
    const size_t n_index = 2 * (size_t)(max_pairs + 1) + 2 * (size_t)(x->n_sm + 1);
    ok = ok && cudaMallocHost((void**)&x->h_tc_ops, sizeof(ScoreOp) * x->max_tc_ops) == cudaSuccess;
    ok = ok && cudaMallocHost((void**)&x->h_tc_index, sizeof(int32_t) * n_index) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_tc_ops, x->max_tc_ops) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_tc_index, n_index) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_tc_sync, 2 * (size_t)max_pairs) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_tc_rowpart, (size_t)x->max_tc_segs * kScoreGroups * 128) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_lse2_tc, (size_t)max_pairs * 128) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_hrow[0], (size_t)max_pairs * 128) == cudaSuccess;
    ok = ok && dev_alloc(&x->d_hrow[1], (size_t)max_pairs * 128) == cudaSuccess;
  }
  // decode-time state: one slot per packed row plus one spare per (request, layer, head)
  x->dec_rows_cap = x->pos_packed_cap + x->max_lists;
  ok = ok && dev_alloc(&x->d_dec_off, (size_t)R * c.n_layers + 1) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_packed_off, (size_t)R * c.n_layers + 1) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_score, (size_t)x->dec_rows_cap) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_tmp, (size_t)c.n_kv_heads * (size_t)(c.n_q_heads / c.n_kv_heads + 1) *
                                          (size_t)(T + R)) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_pos, (size_t)x->dec_rows_cap) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_order, (size_t)x->dec_rows_cap) == cudaSuccess;
  ok = ok && dev_alloc(&x->d_dec_meta, (size_t)x->max_lists) == cudaSuccess;
  ok = ok && cudaMallocHost((void**)&x->h_budget_stage, sizeof(int32_t) * R * c.n_layers) == cudaSuccess;
  ok = ok && cudaMemset(x->d_status, 0, sizeof(int32_t)) == cudaSuccess;
  ok = ok && cudaMemset(x->d_budget[0], 0, sizeof(int32_t) * R * c.n_layers) == cudaSuccess;
  ok = ok && cudaMemset(x->d_budget[1], 0, sizeof(int32_t) * R * c.n_layers) == cudaSuccess;
  ok = ok && cudaMemset(x->d_P, 0, sizeof(double) * R * c.n_layers) == cudaSuccess;
  ok = ok && cudaMemset(x->d_H, 0, sizeof(double) * R * c.n_layers) == cudaSuccess;
  ok = ok && cudaMemset(x->d_V, 0, sizeof(double) * R * c.n_layers) == cudaSuccess;
  if (!ok) { cudaGetLastError(); free_ctx(x); return CAKE_ERR_CUDA; }
  x->n_req = -1;                                  // no batch yet
  *out = x;
  return CAKE_OK;
}

int32_t cake_destroy(cake_ctx* ctx) {
  if (!ctx) return CAKE_ERR_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  free_ctx(ctx);
  return cuda_status(e);
}

int32_t cake_begin(cake_ctx* ctx, int32_t n_req, const int64_t* cu, void* stream) {
  if (!ctx || n_req < 0 || (n_req > 0 && !cu)) return CAKE_ERR_ARG;
  const cake_config& c = ctx->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  if (n_req > c.max_requests) return CAKE_ERR_CAPACITY;
  if (n_req > 0) {
    if (cu[0] != 0) return CAKE_ERR_ARG;
    for (int r = 0; r < n_req; ++r)
      if (cu[r + 1] - cu[r] < c.window) return CAKE_ERR_ARG;
    if (cu[n_req] > c.max_total_tokens) return CAKE_ERR_CAPACITY;
  }
  // the previous batch's cascade must be done before its state is reset or overwritten
  CAKE_CUDA_TRY(main_after_side(ctx, st));
  const int64_t T = n_req > 0 ? cu[n_req] : 0;
  const bool same = ctx->n_req == n_req && n_req > 0 &&
                    memcmp(ctx->h_cu, cu, sizeof(int64_t) * (n_req + 1)) == 0;
  if (!same && n_req > 0) {
    // From here on the host tables are rebuilt in place: until that has succeeded the context
    // describes no batch at all, so a failure cannot leave it half in the old batch and half in
    // the new one (a later cake_begin then rebuilds everything, and other calls are refused).
    ctx->n_req = -1;
    if (ctx->upload_pending) {                    // staging buffers still feed an earlier copy
      CAKE_CUDA_TRY(cudaEventSynchronize(ctx->upload_done));
      ctx->upload_pending = false;
    }
    const int32_t unit_keys = choose_unit_keys(T, c.n_kv_heads, ctx->n_sm);
    int32_t nu = 0, max_split = 0;
    // the pooling / scatter kernels run on the SMs the score kernel leaves free: about two CTAs
    // per such SM over all (request, head) pairs
    const int reserve = ctx->n_sm - ctx->n_sm_score;
    int want_split = (2 * (reserve > 0 ? reserve : 8)) / (n_req * c.n_kv_heads);
    if (want_split < 1) want_split = 1;
    int64_t list_off = 0, bound = 0;
    for (int r = 0; r < n_req; ++r) {
      ReqInfo& q = ctx->h_req[r];
      q.cu = cu[r];
      q.N = (int32_t)(cu[r + 1] - cu[r]);
      q.n = q.N - c.window;
      q.keep_all = q.N <= c.total_budget / c.n_layers ? 1 : 0;
      q.list_off = list_off;
      list_off += (int64_t)q.n * c.n_layers * c.n_kv_heads;
      {
        const int chunks = (q.N + kChunkKeys - 1) / kChunkKeys;
        int ns = chunks < want_split ? chunks : want_split;
        q.span = ((chunks + ns - 1) / ns) * kChunkKeys;
        q.nsplit = (q.N + q.span - 1) / q.span;
        if (q.nsplit > max_split) max_split = q.nsplit;
      }
      q.unit0 = nu;
      for (int32_t k0 = 0; k0 < q.N; k0 += unit_keys) {
        ScoreUnit& u = ctx->h_units[nu++];
        u.req = r; u.key0 = k0; u.nkeys = q.N - k0 < unit_keys ? q.N - k0 : unit_keys; u.pad = 0;
      }
      q.nunits = nu - q.unit0;
      const int64_t full = (int64_t)c.n_layers * q.N;
      bound += (int64_t)c.n_kv_heads * (c.total_budget < full ? c.total_budget : full);
    }
    if (list_off > ctx->list_elems || nu > ctx->max_units) return CAKE_ERR_CAPACITY;
    ctx->n_split = max_split;
    if (ctx->use_tc) {
      const int32_t prc = tc_build_plan(ctx, n_req);
      if (prc != CAKE_OK) return prc;
    }
    ctx->n_units = nu;
    ctx->packed_rows_bound = bound;
    memcpy(ctx->h_cu, cu, sizeof(int64_t) * (n_req + 1));
    CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->d_req, ctx->h_req, sizeof(ReqInfo) * n_req,
                                  cudaMemcpyHostToDevice, st));
    CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->d_units, ctx->h_units, sizeof(ScoreUnit) * nu,
                                  cudaMemcpyHostToDevice, st));
    if (ctx->use_tc && ctx->n_tc_ctas > 0) {
      const size_t n_index = 2 * (size_t)(n_req * c.n_kv_heads + 1) + 2 * (size_t)(ctx->n_sm + 1);
      CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->d_tc_ops, ctx->h_tc_ops,
                                    sizeof(ScoreOp) * (ctx->n_tc_ops_full + ctx->n_tc_ops_b),
                                    cudaMemcpyHostToDevice, st));
      CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->d_tc_index, ctx->h_tc_index, sizeof(int32_t) * n_index,
                                    cudaMemcpyHostToDevice, st));
    }
    CAKE_CUDA_TRY(cudaEventRecord(ctx->upload_done, st));
    ctx->upload_pending = true;
  }
  if (n_req == 0) { ctx->n_units = 0; ctx->n_split = 0; ctx->packed_rows_bound = 0; ctx->n_tc_ctas = 0; }
  if (ctx->use_tc) {
    ctx->tc_epoch = 0;
    CAKE_CUDA_TRY(cudaMemsetAsync(ctx->d_tc_sync, 0, sizeof(uint32_t) * 2 * ctx->max_pairs, st));
  }
  ctx->n_req = n_req;
  ctx->total_tokens = T;
  ctx->debug_epoch_skew = 0;
  ctx->dec_ready = false;
  ctx->n_ind = ctx->n_pref = ctx->n_evicted = 0;
  ctx->alloc_of_buf[0] = ctx->alloc_of_buf[1] = -1;
  ctx->last_alloc = -1;
  CAKE_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), st));
  ctx->pool_recorded[0] = ctx->pool_recorded[1] = false;
  ctx->evict_recorded[0] = ctx->evict_recorded[1] = false;
  CAKE_CUDA_TRY(side_after(ctx, st));
  return CAKE_OK;
}

int32_t cake_score_layer(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                         const float* lse, void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (ctx->n_req > 0 && (!q_win || !k)) return CAKE_ERR_ARG;
  if (layer != ctx->n_ind || ctx->n_evicted != layer) return CAKE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const int par = layer & 1;
  // the score kernel's outputs of this parity were last read by the pooling of layer - 2; the rest
  // of that layer's cascade works on its own data and may still be running
  if (ctx->pool_recorded[par]) CAKE_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev_pool[par], 0));
  int32_t rc = ctx->use_tc ? launch_score_tc(ctx, layer, q_win, k, lse, st)
                           : launch_score_simt(ctx, layer, q_win, k, lse, st);
  if (rc != CAKE_OK) return rc;
  // Pooling and the preference run on their own stream beside the next layer's scoring and
  // beside the budgets and eviction of the layer before; the pooled buffer of this parity was
  // last read by the eviction of layer - 2.
  CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_score[par], st));
  CAKE_CUDA_TRY(cudaStreamWaitEvent(ctx->pool_st, ctx->ev_score[par], 0));
  if (ctx->evict_recorded[par]) CAKE_CUDA_TRY(cudaStreamWaitEvent(ctx->pool_st, ctx->ev_evict[par], 0));
  const int sp = prof_begin(ctx, CAKE_PROF_FINALIZE, ctx->pool_st);
  rc = launch_pool(ctx, layer, true, true, ctx->pool_st);
  prof_end(ctx, sp, ctx->pool_st);
  if (rc != CAKE_OK) return rc;
  CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_pool[par], ctx->pool_st));
  ctx->pool_recorded[par] = true;
  ctx->n_ind = layer + 1;
  if (ctx->n_pref < layer + 1) ctx->n_pref = layer + 1;
  return CAKE_OK;
}

int32_t cake_allocate(cake_ctx* ctx, int32_t stage, void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  if (stage < 0 || stage >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (stage >= ctx->n_pref) return CAKE_ERR_STATE;
  (void)stream;                      // ordered by the internal streams
  // The budgets have a stream of their own, so that those of stage m are computed beside the
  // eviction of stage m-1.  They need the newest layer's preference (pooling stream), and their
  // buffer was last read by the eviction of stage m-2; the budgets of stage m-1, which they fall
  // back to, were written on this stream.
  cudaStream_t ast = ctx->alloc_st;
  if (ctx->pool_recorded[stage & 1]) CAKE_CUDA_TRY(cudaStreamWaitEvent(ast, ctx->ev_pool[stage & 1], 0));
  if (ctx->evict_recorded[stage & 1]) CAKE_CUDA_TRY(cudaStreamWaitEvent(ast, ctx->ev_evict[stage & 1], 0));
  const int sp = prof_begin(ctx, CAKE_PROF_ALLOCATE, ast);
  int32_t rc = launch_allocate(ctx, stage, ast);
  prof_end(ctx, sp, ast);
  if (rc != CAKE_OK) return rc;
  CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_alloc[stage & 1], ast));
  ctx->alloc_of_buf[stage & 1] = stage;
  ctx->last_alloc = stage;
  return CAKE_OK;
}

int32_t cake_evict(cake_ctx* ctx, int32_t stage, void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  if (stage < 0 || stage >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (stage != ctx->n_evicted || ctx->n_ind != stage + 1) return CAKE_ERR_STATE;
  if (ctx->alloc_of_buf[stage & 1] != stage) return CAKE_ERR_STATE;
  if (stage > 0 && ctx->alloc_of_buf[(stage + 1) & 1] != stage - 1) return CAKE_ERR_STATE;
  (void)stream;
  CAKE_CUDA_TRY(cudaStreamWaitEvent(ctx->side, ctx->ev_alloc[stage & 1], 0));
  const int sp = prof_begin(ctx, CAKE_PROF_EVICT, ctx->side);
  int32_t rc = launch_evict(ctx, stage, ctx->side);
  prof_end(ctx, sp, ctx->side);
  if (rc != CAKE_OK) return rc;
  CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_evict[stage & 1], ctx->side));
  ctx->evict_recorded[stage & 1] = true;
  ctx->n_evicted = stage + 1;
  return CAKE_OK;
}

int32_t cake_compact(cake_ctx* ctx, int32_t layer_lo, int32_t layer_hi, const void* const* k_layers,
                     const void* const* v_layers, void* k_out, void* v_out,
                     int64_t* row_offsets_out, int32_t* positions_out, void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  if (layer_lo < 0 || layer_hi > ctx->cfg.n_layers || layer_lo > layer_hi) return CAKE_ERR_ARG;
  if (!row_offsets_out) return CAKE_ERR_ARG;
  if (layer_hi > ctx->n_evicted || ctx->n_evicted < 1) return CAKE_ERR_STATE;
  if (ctx->last_alloc != ctx->n_evicted - 1) return CAKE_ERR_STATE;
  LayerPtrs ptrs;
  memset(&ptrs, 0, sizeof(ptrs));
  if (ctx->n_req > 0 && layer_hi > layer_lo) {
    if (!k_layers || !v_layers || !k_out || !v_out) return CAKE_ERR_ARG;
    for (int l = layer_lo; l < layer_hi; ++l) {
      if (!k_layers[l] || !v_layers[l]) return CAKE_ERR_ARG;
      ptrs.k[l] = k_layers[l];
      ptrs.v[l] = v_layers[l];
    }
  }
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  const int sp = prof_begin(ctx, CAKE_PROF_COMPACT, (cudaStream_t)stream);
  const int32_t rc = launch_compact(ctx, layer_lo, layer_hi, ptrs, k_out, v_out, row_offsets_out,
                                    positions_out, (cudaStream_t)stream);
  prof_end(ctx, sp, (cudaStream_t)stream);
  return rc;
}

int32_t cake_compact_int4(cake_ctx* ctx, int32_t layer_lo, int32_t layer_hi, const void* const* k_layers,
                          const void* const* v_layers, int32_t group, uint8_t* k_codes, float* k_scale,
                          float* k_zero, uint8_t* v_codes, float* v_scale, float* v_zero,
                          int64_t* row_offsets_out, int64_t* kgroup_offsets_out, int32_t* positions_out,
                          void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  const cake_config& c = ctx->cfg;
  if (layer_lo < 0 || layer_hi > c.n_layers || layer_lo > layer_hi) return CAKE_ERR_ARG;
  if ((group != 32 && group != 64 && group != 128) || group > c.head_dim) return CAKE_ERR_ARG;
  if (!row_offsets_out || !kgroup_offsets_out) return CAKE_ERR_ARG;
  if (layer_hi > ctx->n_evicted || ctx->n_evicted < 1) return CAKE_ERR_STATE;
  if (ctx->last_alloc != ctx->n_evicted - 1) return CAKE_ERR_STATE;
  LayerPtrs ptrs;
  memset(&ptrs, 0, sizeof(ptrs));
  if (ctx->n_req > 0 && layer_hi > layer_lo) {
    if (!k_layers || !v_layers || !k_codes || !k_scale || !k_zero || !v_codes || !v_scale || !v_zero)
      return CAKE_ERR_ARG;
    for (int l = layer_lo; l < layer_hi; ++l) {
      if (!k_layers[l] || !v_layers[l]) return CAKE_ERR_ARG;
      ptrs.k[l] = k_layers[l];
      ptrs.v[l] = v_layers[l];
    }
  }
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  const int sp = prof_begin(ctx, CAKE_PROF_COMPACT, (cudaStream_t)stream);
  const int32_t rc = launch_compact_int4(ctx, layer_lo, layer_hi, ptrs, group, k_codes, k_scale, k_zero, v_codes,
                                         v_scale, v_zero, row_offsets_out, kgroup_offsets_out, positions_out,
                                         (cudaStream_t)stream);
  prof_end(ctx, sp, (cudaStream_t)stream);
  return rc;
}

int64_t cake_packed_rows_bound(const cake_ctx* ctx) {
  if (!ctx) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  return ctx->packed_rows_bound;
}

int32_t cake_get_indicators(cake_ctx* ctx, int32_t layer, float* out, void* stream) {
  if (!ctx || !out) return CAKE_ERR_ARG;
  if (ctx->n_req < 0 || layer != ctx->n_ind - 1) return CAKE_ERR_STATE;
  if (ctx->total_tokens == 0) return CAKE_OK;
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  CAKE_CUDA_TRY(cudaMemcpyAsync(out, ctx->d_fresh[layer & 1],
                                sizeof(float) * ctx->cfg.n_kv_heads * ctx->total_tokens,
                                cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return CAKE_OK;
}

int32_t cake_get_preferences(cake_ctx* ctx, double* H, double* V, double* P, void* stream) {
  if (!ctx) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  const size_t bytes = sizeof(double) * ctx->n_req * ctx->cfg.n_layers;
  cudaStream_t st = (cudaStream_t)stream;
  if (bytes == 0) return CAKE_OK;
  CAKE_CUDA_TRY(main_after_side(ctx, st));
  if (H) CAKE_CUDA_TRY(cudaMemcpyAsync(H, ctx->d_H, bytes, cudaMemcpyDeviceToDevice, st));
  if (V) CAKE_CUDA_TRY(cudaMemcpyAsync(V, ctx->d_V, bytes, cudaMemcpyDeviceToDevice, st));
  if (P) CAKE_CUDA_TRY(cudaMemcpyAsync(P, ctx->d_P, bytes, cudaMemcpyDeviceToDevice, st));
  return CAKE_OK;
}

int32_t cake_set_indicators(cake_ctx* ctx, int32_t layer, const float* in, void* stream) {
  if (!ctx || !in) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (layer != ctx->n_ind || ctx->n_evicted != layer) return CAKE_ERR_STATE;
  // earlier stages may still be working on the internal streams
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  if (ctx->total_tokens > 0)
    CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->d_fresh[layer & 1], in,
                                  sizeof(float) * ctx->cfg.n_kv_heads * ctx->total_tokens,
                                  cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  CAKE_CUDA_TRY(side_after(ctx, (cudaStream_t)stream));
  // bucket histogram of the supplied values (they are taken as already pooled)
  const int32_t rc = launch_pool(ctx, layer, false, false, ctx->side);
  if (rc != CAKE_OK) return rc;
  ctx->pool_recorded[layer & 1] = false;             // same stream as the budgets: nothing to wait for
  ctx->n_ind = layer + 1;
  return CAKE_OK;
}

int32_t cake_set_preferences(cake_ctx* ctx, int32_t n_set, const double* P, void* stream) {
  if (!ctx || !P) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  if (n_set < 1 || n_set > ctx->cfg.n_layers) return CAKE_ERR_ARG;
  // A layer that has been evicted stored only the entries its budget could still reach; a new
  // preference could make that budget grow again (Proposition 1 would no longer hold).
  if (ctx->n_evicted > 0) return CAKE_ERR_STATE;
  if (ctx->n_req > 0) {
    CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
    CAKE_CUDA_TRY(cudaMemcpy2DAsync(ctx->d_P, sizeof(double) * ctx->cfg.n_layers, P,
                                    sizeof(double) * n_set, sizeof(double) * n_set, ctx->n_req,
                                    cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    CAKE_CUDA_TRY(side_after(ctx, (cudaStream_t)stream));
  }
  if (ctx->n_pref < n_set) ctx->n_pref = n_set;
  return CAKE_OK;
}

int32_t cake_get_budgets(cake_ctx* ctx, int32_t* out, void* stream) {
  if (!ctx || !out) return CAKE_ERR_ARG;
  if (ctx->n_req < 0 || ctx->last_alloc < 0) return CAKE_ERR_STATE;
  if (ctx->n_req == 0) return CAKE_OK;
  const int total = ctx->n_req * ctx->cfg.n_layers;
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  budgets_with_window<<<(total + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
      ctx->d_budget[ctx->last_alloc & 1], out, ctx->n_req, ctx->cfg.n_layers, ctx->last_alloc + 1,
      ctx->cfg.window);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t cake_get_positions(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* out, int64_t capacity,
                           void* stream) {
  if (!ctx || !out || capacity < 0) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  if (req < 0 || req >= ctx->n_req || layer < 0 || layer >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (layer >= ctx->n_evicted || ctx->last_alloc != ctx->n_evicted - 1) return CAKE_ERR_STATE;
  CAKE_CUDA_TRY(main_after_side(ctx, (cudaStream_t)stream));
  return launch_get_positions(ctx, req, layer, out, capacity, (cudaStream_t)stream);
}

int32_t cake_status(cake_ctx* ctx, int32_t* device_status_out, void* stream) {
  if (!ctx) return CAKE_ERR_ARG;
  int32_t s = 0;
  cudaStream_t st = (cudaStream_t)stream;
  CAKE_CUDA_TRY(main_after_side(ctx, st));
  CAKE_CUDA_TRY(cudaMemcpyAsync(&s, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CAKE_CUDA_TRY(cudaStreamSynchronize(st));
  if (device_status_out) *device_status_out = s;
  return CAKE_OK;
}

int32_t cake_profile_enable(cake_ctx* ctx, int32_t on) {
  if (!ctx) return CAKE_ERR_ARG;
  Profiler& p = ctx->prof;
  if (on && !p.spans) {
    p.cap = 16384;
    p.spans = (ProfSpan*)calloc(p.cap, sizeof(ProfSpan));
    if (!p.spans) { p.cap = 0; return CAKE_ERR_CUDA; }
  }
  p.on = on != 0;
  return CAKE_OK;
}

int32_t cake_profile_read(cake_ctx* ctx, double* ms_out, int64_t* spans_out, void* stream) {
  if (!ctx || !ms_out || !spans_out) return CAKE_ERR_ARG;
  CAKE_CUDA_TRY(cudaStreamSynchronize(ctx->side));
  CAKE_CUDA_TRY(cudaStreamSynchronize(ctx->pool_st));
  CAKE_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  for (int k = 0; k < CAKE_PROF_KINDS; ++k) { ms_out[k] = 0.0; spans_out[k] = 0; }
  Profiler& p = ctx->prof;
  for (int i = 0; i < p.used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.spans[i].a, p.spans[i].b) == cudaSuccess) {
      ms_out[p.spans[i].kind] += ms;
      spans_out[p.spans[i].kind] += 1;
    }
  }
  p.used = 0;
  cudaGetLastError();
  return CAKE_OK;
}

int32_t cake_uses_tensor_cores(const cake_ctx* ctx) {
  if (!ctx) return CAKE_ERR_ARG;
  return ctx->use_tc ? 1 : 0;
}

int64_t cake_decode_rows_bound(const cake_ctx* ctx) {
  if (!ctx) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  return ctx->packed_rows_bound + (int64_t)ctx->n_req * ctx->cfg.n_layers * ctx->cfg.n_kv_heads;
}

int32_t cake_decode_begin(cake_ctx* ctx, const void* const* k_layers, const void* const* v_layers,
                          void* k_cache, void* v_cache, int64_t* row_offsets_out, int32_t update_mode,
                          void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  const cake_config& c = ctx->cfg;
  if (update_mode < CAKE_DECODE_ADD || update_mode > CAKE_DECODE_REPLACE) return CAKE_ERR_ARG;
  if (ctx->n_evicted != c.n_layers || ctx->last_alloc != c.n_layers - 1) return CAKE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  LayerPtrs ptrs;
  memset(&ptrs, 0, sizeof(ptrs));
  if (ctx->n_req > 0) {
    if (!k_layers || !v_layers || !k_cache || !v_cache) return CAKE_ERR_ARG;
    for (int l = 0; l < c.n_layers; ++l) {
      if (!k_layers[l] || !v_layers[l]) return CAKE_ERR_ARG;
      ptrs.k[l] = k_layers[l];
      ptrs.v[l] = v_layers[l];
    }
  }
  CAKE_CUDA_TRY(main_after_side(ctx, st));
  // the step kernel's shared memory is sized from the largest head (up to its limit): read the
  // final budgets back
  ctx->dec_max_cap = 1;
  if (ctx->n_req > 0) {
    const size_t nb = sizeof(int32_t) * ctx->n_req * c.n_layers;
    CAKE_CUDA_TRY(cudaMemcpyAsync(ctx->h_budget_stage, ctx->d_budget[(c.n_layers - 1) & 1], nb,
                                  cudaMemcpyDeviceToHost, st));
    CAKE_CUDA_TRY(cudaStreamSynchronize(st));
    for (int i = 0; i < ctx->n_req * c.n_layers; ++i) {
      const int64_t cap = (int64_t)ctx->h_budget_stage[i] + c.window + 1;
      if (cap > ctx->dec_max_cap) ctx->dec_max_cap = cap;
    }
  }
  const int32_t rc = launch_decode_begin(ctx, ptrs, k_cache, v_cache, row_offsets_out, st);
  if (rc != CAKE_OK) return rc;
  ctx->dec_update_mode = update_mode;
  ctx->dec_ready = true;
  return CAKE_OK;
}

int32_t cake_decode_step(cake_ctx* ctx, int32_t layer, const void* q_new, const void* k_new,
                         const void* v_new, void* k_cache, void* v_cache, void* stream) {
  if (!ctx || ctx->n_req < 0) return ctx ? CAKE_ERR_STATE : CAKE_ERR_ARG;
  if (!ctx->dec_ready) return CAKE_ERR_STATE;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  if (ctx->n_req > 0 && (!q_new || !k_new || !v_new || !k_cache || !v_cache)) return CAKE_ERR_ARG;
  return launch_decode_step(ctx, layer, q_new, k_new, v_new, k_cache, v_cache, (cudaStream_t)stream);
}

int32_t cake_decode_get_state(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* positions_out,
                              float* scores_out, int32_t* slots_out, void* stream) {
  if (!ctx) return CAKE_ERR_ARG;
  if (ctx->n_req < 0 || !ctx->dec_ready) return CAKE_ERR_STATE;
  if (req < 0 || req >= ctx->n_req || layer < 0 || layer >= ctx->cfg.n_layers) return CAKE_ERR_ARG;
  return launch_decode_read(ctx, req, layer, positions_out, scores_out, slots_out, (cudaStream_t)stream);
}

int32_t cake_set_wait_limit(cake_ctx* ctx, int64_t cycles) {
  if (!ctx || cycles < 0) return CAKE_ERR_ARG;
  ctx->wait_limit_cycles = cycles;
  return CAKE_OK;
}

int32_t cake_debug_skew_sync(cake_ctx* ctx, int32_t delta) {
  if (!ctx) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  ctx->debug_epoch_skew = delta;
  return CAKE_OK;
}

int32_t cake_plan_check(const cake_config* cfg, int32_t n_sm, int32_t reserved_sms, int32_t n_req,
                        const int64_t* cu_seqlens_host, int32_t* info8) {
  if (!cfg || !info8 || n_sm < 1 || reserved_sms < 0 || n_req < 0 || (n_req > 0 && !cu_seqlens_host))
    return CAKE_ERR_ARG;
  for (int r = 0; r < n_req; ++r)
    if (cu_seqlens_host[r + 1] - cu_seqlens_host[r] < cfg->window) return CAKE_ERR_ARG;
  return tc_plan_check(*cfg, n_sm, reserved_sms, n_req, cu_seqlens_host, info8);
}

int32_t cake_plan_info(const cake_ctx* ctx, int32_t* out8) {
  if (!ctx || !out8) return CAKE_ERR_ARG;
  if (ctx->n_req < 0) return CAKE_ERR_STATE;
  const bool tc = ctx->use_tc;
  out8[0] = tc ? 1 : 0;
  out8[1] = tc ? ctx->n_tc_ctas : 0;
  out8[2] = tc ? ctx->n_tc_waves : 0;
  out8[3] = tc && ctx->n_tc_ctas > 0 ? ctx->tc_merge_ways : 0;
  out8[4] = tc ? ctx->n_tc_asegs : 0;
  out8[5] = tc ? ctx->n_tc_bsegs : 0;
  out8[6] = tc ? ctx->n_tc_ops_full : 0;
  out8[7] = ctx->n_sm - ctx->n_sm_score;
  return CAKE_OK;
}

const char* cake_strerror(int32_t code) {
  switch (code) {
    case CAKE_OK: return "ok";
    case CAKE_ERR_ARG: return "invalid argument";
    case CAKE_ERR_BUDGET: return "total budget smaller than n_layers * window";
    case CAKE_ERR_CAPACITY: return "batch exceeds the context's capacity";
    case CAKE_ERR_NONFINITE: return "non-finite or negative preference";
    case CAKE_ERR_TIMEOUT: return "device-side wait timed out";
    case CAKE_ERR_CUDA: return "CUDA runtime error";
    case CAKE_ERR_STATE: return "call out of order";
    default: return "unknown error";
  }
}

int64_t cake_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
