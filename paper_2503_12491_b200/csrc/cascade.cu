// Layer finalisation (preference, pooling), the device-side budget allocator and
// the per-head top-k eviction of the cascade.
#include "cake_internal.cuh"

#include <math_constants.h>

namespace cake {
namespace {

__device__ inline void raise_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

// ------------------------------------------------------------------ finalize
// H_h = -ln2 * sum p*log2(p), V_h = sum_j Var_i; layer values are the means over
// the query heads; P = H^(1/tau1) * V^(1/tau2)  (Eq. 4-6).  Partials are added in
// unit order in double precision, so the result does not depend on scheduling.
__global__ void finalize_layer(const float* __restrict__ colpart, const ReqInfo* __restrict__ reqs,
                               double* __restrict__ dH, double* __restrict__ dV,
                               double* __restrict__ dP, int32_t* __restrict__ status, int layer,
                               int L, int Hq, int Hkv, double inv_tau1, double inv_tau2) {
  __shared__ double sh[2][256];
  const int req = blockIdx.x;
  const ReqInfo rq = reqs[req];
  const int G = Hq / Hkv;
  double hsum = 0.0, vsum = 0.0;
  for (int h = threadIdx.x; h < Hq; h += blockDim.x) {      // one head per thread
    const int g = h / G, hl = h - g * G;
    double a = 0.0, b = 0.0;
    for (int u = rq.unit0; u < rq.unit0 + rq.nunits; ++u) {
      const float* p = colpart + (((size_t)u * Hkv + g) * G + hl) * 2;
      a += (double)p[0];
      b += (double)p[1];
    }
    hsum += -0.6931471805599453 * a;
    vsum += b;
  }
  sh[0][threadIdx.x] = hsum;
  sh[1][threadIdx.x] = vsum;
  __syncthreads();
  if (threadIdx.x == 0) {
    double H = 0.0, V = 0.0;
    for (int t = 0; t < blockDim.x; ++t) { H += sh[0][t]; V += sh[1][t]; }
    H /= (double)Hq;
    V /= (double)Hq;
    const double P = pow(H, inv_tau1) * pow(V, inv_tau2);
    dH[(size_t)req * L + layer] = H;
    dV[(size_t)req * L + layer] = V;
    dP[(size_t)req * L + layer] = P;
    if (!(P >= 0.0) || isinf(P)) raise_status(status, CAKE_ERR_NONFINITE);
  }
}

// Same for the tensor-core path: one warp per query head.  Variance partials are indexed
// by (pass-B segment, statistics warp); the entropy comes either from the row pass
// (hrow: sum_j p log2 p of every window row, tile row order r' = i*G + h) or, when the
// caller supplied the denominators, from the column pass partials.
__device__ inline double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void finalize_layer_tc(const float* __restrict__ colpart,
                                  const int32_t* __restrict__ pair_seg,
                                  const float* __restrict__ hrow, int use_hrow, int rows,
                                  double* __restrict__ dH, double* __restrict__ dV,
                                  double* __restrict__ dP, int32_t* __restrict__ status, int layer,
                                  int L, int Hq, int Hkv, double inv_tau1, double inv_tau2) {
  __shared__ double sh[2][32];
  const int req = blockIdx.x;
  const int G = Hq / Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
  double hsum = 0.0, vsum = 0.0;                         // per warp, over its heads
  for (int h = warp; h < Hq; h += nwarp) {
    const int g = h / G, hl = h - g * G;
    const int pair = req * Hkv + g;
    double a = 0.0, b = 0.0;
    const int s_lo = pair_seg[pair] * kScoreWarps, s_hi = pair_seg[pair + 1] * kScoreWarps;
    for (int sg = s_lo + lane; sg < s_hi; sg += 32) {
      const float2 p = *reinterpret_cast<const float2*>(colpart + ((size_t)sg * G + hl) * 2);
      a += (double)p.x;
      b += (double)p.y;
    }
    if (use_hrow) {
      a = 0.0;
      for (int r = hl + lane * G; r < rows; r += 32 * G) a += (double)hrow[(size_t)pair * 128 + r];
    }
    hsum += -0.6931471805599453 * warp_sum_f64(a);
    vsum += warp_sum_f64(b);
  }
  if (lane == 0) { sh[0][warp] = hsum; sh[1][warp] = vsum; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double H = 0.0, V = 0.0;
    for (int t = 0; t < nwarp; ++t) { H += sh[0][t]; V += sh[1][t]; }
    H /= (double)Hq;
    V /= (double)Hq;
    const double P = pow(H, inv_tau1) * pow(V, inv_tau2);
    dH[(size_t)req * L + layer] = H;
    dV[(size_t)req * L + layer] = V;
    dP[(size_t)req * L + layer] = P;
    if (!(P >= 0.0) || isinf(P)) raise_status(status, CAKE_ERR_NONFINITE);
  }
}

// --------------------------------------------------------------------- pool
// fresh[g][t] = pool(raw[g][.]) over the request's non-window tokens; window
// slots get +inf (Section 4.3).
__global__ void pool_indicators(const float* __restrict__ raw, float* __restrict__ fresh,
                                const ReqInfo* __restrict__ reqs, int n_req, int64_t T, int kp,
                                int mode) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const int g = blockIdx.y;
  int lo = 0, hi = n_req - 1;                 // last request with cu <= t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].cu <= t) lo = mid; else hi = mid - 1;
  }
  const ReqInfo rq = reqs[lo];
  const int j = (int)(t - rq.cu);
  float out;
  if (j >= rq.n) {
    out = CUDART_INF_F;
  } else {
    const float* src = raw + (size_t)g * T + rq.cu;
    const int r = kp >> 1;
    const int a = max(0, j - r), b = min(rq.n, j + r + 1);
    if (mode == CAKE_POOL_MAX) {
      float m = src[a];
      for (int x = a + 1; x < b; ++x) m = fmaxf(m, src[x]);
      out = m;
    } else {
      float s = 0.f;
      for (int x = a; x < b; ++x) s += src[x];
      out = s / (float)kp;
    }
  }
  fresh[(size_t)g * T + t] = out;
}

// ----------------------------------------------------------------- allocate
// Number of s in [0, lim) with P/(s + 1/2) >= x (IEEE double division).
__device__ inline int64_t count_ge(double P, double x, int64_t lim) {
  if (!(P > 0.0) || isinf(x)) return 0;
  const double est = floor(P / x - 0.5) + 1.0;
  int64_t c = est < 0.0 ? 0 : (est > (double)lim ? lim : (int64_t)est);
  while (c > 0 && P / ((double)(c - 1) + 0.5) < x) --c;
  while (c < lim && P / ((double)c + 0.5) >= x) ++c;
  return c;
}

__device__ inline int64_t warp_sum64(int64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

constexpr int kMaxCand = 1024;

// One warp per request.  Webster / Sainte-Lague: the `seats` largest priorities
// P_l/(s+1/2) win, ties to the lower layer then the lower s.  The common divisor
// is bracketed analytically (sum_l round(P_l/x) is within L/2 of sum(P)/x), the few
// priorities inside the bracket are ranked exactly; if the bracket ever fails the
// threshold is found by bisection over the bit patterns of the doubles.
__global__ void allocate_budgets(const double* __restrict__ dP, const ReqInfo* __restrict__ reqs,
                                 const int32_t* __restrict__ prev, int32_t* __restrict__ cur,
                                 int32_t* __restrict__ status, int stage, int L, int64_t seats) {
  __shared__ double sP[CAKE_MAX_LAYERS];
  __shared__ int64_t s_lo[CAKE_MAX_LAYERS];
  __shared__ int32_t s_off[CAKE_MAX_LAYERS + 1];
  __shared__ int32_t s_win[CAKE_MAX_LAYERS];
  __shared__ double c_val[kMaxCand];
  __shared__ int32_t c_lay[kMaxCand];
  __shared__ int32_t c_s[kMaxCand];
  const int req = blockIdx.x, lane = threadIdx.x;
  const ReqInfo rq = reqs[req];
  const int La = stage + 1;
  int32_t* out = cur + (size_t)req * L;
  const int32_t* old = prev + (size_t)req * L;
  for (int l = La + lane; l < L; l += 32) out[l] = 0;

  bool bad = false;
  bool anypos = false;
  for (int l = lane; l < La; l += 32) {
    const double p = dP[(size_t)req * L + l];
    sP[l] = p;
    if (!(p >= 0.0) || isinf(p)) bad = true;
    if (p > 0.0) anypos = true;
  }
  bad = __any_sync(0xffffffffu, bad);
  anypos = __any_sync(0xffffffffu, anypos);
  __syncwarp();
  if (bad) {                                   // keep the previous stage's budgets
    raise_status(status, CAKE_ERR_NONFINITE);
    for (int l = lane; l < La; l += 32) out[l] = (l < stage && stage > 0) ? old[l] : 0;
    return;
  }
  if (rq.keep_all) {
    for (int l = lane; l < La; l += 32) out[l] = rq.n;
    return;
  }
  if (!anypos) {
    for (int l = lane; l < La; l += 32) sP[l] = 1.0;
    __syncwarp();
  }
  if (seats <= 0) {
    for (int l = lane; l < La; l += 32) out[l] = 0;
    return;
  }
  double SP = 0.0;                             // same order on every lane
  for (int l = 0; l < La; ++l) SP += sP[l];
  if (isinf(SP)) {
    raise_status(status, CAKE_ERR_NONFINITE);
    for (int l = lane; l < La; l += 32) out[l] = (l < stage && stage > 0) ? old[l] : 0;
    return;
  }
  const int64_t lim = seats + La + 8;
  const double x_lo = SP / (double)(seats + La + 1);
  const double x_hi = seats > La + 1 ? SP / (double)(seats - La - 1) : CUDART_INF;
  int64_t clo = 0, chi = 0;
  for (int l = lane; l < La; l += 32) {
    const int64_t a = count_ge(sP[l], x_hi, lim);
    const int64_t b = count_ge(sP[l], x_lo, lim);
    s_lo[l] = a;
    s_win[l] = 0;
    const int64_t nc = b - a;
    s_off[l + 1] = (int32_t)(nc > kMaxCand ? kMaxCand + 1 : nc);
    clo += a;
    chi += b;
  }
  clo = warp_sum64(clo);
  chi = warp_sum64(chi);
  __syncwarp();
  const bool bracket_ok = clo <= seats && chi >= seats && (chi - clo) <= kMaxCand;
  if (bracket_ok) {
    if (lane == 0) {
      s_off[0] = 0;
      for (int l = 0; l < La; ++l) s_off[l + 1] += s_off[l];
    }
    __syncwarp();
    const int ncand = s_off[La];
    const int64_t need = seats - clo;
    for (int l = lane; l < La; l += 32) {
      const int base = s_off[l], cnt = s_off[l + 1] - base;
      for (int e = 0; e < cnt; ++e) {
        const int64_t s = s_lo[l] + e;
        c_val[base + e] = sP[l] / ((double)s + 0.5);
        c_lay[base + e] = l;
        c_s[base + e] = e;
      }
    }
    __syncwarp();
    for (int c = lane; c < ncand; c += 32) {
      const double v = c_val[c];
      const int l = c_lay[c], e = c_s[c];
      int64_t ahead = 0;
      for (int o = 0; o < ncand; ++o) {
        const double vo = c_val[o];
        const int lo2 = c_lay[o], eo = c_s[o];
        ahead += (vo > v) || (vo == v && (lo2 < l || (lo2 == l && eo < e)));
      }
      if (ahead < need) atomicAdd(&s_win[l], 1);
    }
    __syncwarp();
    for (int l = lane; l < La; l += 32) {
      const int64_t b = s_lo[l] + s_win[l];
      out[l] = (int32_t)(b < (int64_t)rq.n ? b : (int64_t)rq.n);
    }
    return;
  }
  // Fallback: T = largest double x with C(x) >= seats, by bisection on bit patterns.
  double pmax = 0.0;
  for (int l = 0; l < La; ++l) pmax = fmax(pmax, sP[l]);
  unsigned long long lo_bits = 1ull;                                   // C(lo) >= seats
  unsigned long long hi_bits = (unsigned long long)__double_as_longlong(pmax / 0.5) + 1ull;  // C(hi) = 0
  if (hi_bits > 0x7FF0000000000000ull) hi_bits = 0x7FF0000000000000ull;
  for (int it = 0; it < 70 && hi_bits - lo_bits > 1ull; ++it) {
    const unsigned long long mid = lo_bits + ((hi_bits - lo_bits) >> 1);
    const double x = __longlong_as_double((long long)mid);
    int64_t c = 0;
    for (int l = lane; l < La; l += 32) c += count_ge(sP[l], x, lim);
    c = warp_sum64(c);
    if (c >= seats) lo_bits = mid; else hi_bits = mid;
  }
  const double Tthr = __longlong_as_double((long long)lo_bits);
  const double Tnext = __longlong_as_double((long long)(lo_bits + 1ull));
  int64_t gt_sum = 0;
  for (int l = lane; l < La; l += 32) {
    const int64_t gt = count_ge(sP[l], Tnext, lim);
    const int64_t ge = count_ge(sP[l], Tthr, lim);
    s_lo[l] = gt;
    s_win[l] = (int32_t)(ge - gt);            // 0 or 1: priorities strictly decrease in s
    gt_sum += gt;
  }
  gt_sum = warp_sum64(gt_sum);
  __syncwarp();
  if (lane == 0) {
    int64_t need = seats - gt_sum;
    for (int l = 0; l < La; ++l) {
      int64_t b = s_lo[l];
      if (s_win[l] > 0 && need > 0) { b += 1; need -= 1; }
      out[l] = (int32_t)(b < (int64_t)rq.n ? b : (int64_t)rq.n);
    }
  }
}

// -------------------------------------------------------------------- evict
constexpr int EV_THREADS = 1024;
constexpr int EV_ITEMS = 8;

__device__ inline uint32_t ordered_key(float v) {
  const uint32_t b = __float_as_uint(v);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive block scan of two counters packed as (hi: a, lo: b) in 64 bits.
__device__ inline unsigned long long block_excl_scan(unsigned long long v, unsigned long long* warp_tot,
                                                     unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = lane < EV_THREADS / 32 ? warp_tot[lane] : 0ull;
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_tot[lane] = winc - w;                 // exclusive prefix of warp totals
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  return warp_tot[warp] + inc - v;
}

// One CTA per (KV head, layer <= stage, request).  The newest layer reads the
// pooled indicators with implicit positions; older layers read their stored list
// and are compacted in place (an output slot never lies behind its source).
__global__ void __launch_bounds__(EV_THREADS)
evict_layers(const float* __restrict__ fresh, float* __restrict__ list_vals,
             int32_t* __restrict__ list_pos, const ReqInfo* __restrict__ reqs,
             const int32_t* __restrict__ prev, const int32_t* __restrict__ cur, int stage, int L,
             int Hkv, int64_t T) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_krem;
  __shared__ unsigned long long warp_tot[32];
  __shared__ unsigned long long s_total;
  const int g = blockIdx.x, layer = blockIdx.y, req = blockIdx.z;
  const ReqInfo rq = reqs[req];
  const bool is_new = layer == stage;
  const int count = is_new ? rq.n : prev[(size_t)req * L + layer];
  int k = cur[(size_t)req * L + layer];
  k = min(k, count);
  const size_t lbase = rq.list_off + ((size_t)layer * Hkv + g) * rq.cap;
  float* lv = list_vals + lbase;
  int32_t* lp = list_pos + lbase;
  const float* src = is_new ? fresh + (size_t)g * T + rq.cu : lv;
  if (k <= 0) return;
  if (k >= count) {
    if (is_new)
      for (int j = threadIdx.x; j < count; j += EV_THREADS) { lv[j] = src[j]; lp[j] = j; }
    return;
  }
  // ---- radix select of the k-th largest key, 8 bits per pass from the top
  uint32_t prefix = 0, mask = 0, krem = (uint32_t)k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = threadIdx.x; b < 256; b += EV_THREADS) hist[b] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < count; j += EV_THREADS) {
      const uint32_t key = ordered_key(src[j]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t above = 0;
      int dsel = 0;
      for (int dg = 255; dg >= 0; --dg) {
        const uint32_t h = hist[dg];
        if (above + h >= krem) { dsel = dg; break; }
        above += h;
      }
      s_prefix = prefix | ((uint32_t)dsel << shift);
      s_krem = krem - above;
    }
    __syncthreads();
    prefix = s_prefix;
    krem = s_krem;
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t thr = prefix;           // key of the k-th largest element
  const uint32_t need_eq = krem;         // how many elements equal to it are kept (first by position)
  // ---- ordered compaction
  uint32_t gt_base = 0, eq_base = 0;
  for (int c0 = 0; c0 < count; c0 += EV_THREADS * EV_ITEMS) {
    float v[EV_ITEMS];
    int32_t p[EV_ITEMS];
    uint32_t fl[EV_ITEMS];
    uint32_t cg = 0, ce = 0;
    const int j0 = c0 + threadIdx.x * EV_ITEMS;
#pragma unroll
    for (int e = 0; e < EV_ITEMS; ++e) {
      const int j = j0 + e;
      fl[e] = 0;
      if (j < count) {
        v[e] = src[j];
        p[e] = is_new ? j : lp[j];
        const uint32_t key = ordered_key(v[e]);
        fl[e] = key > thr ? 1u : (key == thr ? 2u : 0u);
        cg += fl[e] == 1u;
        ce += fl[e] == 2u;
      }
    }
    unsigned long long tot;
    const unsigned long long ex =
        block_excl_scan(((unsigned long long)cg << 32) | ce, warp_tot, &s_total);
    tot = s_total;
    uint32_t gt_before = gt_base + (uint32_t)(ex >> 32);
    uint32_t eq_before = eq_base + (uint32_t)(ex & 0xffffffffu);
    // all reads of this chunk are done (block_excl_scan synchronised) -> safe to write in place
#pragma unroll
    for (int e = 0; e < EV_ITEMS; ++e) {
      if (fl[e] == 1u) {
        const uint32_t o = gt_before + min(eq_before, need_eq);
        lv[o] = v[e]; lp[o] = p[e];
        ++gt_before;
      } else if (fl[e] == 2u) {
        if (eq_before < need_eq) {
          const uint32_t o = gt_before + eq_before;
          lv[o] = v[e]; lp[o] = p[e];
        }
        ++eq_before;
      }
    }
    gt_base += (uint32_t)(tot >> 32);
    eq_base += (uint32_t)(tot & 0xffffffffu);
    __syncthreads();
  }
}

}  // namespace

int32_t launch_finalize_layer(cake_ctx* ctx, int32_t layer, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  if (ctx->use_tc) {
    finalize_layer_tc<<<ctx->n_req, 1024, 0, st>>>(
        ctx->d_colpart, ctx->d_tc_index + (ctx->n_req * c.n_kv_heads + 1), ctx->d_hrow,
        ctx->hhead_from_rows ? 1 : 0, ctx->rows, ctx->d_H,
        ctx->d_V, ctx->d_P, ctx->d_status, layer, c.n_layers, c.n_q_heads, c.n_kv_heads,
        1.0 / (double)c.tau1, 1.0 / (double)c.tau2);
    count_launch();
    return cuda_status(cudaGetLastError());
  }
  finalize_layer<<<ctx->n_req, 128, 0, st>>>(ctx->d_colpart, ctx->d_req, ctx->d_H, ctx->d_V,
                                              ctx->d_P, ctx->d_status, layer, c.n_layers,
                                              c.n_q_heads, c.n_kv_heads, 1.0 / (double)c.tau1,
                                              1.0 / (double)c.tau2);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_pool(cake_ctx* ctx, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0 || ctx->total_tokens == 0) return CAKE_OK;
  const dim3 grid((unsigned)((ctx->total_tokens + 255) / 256), c.n_kv_heads);
  pool_indicators<<<grid, 256, 0, st>>>(ctx->d_raw, ctx->d_fresh, ctx->d_req, ctx->n_req,
                                        ctx->total_tokens, c.pool_kernel, c.pool_mode);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_allocate(cake_ctx* ctx, int32_t stage, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  allocate_budgets<<<ctx->n_req, 32, 0, st>>>(ctx->d_P, ctx->d_req, ctx->d_budget[(stage + 1) & 1],
                                              ctx->d_budget[stage & 1], ctx->d_status, stage,
                                              c.n_layers, ctx->sel_budget);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_evict(cake_ctx* ctx, int32_t stage, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  const dim3 grid(c.n_kv_heads, stage + 1, ctx->n_req);
  evict_layers<<<grid, EV_THREADS, 0, st>>>(ctx->d_fresh, ctx->list_vals, ctx->list_pos, ctx->d_req,
                                            ctx->d_budget[(stage + 1) & 1], ctx->d_budget[stage & 1],
                                            stage, c.n_layers, c.n_kv_heads, ctx->total_tokens);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
