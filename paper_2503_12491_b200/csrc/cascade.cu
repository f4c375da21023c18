// Layer finalisation (preference, pooling), the device-side budget allocator and
// the per-head top-k eviction of the cascade on bucket-sorted survivor lists.
#include "cake_internal.cuh"

#include <math_constants.h>

#include <cstring>

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

// --------------------------------------------------------------- pool + bins
// Survivor lists are kept sorted by bucket, not by position.  A key's bucket is the top
// kBinBits bits of its order-preserving integer image, counted from the top (bucket 0 holds
// the largest values).  When a layer arrives, its pooled indicators are histogrammed here and
// scattered into bucket order by the eviction kernel; from then on "keep the top b" means
// "all buckets before the one that contains the b-th element, plus the best part of that
// bucket", so a later, smaller budget only moves a threshold and rewrites nothing.
// Order-preserving integer image of a float; -0 and +0 compare equal, as they do as floats.
__device__ inline uint32_t ordered_key(float v) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ inline int bucket_of(uint32_t key) { return (kBins - 1) - (int)(key >> (32 - kBinBits)); }

// Exclusive block scan (blockDim.x <= 1024) of one int per thread; *total gets the sum.
__device__ inline int block_excl_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < nw ? warp_tot[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_tot[lane] = winc - w;
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  const int r = warp_tot[warp] + inc - v;
  __syncthreads();
  return r;
}

constexpr int PH_THREADS = 1024;
constexpr int PH_PER = 4;                            // consecutive tokens per thread and pass

struct FinalizeArgs {        // preference of the layer from the tensor-core kernel's partials
  const float* colpart;      // [pass-B segment][statistics warp][G][2]
  const int32_t* pair_seg;   // [pairs + 1]
  const float* hrow;         // [pair][128] or unused
  double* headsum;           // [req][H_q][2] scratch
  uint32_t* fin_arrivals;    // [req], zero at rest
  double* dH; double* dV; double* dP;
  int32_t* status;
  int units;                 // extra CTAs per (KV head, request): G (0 = none)
  int use_hrow, rows, Hq;
  double inv_tau1, inv_tau2;
};

// H_h = -ln2 * sum p*log2(p), V_h = sum_j Var_i of one query head; the CTA that finishes a
// request's last head averages over the heads and sets P = H^(1/tau1) * V^(1/tau2) (Eq. 4-6).
// All sums run in a fixed order in double precision.
__device__ void finalize_head(const FinalizeArgs& F, int req, int g, int hl, int layer, int L, int Hkv) {
  __shared__ double red[2][PH_THREADS / 32];
  __shared__ int s_last;
  const int G = F.Hq / Hkv;
  const int pair = req * Hkv + g;
  double a = 0.0, b = 0.0;
  const int s_lo = F.pair_seg[pair] * kScoreWarps, s_hi = F.pair_seg[pair + 1] * kScoreWarps;
  for (int sg = s_lo + (int)threadIdx.x; sg < s_hi; sg += PH_THREADS) {
    const float2 p = __ldcg(reinterpret_cast<const float2*>(F.colpart + ((size_t)sg * G + hl) * 2));
    a += (double)p.x;
    b += (double)p.y;
  }
  if (F.use_hrow) {
    a = 0.0;
    for (int r = hl + (int)threadIdx.x * G; r < F.rows; r += PH_THREADS * G)
      a += (double)__ldcg(&F.hrow[(size_t)pair * 128 + r]);
  }
  a = warp_sum_f64(a);
  b = warp_sum_f64(b);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = a; red[1][threadIdx.x >> 5] = b; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ha = 0.0, vb = 0.0;
    for (int w = 0; w < PH_THREADS / 32; ++w) { ha += red[0][w]; vb += red[1][w]; }
    double* hs = F.headsum + ((size_t)req * F.Hq + g * G + hl) * 2;
    hs[0] = -0.6931471805599453 * ha;
    hs[1] = vb;
    __threadfence();
    const uint32_t old = atomicAdd(&F.fin_arrivals[req], 1u);
    s_last = (old + 1u == (uint32_t)F.Hq) ? 1 : 0;
    if (s_last) {
      __threadfence();
      F.fin_arrivals[req] = 0;
      double H = 0.0, V = 0.0;
      for (int h = 0; h < F.Hq; ++h) {
        H += __ldcg(&F.headsum[((size_t)req * F.Hq + h) * 2]);
        V += __ldcg(&F.headsum[((size_t)req * F.Hq + h) * 2 + 1]);
      }
      H /= (double)F.Hq;
      V /= (double)F.Hq;
      const double P = pow(H, F.inv_tau1) * pow(V, F.inv_tau2);
      F.dH[(size_t)req * L + layer] = H;
      F.dV[(size_t)req * L + layer] = V;
      F.dP[(size_t)req * L + layer] = P;
      if (!(P >= 0.0) || isinf(P)) raise_status(F.status, CAKE_ERR_NONFINITE);
    }
  }
}

// One CTA per (split of a request's tokens, KV head, request); a thread owns PH_PER consecutive
// tokens per pass.  fresh[g][t] = pool(raw[g][.]) over the request's non-window tokens, +inf on
// the window (Section 4.3); with do_pool = 0 the pooled values are already in `fresh`.  The
// bucket histogram of the (request, head) is accumulated in `hist`; the CTA that adds the last
// split turns it into the list's bucket offsets.  R = pool_kernel / 2 when that is at most 3,
// else -1 (any kernel size, one global read per tap).  CTAs with blockIdx.x >= n_split finalise
// the layer's preference (tensor-core path).  The grid is small on purpose: it runs on the few
// SMs the score kernel of the next layer leaves free.
template <int R>
__global__ void __launch_bounds__(PH_THREADS)
pool_hist(const float* __restrict__ raw, float* __restrict__ fresh, const ReqInfo* __restrict__ reqs,
          uint32_t* __restrict__ hist, uint32_t* __restrict__ arrivals, int32_t* __restrict__ prefix,
          int n_split, int layer, int L, int Hkv, int64_t T, int kp, int mode, int do_pool,
          const FinalizeArgs F) {
  const int g = blockIdx.y, req = blockIdx.z;
  if ((int)blockIdx.x >= n_split) {
    finalize_head(F, req, g, (int)blockIdx.x - n_split, layer, L, Hkv);
    return;
  }
  __shared__ uint32_t sh[kBins];
  __shared__ int warp_tot[32];
  __shared__ int s_total, s_last;
  const ReqInfo rq = reqs[req];
  if ((int)blockIdx.x >= rq.nsplit) return;
  const int pair = req * Hkv + g;
  for (int b = threadIdx.x; b < kBins; b += PH_THREADS) sh[b] = 0;
  __syncthreads();
  const float* src = raw + (size_t)g * T + rq.cu;
  float* dst = fresh + (size_t)g * T + rq.cu;
  const int t0 = (int)blockIdx.x * rq.span, t1 = min(rq.N, t0 + rq.span);
  for (int j0 = t0 + (int)threadIdx.x * PH_PER; j0 < t1; j0 += PH_THREADS * PH_PER) {
    float out[PH_PER];
    if (!do_pool) {
#pragma unroll
      for (int e = 0; e < PH_PER; ++e) out[e] = j0 + e < rq.n ? dst[j0 + e] : CUDART_INF_F;
    } else if (R >= 0) {
      const float pad = mode == CAKE_POOL_MAX ? -CUDART_INF_F : 0.f;
      float w[PH_PER + 2 * (R >= 0 ? R : 0)];
#pragma unroll
      for (int x = 0; x < PH_PER + 2 * R; ++x) {
        const int j = j0 - R + x;
        w[x] = (j >= 0 && j < rq.n) ? src[j] : pad;
      }
#pragma unroll
      for (int e = 0; e < PH_PER; ++e) {
        float m = w[e];
#pragma unroll
        for (int x = 1; x <= 2 * R; ++x) m = mode == CAKE_POOL_MAX ? fmaxf(m, w[e + x]) : m + w[e + x];
        out[e] = mode == CAKE_POOL_MAX ? m : m / (float)kp;
      }
    } else {
      const int r = kp >> 1;
#pragma unroll 1
      for (int e = 0; e < PH_PER; ++e) {
        const int j = j0 + e;
        float m = 0.f;
        if (j < rq.n) {
          const int a = max(0, j - r), b = min(rq.n, j + r + 1);
          m = src[a];
          for (int x = a + 1; x < b; ++x) m = mode == CAKE_POOL_MAX ? fmaxf(m, src[x]) : m + src[x];
          if (mode != CAKE_POOL_MAX) m /= (float)kp;
        }
        out[e] = m;
      }
    }
    // write back and count buckets; neighbours often share a bucket, so runs are counted once
    int run_bin = -1;
    uint32_t run_len = 0;
#pragma unroll
    for (int e = 0; e < PH_PER; ++e) {
      const int j = j0 + e;
      if (j < t1) {
        if (j >= rq.n) {
          dst[j] = CUDART_INF_F;
        } else {
          if (do_pool) dst[j] = out[e];
          const int q = bucket_of(ordered_key(out[e]));
          if (q != run_bin) {
            if (run_len) atomicAdd(&sh[run_bin], run_len);
            run_bin = q;
            run_len = 0;
          }
          ++run_len;
        }
      }
    }
    if (run_len) atomicAdd(&sh[run_bin], run_len);
  }
  __syncthreads();
  uint32_t* gh = hist + (size_t)pair * kBins;
  for (int b = threadIdx.x; b < kBins; b += PH_THREADS)
    if (sh[b]) atomicAdd(&gh[b], sh[b]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t old = atomicAdd(&arrivals[pair], 1u);
    s_last = (old + 1u == (uint32_t)rq.nsplit) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // bucket offsets of the new list: prefix[i] = elements in buckets before i
  int32_t* pf = prefix + (((size_t)req * L + layer) * Hkv + g) * (kBins + 1);
  constexpr int PER = kBins / PH_THREADS;
  int cnt[PER], sum = 0;
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    cnt[e] = (int)__ldcg(&gh[threadIdx.x * PER + e]);
    sum += cnt[e];
  }
  int run = block_excl_scan(sum, warp_tot, &s_total);
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    pf[threadIdx.x * PER + e] = run;
    run += cnt[e];
    gh[threadIdx.x * PER + e] = 0;              // ready for the next layer
  }
  if (threadIdx.x == PH_THREADS - 1) pf[kBins] = run;
  if (threadIdx.x == 0) arrivals[pair] = 0;
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
                                 int32_t* __restrict__ status, int stage, int L, int64_t seats,
                                 int alloc_mode, double slope) {
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
    // what the split is proportional to: the preference (Eq. 7 / Eq. 9), or one of the fixed
    // patterns of the paper's allocation ablation (Section 5.3)
    double p = dP[(size_t)req * L + l];
    if (alloc_mode == CAKE_ALLOC_UNIFORM) p = 1.0;
    else if (alloc_mode == CAKE_ALLOC_PYRAMID) p = L > 1 ? 1.0 + slope * (double)(L - 1 - 2 * l) / (double)(L - 1) : 1.0;
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
constexpr int EV_THREADS = 256;
constexpr int kTieCap = 2048;

struct EvictSmem {
  uint32_t hist[1024];
  int32_t ties[kTieCap];
  int warp_tot[32];
  int total;
  uint32_t sel_digit, sel_rem, sel_cnt;
  int32_t tie_count, pos_cut;
};

// Among `cnt` entries (all in one bucket), finds the digit (10 bits at `shift`) that holds the
// krem-th largest key among the entries whose bits above shift+10 equal `prefix_bits`.
__device__ inline void radix_digit(const uint2* __restrict__ e, int cnt, uint32_t mask,
                                   uint32_t prefix_bits, int shift, uint32_t krem, EvictSmem& S) {
  for (int b = threadIdx.x; b < 1024; b += blockDim.x) S.hist[b] = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    const uint32_t key = __ldcg(&e[i]).x;
    if ((key & mask) == prefix_bits) atomicAdd(&S.hist[(key >> shift) & 1023u], 1u);
  }
  __syncthreads();
  // digits from the top: thread t owns digits 1023-4t .. 1020-4t
  const int per = 1024 / blockDim.x;
  int mine = 0;
  for (int q = 0; q < per; ++q) mine += (int)S.hist[1023 - (threadIdx.x * per + q)];
  int above = block_excl_scan(mine, S.warp_tot, &S.total);
  for (int q = 0; q < per; ++q) {
    const int dg = 1023 - (threadIdx.x * per + q);
    const int h = (int)S.hist[dg];
    if ((uint32_t)above < krem && (uint32_t)(above + h) >= krem) {
      S.sel_digit = (uint32_t)dg;
      S.sel_rem = krem - (uint32_t)above;
      S.sel_cnt = (uint32_t)h;
    }
    above += h;
  }
  __syncthreads();
}

// Moves the threshold of one list to the budget b: the retained set becomes the first b entries
// in the order (indicator descending, position ascending)  (Section 4.2 EVICT, Eq. 12).
// `hint` >= 0 is the list's previous threshold bucket: budgets only shrink, so the new one is
// that bucket or one shortly before it.
__device__ void set_threshold(const int32_t* __restrict__ pf, const uint2* __restrict__ list, int b,
                              int hint, ListState* __restrict__ out, EvictSmem& S) {
  if (b <= 0) {
    if (threadIdx.x == 0) *out = ListState{-1, 0xFFFFFFFFu, -1, 0};
    return;
  }
  // threshold bucket d: first bucket with prefix[d+1] >= b
  if (threadIdx.x == 0) S.total = -1;
  __syncthreads();
  if (hint >= 0) {
    const int q = hint - (int)threadIdx.x;
    if (q >= 0 && __ldcg(&pf[q]) < b && __ldcg(&pf[q + 1]) >= b) S.total = q;
  }
  __syncthreads();
  if (S.total < 0) {
    __syncthreads();
    int less = 0;
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) less += __ldcg(&pf[i + 1]) < b ? 1 : 0;
    block_excl_scan(less, S.warp_tot, &S.total);
  }
  const int d = S.total;
  __syncthreads();
  if (d >= kBins) {                                  // b exceeds the stored entries: keep all
    if (threadIdx.x == 0) *out = ListState{kBins - 1, 0u, 0x7FFFFFFF, __ldcg(&pf[kBins])};
    return;
  }
  const int start = __ldcg(&pf[d]), cnt = __ldcg(&pf[d + 1]) - start;
  const uint32_t rem = (uint32_t)(b - start);
  if ((int)rem >= cnt) {
    if (threadIdx.x == 0) *out = ListState{d, 0u, 0x7FFFFFFF, b};
    return;
  }
  const uint2* e = list + start;
  constexpr int low = 32 - kBinBits;                 // key bits below the bucket bits (20)
  radix_digit(e, cnt, 0u, 0u, low - 10, rem, S);
  uint32_t pre = S.sel_digit << (low - 10);
  uint32_t krem = S.sel_rem;
  __syncthreads();
  radix_digit(e, cnt, 1023u << (low - 10), pre, 0, krem, S);
  pre |= S.sel_digit;
  const uint32_t need_eq = S.sel_rem, n_eq = S.sel_cnt;
  __syncthreads();
  // full key of the threshold: bucket bits + the 20 selected bits
  const uint32_t thr = ((uint32_t)(kBins - 1 - d) << low) | pre;
  int32_t pos_cut = 0x7FFFFFFF;
  if (need_eq < n_eq) {
    // ties at the threshold: the need_eq lowest positions win
    if (threadIdx.x == 0) { S.tie_count = 0; S.pos_cut = 0x7FFFFFFF; }
    __syncthreads();
    if (n_eq <= (uint32_t)kTieCap) {
      for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
        const uint2 v = __ldcg(&e[i]);
        if (v.x == thr) S.ties[atomicAdd(&S.tie_count, 1)] = (int32_t)v.y;
      }
      __syncthreads();
      for (int i = threadIdx.x; i < (int)n_eq; i += blockDim.x) {
        const int32_t p = S.ties[i];
        uint32_t r = 0;
        for (int o = 0; o < (int)n_eq; ++o) r += S.ties[o] < p ? 1u : 0u;
        if (r == need_eq - 1) S.pos_cut = p;
      }
      __syncthreads();
    } else {
      // many ties: bisect the position (positions are distinct)
      int lo = 0, hi = 0x7FFFFFFF;                   // smallest cut with count(pos <= cut) >= need_eq
      while (lo < hi) {
        const int mid = lo + ((hi - lo) >> 1);
        int c = 0;
        for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
          const uint2 v = __ldcg(&e[i]);
          c += (v.x == thr && (int32_t)v.y <= mid) ? 1 : 0;
        }
        block_excl_scan(c, S.warp_tot, &S.total);
        const int tot = S.total;
        __syncthreads();
        if ((uint32_t)tot >= need_eq) hi = mid; else lo = mid + 1;
      }
      if (threadIdx.x == 0) S.pos_cut = lo;
      __syncthreads();
    }
    pos_cut = S.pos_cut;
  }
  if (threadIdx.x == 0) *out = ListState{d, thr, pos_cut, b};
}

struct EvictArgs {
  const float* fresh;
  uint2* lists;
  const int32_t* prefix_all;
  ListState* states;
  uint32_t* fill;          // [pairs][kBins], zero between launches
  uint32_t* arrivals;      // [pairs]
  const ReqInfo* reqs;
  const int32_t* cur;      // budgets of this stage
  int stage, L, Hkv;
  int64_t T;
};

constexpr int SC_THREADS = 1024;
constexpr int SC_PER = 4;

// Newest layer of stage `stage`: one CTA per (split of a request's tokens, KV head, request)
// scatters the pooled indicators into bucket order.  Only the buckets the layer's budget can
// ever reach are stored (the budget never grows again, Proposition 1).  The CTA that completes
// a list sets its threshold.
__global__ void __launch_bounds__(SC_THREADS)
scatter_new(const EvictArgs A) {
  __shared__ EvictSmem S;
  __shared__ uint32_t s_cnt[kBins];
  __shared__ uint32_t s_base[kBins];
  __shared__ int s_last;
  const int g = blockIdx.y, req = blockIdx.z;
  const ReqInfo rq = A.reqs[req];
  if ((int)blockIdx.x >= rq.nsplit) return;
  const int pair = req * A.Hkv + g;
  const size_t lid = ((size_t)req * A.L + A.stage) * A.Hkv + g;
  const int32_t* pf = A.prefix_all + lid * (kBins + 1);
  uint2* list = A.lists + rq.list_off + ((size_t)A.stage * A.Hkv + g) * rq.n;
  const int b = min(A.cur[(size_t)req * A.L + A.stage], rq.n);
  // last bucket worth storing
  int less = 0;
  for (int i = threadIdx.x; i < kBins; i += SC_THREADS) {
    less += __ldcg(&pf[i + 1]) < b ? 1 : 0;
    s_cnt[i] = 0;
  }
  block_excl_scan(less, S.warp_tot, &S.total);
  const int d_last = b > 0 ? min(S.total, kBins - 1) : -1;
  __syncthreads();
  const float* src = A.fresh + (size_t)g * A.T + rq.cu;
  const int t0 = (int)blockIdx.x * rq.span, t1 = min(rq.n, t0 + rq.span);
  // pass 1: count this split's entries per bucket (runs of equal buckets at once)
  for (int j0 = t0 + (int)threadIdx.x * SC_PER; j0 < t1; j0 += SC_THREADS * SC_PER) {
    int run_bin = -1;
    uint32_t run_len = 0;
#pragma unroll
    for (int e = 0; e < SC_PER; ++e) {
      int q = -1;
      if (j0 + e < t1) {
        q = bucket_of(ordered_key(src[j0 + e]));
        if (q > d_last) q = -1;
      }
      if (q != run_bin) {
        if (run_len && run_bin >= 0) atomicAdd(&s_cnt[run_bin], run_len);
        run_bin = q;
        run_len = 0;
      }
      ++run_len;
    }
    if (run_len && run_bin >= 0) atomicAdd(&s_cnt[run_bin], run_len);
  }
  __syncthreads();
  // reserve this split's range inside every bucket of the list
  uint32_t* gf = A.fill + (size_t)pair * kBins;
  for (int q = threadIdx.x; q < kBins; q += SC_THREADS) {
    const uint32_t c = s_cnt[q];
    if (c) s_base[q] = (uint32_t)__ldcg(&pf[q]) + atomicAdd(&gf[q], c);
    s_cnt[q] = 0;
  }
  __syncthreads();
  // pass 2: place the entries
  for (int j0 = t0 + (int)threadIdx.x * SC_PER; j0 < t1; j0 += SC_THREADS * SC_PER) {
    uint32_t key[SC_PER];
    int bk[SC_PER];
#pragma unroll
    for (int e = 0; e < SC_PER; ++e) {
      bk[e] = -1;
      if (j0 + e < t1) {
        key[e] = ordered_key(src[j0 + e]);
        const int q = bucket_of(key[e]);
        if (q <= d_last) bk[e] = q;
      }
    }
    int run_bin = -1;
    uint32_t run_off = 0;
#pragma unroll
    for (int e = 0; e < SC_PER; ++e) {
      if (bk[e] != run_bin) {
        run_bin = bk[e];
        if (run_bin >= 0) {
          uint32_t len = 1;
#pragma unroll
          for (int f = e + 1; f < SC_PER; ++f) {
            if (bk[f] != run_bin) break;
            ++len;
          }
          run_off = s_base[run_bin] + atomicAdd(&s_cnt[run_bin], len);
        }
      }
      if (run_bin >= 0) list[run_off++] = make_uint2(key[e], (uint32_t)(j0 + e));
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t old = atomicAdd(&A.arrivals[pair], 1u);
    s_last = (old + 1u == (uint32_t)rq.nsplit) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int q = threadIdx.x; q < kBins; q += SC_THREADS) gf[q] = 0;       // ready for the next stage
  if (threadIdx.x == 0) A.arrivals[pair] = 0;
  set_threshold(pf, list, b, -1, &A.states[lid], S);
}

// Older layers of stage `stage`: one CTA per (KV head, layer < stage, request) moves the list's
// threshold to its new budget.
__global__ void __launch_bounds__(EV_THREADS)
thresholds_old(const EvictArgs A) {
  __shared__ EvictSmem S;
  const int g = blockIdx.x, layer = blockIdx.y, req = blockIdx.z;
  const ReqInfo rq = A.reqs[req];
  const size_t lid = ((size_t)req * A.L + layer) * A.Hkv + g;
  const ListState old = A.states[lid];
  // a list never grows again (Proposition 1): entries beyond its earlier budget were not stored
  const int b = min(min(A.cur[(size_t)req * A.L + layer], rq.n), old.kept);
  if (old.kept == b) return;                                   // budget unchanged
  set_threshold(A.prefix_all + lid * (kBins + 1),
                A.lists + rq.list_off + ((size_t)layer * A.Hkv + g) * rq.n, b, old.bucket,
                &A.states[lid], S);
}

}  // namespace

// Pooling + bucket histogram of layer `layer`; with `finalize` also the layer's preference
// (tensor-core path: extra CTAs of the same launch; SIMT path: its own small kernel).
int32_t launch_pool(cake_ctx* ctx, int32_t layer, bool do_pool, bool finalize, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  if (finalize && !ctx->use_tc) {
    finalize_layer<<<ctx->n_req, 128, 0, st>>>(ctx->d_colpart[layer & 1], ctx->d_req, ctx->d_H, ctx->d_V,
                                                ctx->d_P, ctx->d_status, layer, c.n_layers,
                                                c.n_q_heads, c.n_kv_heads, 1.0 / (double)c.tau1,
                                                1.0 / (double)c.tau2);
    count_launch();
  }
  FinalizeArgs F;
  memset(&F, 0, sizeof(F));
  F.Hq = c.n_q_heads;
  if (finalize && ctx->use_tc) {
    F.colpart = ctx->d_colpart[layer & 1];
    F.pair_seg = ctx->d_tc_index + (ctx->n_req * c.n_kv_heads + 1);
    F.hrow = ctx->d_hrow[layer & 1];
    F.headsum = ctx->d_headsum;
    F.fin_arrivals = ctx->d_arrivals + ctx->max_pairs;
    F.dH = ctx->d_H; F.dV = ctx->d_V; F.dP = ctx->d_P;
    F.status = ctx->d_status;
    F.units = c.n_q_heads / c.n_kv_heads;
    F.use_hrow = ctx->hhead_from_rows ? 1 : 0;
    F.rows = ctx->rows;
    F.inv_tau1 = 1.0 / (double)c.tau1;
    F.inv_tau2 = 1.0 / (double)c.tau2;
  }
  const dim3 grid((unsigned)(ctx->n_split + F.units), c.n_kv_heads, ctx->n_req);
  const int r = c.pool_kernel / 2;
#define CAKE_POOL_LAUNCH(RR)                                                                     \
  pool_hist<RR><<<grid, PH_THREADS, 0, st>>>(ctx->d_raw[layer & 1], ctx->d_fresh[layer & 1], ctx->d_req,    \
                                             ctx->d_hist, ctx->d_arrivals + ctx->max_pairs + c.max_requests, ctx->d_prefix, \
                                             ctx->n_split, layer, c.n_layers, c.n_kv_heads,      \
                                             ctx->total_tokens, c.pool_kernel, c.pool_mode,      \
                                             do_pool ? 1 : 0, F)
  switch (r) {
    case 0: CAKE_POOL_LAUNCH(0); break;
    case 1: CAKE_POOL_LAUNCH(1); break;
    case 2: CAKE_POOL_LAUNCH(2); break;
    case 3: CAKE_POOL_LAUNCH(3); break;
    default: CAKE_POOL_LAUNCH(-1); break;
  }
#undef CAKE_POOL_LAUNCH
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_allocate(cake_ctx* ctx, int32_t stage, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  allocate_budgets<<<ctx->n_req, 32, 0, st>>>(ctx->d_P, ctx->d_req, ctx->d_budget[(stage + 1) & 1],
                                              ctx->d_budget[stage & 1], ctx->d_status, stage,
                                              c.n_layers, ctx->sel_budget, c.alloc_mode,
                                              (double)c.pyramid_slope);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_evict(cake_ctx* ctx, int32_t stage, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  EvictArgs A;
  A.fresh = ctx->d_fresh[stage & 1];
  A.lists = ctx->d_lists;
  A.prefix_all = ctx->d_prefix;
  A.states = ctx->d_lstate;
  A.fill = ctx->d_fill;
  A.arrivals = ctx->d_arrivals;
  A.reqs = ctx->d_req;
  A.cur = ctx->d_budget[stage & 1];
  A.stage = stage; A.L = c.n_layers; A.Hkv = c.n_kv_heads;
  A.T = ctx->total_tokens;
  // The older layers' lists and the newest layer's list share nothing: the two kernels run side
  // by side, the thresholds on a second internal stream that forks from and joins `st`.
  if (stage > 0) {
    CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_fork, st));
    CAKE_CUDA_TRY(cudaStreamWaitEvent(ctx->side2, ctx->ev_fork, 0));
    thresholds_old<<<dim3(c.n_kv_heads, stage, ctx->n_req), EV_THREADS, 0, ctx->side2>>>(A);
    count_launch();
    CAKE_CUDA_TRY(cudaEventRecord(ctx->ev_join, ctx->side2));
  }
  scatter_new<<<dim3(ctx->n_split, c.n_kv_heads, ctx->n_req), SC_THREADS, 0, st>>>(A);
  count_launch();
  if (stage > 0) CAKE_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev_join, 0));
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
