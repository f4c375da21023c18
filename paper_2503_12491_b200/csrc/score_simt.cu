// Window-score kernels, plain fp32 SIMT version.
//
// Serves fp32 inputs (and any shape the tensor-core path does not take).  Two
// passes over the keys of every (request, KV head):
//   pass A  row statistics  -> base-2 log-sum-exp of every window row over its
//           visible keys (softmax denominator, Section 2 Eq. 2)
//   pass B  column statistics of the normalised probabilities of the
//           non-window keys -> raw indicator (Eq. 11), per-head sums for the
//           dispersion (Eq. 4) and the shift (Eq. 5)
// Both passes recompute q.k on chip; the S_w x N score matrix never leaves the SM.
#include "cake_internal.cuh"

#include <math_constants.h>

namespace cake {
namespace {

constexpr int TK = kSimtTileKeys;   // 64 keys per tile
constexpr int S_STRIDE = 72;        // padded row stride of the score tile
constexpr int NT = kSimtThreads;    // 256 threads

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ static void unpack(const uint4& v, float* o) {
    o[0] = __uint_as_float(v.x); o[1] = __uint_as_float(v.y);
    o[2] = __uint_as_float(v.z); o[3] = __uint_as_float(v.w);
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void unpack(const uint4& v, float* o) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = __uint_as_float(w[i] << 16);
      o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

struct SmemLayout {
  float* q;     // [rows8][d]
  float* k;     // [TK][d+4]
  float* s;     // [rows8][S_STRIDE]
  float* aux;   // [2*kMaxRows]
};

__device__ inline SmemLayout carve(float* base, int rows8, int d) {
  SmemLayout L;
  L.q = base;
  L.k = L.q + rows8 * d;
  L.s = L.k + TK * (d + 4);
  L.aux = L.s + rows8 * S_STRIDE;
  return L;
}

inline size_t smem_bytes(int rows, int d) {
  int rows8 = (rows + 7) / 8 * 8;
  return sizeof(float) * ((size_t)rows8 * d + (size_t)TK * (d + 4) + (size_t)rows8 * S_STRIDE +
                          2 * kMaxRows);
}

template <typename T>
__device__ inline void load_q(const T* q_grp, float* qs, int rows, int rows8, int d) {
  constexpr int E = Vec16<T>::kElems;
  const int nvec = rows * d / E;
  const uint4* src = reinterpret_cast<const uint4*>(q_grp);
  for (int v = threadIdx.x; v < nvec; v += NT) {
    float o[E];
    Vec16<T>::unpack(src[v], o);
#pragma unroll
    for (int e = 0; e < E; ++e) qs[v * E + e] = o[e];
  }
  for (int idx = rows * d + threadIdx.x; idx < rows8 * d; idx += NT) qs[idx] = 0.f;
}

template <typename T>
__device__ inline void load_k_tile(const T* k_rows, float* ks, int count, int d) {
  constexpr int E = Vec16<T>::kElems;
  const int vpr = d / E;                 // 16-byte vectors per row
  const int kstride = d + 4;
  for (int v = threadIdx.x; v < TK * vpr; v += NT) {
    const int row = v / vpr, cv = v - row * vpr;
    float o[E];
    if (row < count) {
      uint4 raw = reinterpret_cast<const uint4*>(k_rows + (size_t)row * d)[cv];
      Vec16<T>::unpack(raw, o);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) o[e] = 0.f;
    }
    float* dst = ks + row * kstride + cv * E;
#pragma unroll
    for (int e = 0; e < E; e += 4)
      *reinterpret_cast<float4*>(dst + e) = make_float4(o[e], o[e + 1], o[e + 2], o[e + 3]);
  }
}

// S[row][key] = (q_row . k_key) * scale2 for the 64-key tile; thread tile 8 rows x 4 keys.
__device__ inline void tile_scores(const SmemLayout& L, int rows8, int d, float scale2) {
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int kstride = d + 4;
  for (int rb = ty * 8; rb < rows8; rb += 128) {
    float acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
    for (int c0 = 0; c0 < d; c0 += 4) {
      float4 kv[4];
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
        kv[kk] = *reinterpret_cast<const float4*>(L.k + (tx + 16 * kk) * kstride + c0);
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const float4 qv = *reinterpret_cast<const float4*>(L.q + (rb + r) * d + c0);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          acc[r][kk] = fmaf(qv.x, kv[kk].x, acc[r][kk]);
          acc[r][kk] = fmaf(qv.y, kv[kk].y, acc[r][kk]);
          acc[r][kk] = fmaf(qv.z, kv[kk].z, acc[r][kk]);
          acc[r][kk] = fmaf(qv.w, kv[kk].w, acc[r][kk]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) L.s[(rb + r) * S_STRIDE + tx + 16 * kk] = acc[r][kk] * scale2;
  }
}

__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------- pass A
template <typename T>
__global__ void __launch_bounds__(NT)
score_rowstats_simt(const T* __restrict__ q_win, const T* __restrict__ k,
                    const ReqInfo* __restrict__ reqs, const ScoreUnit* __restrict__ units,
                    float2* __restrict__ rowpart, int Hq, int Hkv, int Sw, int d, int64_t T_tokens,
                    float scale2) {
  extern __shared__ __align__(16) float smem[];
  const int G = Hq / Hkv, rows = G * Sw, rows8 = (rows + 7) / 8 * 8;
  const SmemLayout L = carve(smem, rows8, d);
  const ScoreUnit u = units[blockIdx.x];
  const int g = blockIdx.y;
  const ReqInfo rq = reqs[u.req];
  float* run_m = L.aux;
  float* run_z = L.aux + kMaxRows;
  for (int r = threadIdx.x; r < rows; r += NT) { run_m[r] = -CUDART_INF_F; run_z[r] = 0.f; }
  load_q(q_win + ((size_t)u.req * Hq + (size_t)g * G) * Sw * d, L.q, rows, rows8, d);
  const T* kbase = k + ((size_t)g * T_tokens + rq.cu) * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t0 = 0; t0 < u.nkeys; t0 += TK) {
    const int key0 = u.key0 + t0;
    const int count = min(TK, u.nkeys - t0);
    __syncthreads();
    load_k_tile(kbase + (size_t)key0 * d, L.k, count, d);
    __syncthreads();
    tile_scores(L, rows8, d, scale2);
    __syncthreads();
    for (int row = warp; row < rows; row += NT / 32) {
      const int i = row % Sw;
      const int last = rq.n + i;                       // last key row i may see
      const int j0 = key0 + lane, j1 = j0 + 32;
      const bool ok0 = lane < count && j0 <= last;
      const bool ok1 = lane + 32 < count && j1 <= last;
      const float v0 = ok0 ? L.s[row * S_STRIDE + lane] : -CUDART_INF_F;
      const float v1 = ok1 ? L.s[row * S_STRIDE + lane + 32] : -CUDART_INF_F;
      const float m = warp_max(fmaxf(v0, v1));
      if (m == -CUDART_INF_F) continue;
      float e = (ok0 ? exp2f(v0 - m) : 0.f) + (ok1 ? exp2f(v1 - m) : 0.f);
      e = warp_sum(e);
      if (lane == 0) {
        const float mo = run_m[row], zo = run_z[row];
        const float mn = fmaxf(mo, m);
        run_z[row] = zo * exp2f(mo - mn) + e * exp2f(m - mn);   // exp2f(-inf) = 0 on first tile
        run_m[row] = mn;
      }
    }
  }
  __syncthreads();
  float2* out = rowpart + ((size_t)blockIdx.x * Hkv + g) * rows;
  for (int r = threadIdx.x; r < rows; r += NT) out[r] = make_float2(run_m[r], run_z[r]);
}

__global__ void rowstats_combine(const float2* __restrict__ rowpart,
                                 const ReqInfo* __restrict__ reqs, float* __restrict__ lse2,
                                 int Hkv, int rows) {
  const int req = blockIdx.x, g = blockIdx.y, row = threadIdx.x;
  if (row >= rows) return;
  const ReqInfo rq = reqs[req];
  float m = -CUDART_INF_F, z = 0.f;
  for (int u = rq.unit0; u < rq.unit0 + rq.nunits; ++u) {
    const float2 p = rowpart[((size_t)u * Hkv + g) * rows + row];
    if (p.x == -CUDART_INF_F) continue;
    const float mn = fmaxf(m, p.x);
    z = z * exp2f(m - mn) + p.y * exp2f(p.x - mn);
    m = mn;
  }
  lse2[((size_t)req * Hkv + g) * rows + row] = m + log2f(z);
}

__global__ void lse_to_base2(const float* __restrict__ lse, float* __restrict__ lse2, int64_t count) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) lse2[i] = lse[i] * 1.4426950408889634f;
}

// ---------------------------------------------------------------- pass B
template <typename T>
__global__ void __launch_bounds__(NT)
score_colstats_simt(const T* __restrict__ q_win, const T* __restrict__ k,
                    const ReqInfo* __restrict__ reqs, const ScoreUnit* __restrict__ units,
                    const float* __restrict__ lse2, float* __restrict__ raw,
                    float* __restrict__ colpart, int Hq, int Hkv, int Sw, int d, int64_t T_tokens,
                    float scale2, float gamma, int ddof, int ind_mode) {
  extern __shared__ __align__(16) float smem[];
  const int G = Hq / Hkv, rows = G * Sw, rows8 = (rows + 7) / 8 * 8;
  const SmemLayout L = carve(smem, rows8, d);
  const ScoreUnit u = units[blockIdx.x];
  const int g = blockIdx.y;
  const ReqInfo rq = reqs[u.req];
  float* lse_s = L.aux;
  for (int r = threadIdx.x; r < rows; r += NT)
    lse_s[r] = lse2[((size_t)u.req * Hkv + g) * rows + r];
  float hs[8], vacc[8];
#pragma unroll
  for (int h = 0; h < 8; ++h) { hs[h] = 0.f; vacc[h] = 0.f; }
  const int nkeys = min(u.nkeys, rq.n - u.key0);       // only non-window keys
  if (nkeys > 0) load_q(q_win + ((size_t)u.req * Hq + (size_t)g * G) * Sw * d, L.q, rows, rows8, d);
  const T* kbase = k + ((size_t)g * T_tokens + rq.cu) * d;
  const int key_l = threadIdx.x >> 2, q4 = threadIdx.x & 3;
  const float inv_sw = 1.f / (float)Sw, inv_g = 1.f / (float)G;
  const float bessel = ddof ? (float)Sw / (float)(Sw - 1) : 1.f;
  for (int t0 = 0; t0 < nkeys; t0 += TK) {
    const int key0 = u.key0 + t0;
    const int count = min(TK, nkeys - t0);
    __syncthreads();
    load_k_tile(kbase + (size_t)key0 * d, L.k, count, d);
    __syncthreads();
    tile_scores(L, rows8, d, scale2);
    __syncthreads();
    float s1[8], s2[8], a1 = 0.f, a2 = 0.f;
#pragma unroll
    for (int h = 0; h < 8; ++h) { s1[h] = 0.f; s2[h] = 0.f; }
    const bool valid = key_l < count;
    if (valid) {
      for (int i = q4; i < Sw; i += 4) {
        float a = 0.f;
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          if (h < G) {
            const int r = h * Sw + i;
            const float t = L.s[r * S_STRIDE + key_l] - lse_s[r];
            const float p = exp2f(t);
            hs[h] = fmaf(p, t, hs[h]);
            s1[h] += p;
            s2[h] = fmaf(p, p, s2[h]);
            a += p;
          }
        }
        a *= inv_g;
        a1 += a;
        a2 = fmaf(a, a, a2);
      }
    }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      a1 += __shfl_xor_sync(0xffffffffu, a1, o);
      a2 += __shfl_xor_sync(0xffffffffu, a2, o);
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        if (h < G) {
          s1[h] += __shfl_xor_sync(0xffffffffu, s1[h], o);
          s2[h] += __shfl_xor_sync(0xffffffffu, s2[h], o);
        }
      }
    }
    if (valid && q4 == 0) {
      const float mean = a1 * inv_sw;
      const float var = fmaxf(a2 * inv_sw - mean * mean, 0.f) * bessel;
      raw[(size_t)g * T_tokens + rq.cu + key0 + key_l] = combine_indicator(ind_mode, gamma, mean, var, (float)Sw);
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        if (h < G) {
          const float mh = s1[h] * inv_sw;
          vacc[h] += fmaxf(s2[h] * inv_sw - mh * mh, 0.f) * bessel;
        }
      }
    }
  }
  // deterministic block reduction of hs / vacc: warp shuffle tree, then warp 0 in order
  __syncthreads();
  float* red = L.s;                       // reuse: [8 warps][16]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int h = 0; h < 8; ++h) {
    const float a = warp_sum(hs[h]);
    const float b = warp_sum(vacc[h]);
    if (lane == 0) { red[warp * 16 + h] = a; red[warp * 16 + 8 + h] = b; }
  }
  __syncthreads();
  if (threadIdx.x < 2 * G) {
    const int h = threadIdx.x >> 1, which = threadIdx.x & 1;
    float acc = 0.f;
    for (int w = 0; w < NT / 32; ++w) acc += red[w * 16 + which * 8 + h];
    colpart[(((size_t)blockIdx.x * Hkv + g) * G + h) * 2 + which] = acc;
  }
}

template <typename T>
int32_t run(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k, const float* lse,
            cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int rows = ctx->rows;
  const size_t smem = smem_bytes(rows, c.head_dim);
  const float scale2 = 1.4426950408889634f / sqrtf((float)c.head_dim);
  static PerDeviceOnce attr[2];
  const int ti = sizeof(T) == 4 ? 0 : 1;
  if (attr[ti].need(ctx->device)) {
    CAKE_CUDA_TRY(cudaFuncSetAttribute(score_rowstats_simt<T>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    CAKE_CUDA_TRY(cudaFuncSetAttribute(score_colstats_simt<T>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr[ti].mark(ctx->device);
  }
  const dim3 grid(ctx->n_units, c.n_kv_heads);
  const int64_t n_lse = (int64_t)ctx->n_req * c.n_q_heads * c.window;
  int sp = prof_begin(ctx, CAKE_PROF_SCORE, st);
  if (lse) {
    lse_to_base2<<<(unsigned)((n_lse + 255) / 256), 256, 0, st>>>(lse, ctx->d_lse2, n_lse);
    count_launch();
  } else {
    score_rowstats_simt<T><<<grid, NT, smem, st>>>(
        (const T*)q_win, (const T*)k, ctx->d_req, ctx->d_units, ctx->d_rowpart, c.n_q_heads,
        c.n_kv_heads, c.window, c.head_dim, ctx->total_tokens, scale2);
    rowstats_combine<<<dim3(ctx->n_req, c.n_kv_heads), kMaxRows, 0, st>>>(
        ctx->d_rowpart, ctx->d_req, ctx->d_lse2, c.n_kv_heads, rows);
    count_launch(2);
  }
  prof_end(ctx, sp, st);
  sp = prof_begin(ctx, CAKE_PROF_SCORE, st);
  score_colstats_simt<T><<<grid, NT, smem, st>>>(
      (const T*)q_win, (const T*)k, ctx->d_req, ctx->d_units, ctx->d_lse2, ctx->d_raw[layer & 1],
      ctx->d_colpart[layer & 1], c.n_q_heads, c.n_kv_heads, c.window, c.head_dim, ctx->total_tokens, scale2,
      c.gamma, c.var_ddof, c.indicator_mode);
  count_launch();
  prof_end(ctx, sp, st);
  return cuda_status(cudaGetLastError());
}

}  // namespace

int32_t launch_score_simt(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                          const float* lse, cudaStream_t st) {
  if (ctx->n_units == 0) return CAKE_OK;
  if (ctx->cfg.dtype == CAKE_DTYPE_FP32) return run<float>(ctx, layer, q_win, k, lse, st);
  return run<__nv_bfloat16>(ctx, layer, q_win, k, lse, st);
}

}  // namespace cake
