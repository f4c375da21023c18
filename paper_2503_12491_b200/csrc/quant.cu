// Quantised gather-compaction: the retained K/V rows (Eq. 12) written as asymmetric 4-bit codes,
// keys per channel and values per token -- the "KIVI-INT4 with CAKE" combination of the paper's
// appendix "Comparison and Compatibility with Quantization Methods".
//
// A group of `group` values shares zero = min and scale = (max - min) / 15 (scale = 1 when
// max = min); code = clamp(rint((x - zero) / scale), 0, 15), all in IEEE fp32 (round to nearest
// even), two codes per byte (the even-numbered channel in the low nibble).
//   values: a group is `group` consecutive channels of one retained row;
//   keys:   a group is one channel over `group` consecutive retained rows of one (request, layer,
//           head) in packed order (ascending position, window last); the last group of a head
//           may be shorter.
#include "cake_internal.cuh"

#include <math_constants.h>

namespace cake {
namespace {

template <typename T> __device__ __forceinline__ float ld_f32(const T* p);
template <> __device__ __forceinline__ float ld_f32<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// A lane's `per` (2 or 4) consecutive elements of a row in one load of 4, 8 or 16 bytes.
template <typename T> __device__ __forceinline__ void ld_lane(const T* p, int per, float (&x)[4]);
template <> __device__ __forceinline__ void ld_lane<float>(const float* p, int per, float (&x)[4]) {
  if (per == 4) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  } else {
    const float2 v = *reinterpret_cast<const float2*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = 0.f; x[3] = 0.f;
  }
}
template <> __device__ __forceinline__ void ld_lane<__nv_bfloat16>(const __nv_bfloat16* p, int per, float (&x)[4]) {
  uint2 v = make_uint2(0u, 0u);
  if (per == 4) v = *reinterpret_cast<const uint2*>(p);
  else v.x = *reinterpret_cast<const uint32_t*>(p);
  x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
  x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
}

__device__ __forceinline__ uint32_t code4(float x, float zero, float scale) {
  const float q = rintf(__fdiv_rn(__fsub_rn(x, zero), scale));
  return (uint32_t)fminf(fmaxf(q, 0.f), 15.f);
}
// The same code from a multiplication by rcp = 1 / scale (rounded to nearest).  x * rcp is within
// a few 1e-6 of the exact quotient (codes are at most 15), so it rounds to the same integer as the
// IEEE quotient unless it lies that close to a half-integer; only then (and for non-finite
// operands, which fail the comparison) the IEEE division decides.
__device__ __forceinline__ uint32_t code4_rcp(float x, float zero, float scale, float rcp) {
  const float dlt = __fsub_rn(x, zero);
  const float q0 = __fmul_rn(dlt, rcp);
  const float h = q0 - floorf(q0);
  if (!(fabsf(h - 0.5f) >= 1e-4f)) return code4(x, zero, scale);
  return (uint32_t)fminf(fmaxf(rintf(q0), 0.f), 15.f);
}
__device__ __forceinline__ float scale_of(float mn, float mx) {
  return mx > mn ? __fdiv_rn(__fsub_rn(mx, mn), 15.f) : 1.f;
}

// key-group offsets: block (r, l) holds H_kv * ceil(len / group) groups
__global__ void key_group_offsets(const int32_t* __restrict__ budget, int64_t* __restrict__ offsets,
                               int n_req, int L, int lo, int hi, int Hkv, int Sw, int group) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int64_t acc = 0;
  for (int r = 0; r < n_req; ++r)
    for (int l = 0; l < L; ++l) {
      offsets[(size_t)r * L + l] = acc;
      if (l >= lo && l < hi) acc += (int64_t)Hkv * ((budget[(size_t)r * L + l] + Sw + group - 1) / group);
    }
  offsets[(size_t)n_req * L] = acc;
}

// Values, one warp per packed row: d / 32 channels per lane; a group spans group / (d / 32) lanes.
template <typename T>
__global__ void __launch_bounds__(256)
quant_values(LayerPtrs ptrs, const int64_t* __restrict__ offsets, const int32_t* __restrict__ budget,
             const int32_t* __restrict__ pos_packed, const ReqInfo* __restrict__ reqs,
             uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ zero, int n_req,
             int L, int Hkv, int Sw, int64_t T_tokens, int d, int group) {
  const int64_t total = offsets[(size_t)n_req * L];
  const int nblk = n_req * L;
  const int lane = threadIdx.x & 31;
  const int per = d / 32;                            // 2 (d = 64) or 4 (d = 128) channels per lane
  const int lanes_per_group = group / per;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  // four rows per warp and round trip: their addresses first, then their values
  for (int64_t row0 = warp0 * 4; row0 < total; row0 += n_warps * 4) {
    const T* src[4];
    float x[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t row = row0 + u;
      src[u] = nullptr;
      if (row < total) {
        int lo = 0, hi = nblk - 1;                   // last block with offset <= row
        while (lo < hi) {
          const int mid = (lo + hi + 1) >> 1;
          if (offsets[mid] <= row) lo = mid; else hi = mid - 1;
        }
        const int r = lo / L, l = lo - r * L;
        const int len = budget[lo] + Sw;
        const int g = (int)((row - offsets[lo]) / len);
        src[u] = reinterpret_cast<const T*>(ptrs.v[l]) +
                 ((size_t)g * T_tokens + reqs[r].cu + pos_packed[row]) * d + lane * per;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      x[u][0] = x[u][1] = x[u][2] = x[u][3] = 0.f;
      if (src[u]) ld_lane<T>(src[u], per, x[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t row = row0 + u;
      if (row >= total) break;                       // uniform over the warp
      float mn = CUDART_INF_F, mx = -CUDART_INF_F;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e < per) { mn = fminf(mn, x[u][e]); mx = fmaxf(mx, x[u][e]); }
      for (int o = 1; o < lanes_per_group; o <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      const float sc = scale_of(mn, mx);
      const float rc = __frcp_rn(sc);
      uint32_t packed = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e < per) packed |= code4_rcp(x[u][e], mn, sc, rc) << (4 * e);
      uint8_t* dst = codes + (size_t)row * (d / 2) + lane * (per / 2);
      if (per == 4) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)packed;
      else dst[0] = (uint8_t)(packed & 0xFF);
      if (lane % lanes_per_group == 0) {
        const size_t gi = (size_t)row * (d / group) + lane / lanes_per_group;
        scale[gi] = sc;
        zero[gi] = mn;
      }
    }
  }
}

// Keys, one CTA of d threads per (head, token group) of a block: thread = channel.
template <typename T>
__global__ void quant_keys(LayerPtrs ptrs, const int64_t* __restrict__ offsets,
                           const int64_t* __restrict__ kg_off, const int32_t* __restrict__ budget,
                           const int32_t* __restrict__ pos_packed, const ReqInfo* __restrict__ reqs,
                           uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ zero,
                           int n_req, int L, int Hkv, int Sw, int64_t T_tokens, int d, int group) {
  const int64_t total_groups = kg_off[(size_t)n_req * L];
  const int nblk = n_req * L;
  const int c = threadIdx.x;
  for (int64_t gi = blockIdx.x; gi < total_groups; gi += gridDim.x) {
    int lo = 0, hi = nblk - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (kg_off[mid] <= gi) lo = mid; else hi = mid - 1;
    }
    const int r = lo / L, l = lo - r * L;
    const int len = budget[lo] + Sw;
    const int gpb = (len + group - 1) / group;       // groups per head of this block
    const int64_t rel = gi - kg_off[lo];
    const int g = (int)(rel / gpb);
    const int t0 = (int)(rel - (int64_t)g * gpb) * group, t1 = min(len, t0 + group);
    const int64_t row0 = offsets[lo] + (int64_t)g * len;
    const T* base = reinterpret_cast<const T*>(ptrs.k[l]) + ((size_t)g * T_tokens + reqs[r].cu) * d + c;
    // eight rows per round trip: their positions first, then their values
    float mn = CUDART_INF_F, mx = -CUDART_INF_F;
    for (int t = t0; t < t1; t += 8) {
      int ps[8];
      float xs[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) ps[u] = t + u < t1 ? pos_packed[row0 + t + u] : -1;
#pragma unroll
      for (int u = 0; u < 8; ++u) xs[u] = ps[u] >= 0 ? ld_f32(base + (size_t)ps[u] * d) : 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (ps[u] >= 0) { mn = fminf(mn, xs[u]); mx = fmaxf(mx, xs[u]); }
    }
    const float sc = scale_of(mn, mx);
    const float rc = __frcp_rn(sc);
    scale[(size_t)gi * d + c] = sc;
    zero[(size_t)gi * d + c] = mn;
    for (int t = t0; t < t1; t += 8) {
      int ps[8];
      float xs[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) ps[u] = t + u < t1 ? pos_packed[row0 + t + u] : -1;
#pragma unroll
      for (int u = 0; u < 8; ++u) xs[u] = ps[u] >= 0 ? ld_f32(base + (size_t)ps[u] * d) : 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t q = code4_rcp(xs[u], mn, sc, rc);  // every lane takes part in the shuffle
        const uint32_t hi4 = __shfl_down_sync(0xffffffffu, q, 1);
        if (ps[u] >= 0 && (c & 1) == 0) codes[(size_t)(row0 + t + u) * (d / 2) + (c >> 1)] = (uint8_t)(q | (hi4 << 4));
      }
    }
  }
}

}  // namespace

int32_t run_packed_positions(cake_ctx* ctx, int32_t lo, int32_t hi, int64_t* row_offsets, int32_t* positions,
                             cudaStream_t st);

int32_t launch_compact_int4(cake_ctx* ctx, int32_t lo, int32_t hi, const LayerPtrs& ptrs, int32_t group,
                            uint8_t* k_codes, float* k_scale, float* k_zero, uint8_t* v_codes,
                            float* v_scale, float* v_zero, int64_t* row_offsets, int64_t* kgroup_offsets,
                            int32_t* positions, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  int32_t* pos = positions ? positions : ctx->d_pos_packed;
  const int32_t rc = run_packed_positions(ctx, lo, hi, row_offsets, pos, st);
  if (rc != CAKE_OK) return rc;
  key_group_offsets<<<1, 32, 0, st>>>(budget, kgroup_offsets, ctx->n_req, c.n_layers, lo, hi, c.n_kv_heads,
                                   c.window, group);
  count_launch();
  if (ctx->n_req == 0 || hi <= lo) return cuda_status(cudaGetLastError());
  const int grid = ctx->n_sm * 8;
  if (c.dtype == CAKE_DTYPE_FP32) {
    quant_values<float><<<grid, 256, 0, st>>>(ptrs, row_offsets, budget, pos, ctx->d_req, v_codes, v_scale,
                                              v_zero, ctx->n_req, c.n_layers, c.n_kv_heads, c.window,
                                              ctx->total_tokens, c.head_dim, group);
    quant_keys<float><<<grid, c.head_dim, 0, st>>>(ptrs, row_offsets, kgroup_offsets, budget, pos, ctx->d_req,
                                                   k_codes, k_scale, k_zero, ctx->n_req, c.n_layers,
                                                   c.n_kv_heads, c.window, ctx->total_tokens, c.head_dim, group);
  } else {
    quant_values<__nv_bfloat16><<<grid, 256, 0, st>>>(ptrs, row_offsets, budget, pos, ctx->d_req, v_codes,
                                                      v_scale, v_zero, ctx->n_req, c.n_layers, c.n_kv_heads,
                                                      c.window, ctx->total_tokens, c.head_dim, group);
    quant_keys<__nv_bfloat16><<<grid, c.head_dim, 0, st>>>(ptrs, row_offsets, kgroup_offsets, budget, pos,
                                                           ctx->d_req, k_codes, k_scale, k_zero, ctx->n_req,
                                                           c.n_layers, c.n_kv_heads, c.window,
                                                           ctx->total_tokens, c.head_dim, group);
  }
  count_launch(2);
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
