// Gather-compaction of the retained K/V rows into the packed varlen cache
// (Eq. 12: K^ = K[D,:], V^ = V[D,:]) and the position getter.
#include "cake_internal.cuh"

namespace cake {
namespace {

// row_offsets[r*L + l] = first packed row of block (r, l); lengths of layers
// outside [lo, hi) or not yet evicted count as zero.
__global__ void packed_offsets(const int32_t* __restrict__ budget, int64_t* __restrict__ offsets,
                               int n_req, int L, int lo, int hi, int Hkv, int Sw) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int64_t acc = 0;
  for (int r = 0; r < n_req; ++r)
    for (int l = 0; l < L; ++l) {
      offsets[(size_t)r * L + l] = acc;
      if (l >= lo && l < hi) acc += (int64_t)Hkv * (budget[(size_t)r * L + l] + Sw);
    }
  offsets[(size_t)n_req * L] = acc;
}

constexpr int GA_THREADS = 256;

// Persistent grid: each warp copies whole rows, `rpp` rows per pass, 16 bytes per lane.
__global__ void __launch_bounds__(GA_THREADS)
gather_rows(LayerPtrs ptrs, const int64_t* __restrict__ offsets, const int32_t* __restrict__ budget,
            const int32_t* __restrict__ list_pos, const ReqInfo* __restrict__ reqs,
            uint4* __restrict__ k_out, uint4* __restrict__ v_out, int32_t* __restrict__ pos_out,
            int n_req, int L, int Hkv, int Sw, int64_t T, int cpr /* 16-byte chunks per row */) {
  const int64_t total = offsets[(size_t)n_req * L];
  const int nblk = n_req * L;
  const int lane = threadIdx.x & 31;
  const int rpp = 32 / cpr;
  const int sub = lane / cpr, chunk = lane - sub * cpr;
  const int64_t warp_global = ((int64_t)blockIdx.x * GA_THREADS + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * GA_THREADS) >> 5;
  for (int64_t base = warp_global * rpp * 4; base < total; base += n_warps * rpp * 4) {
    uint4 kv[4], vv[4];
    int64_t dst[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t row = base + (int64_t)u * rpp + sub;
      dst[u] = -1;
      if (row < total) {
        int lo = 0, hi = nblk - 1;                   // last block with offset <= row
        while (lo < hi) {
          const int mid = (lo + hi + 1) >> 1;
          if (offsets[mid] <= row) lo = mid; else hi = mid - 1;
        }
        const int r = lo / L, l = lo - r * L;
        const ReqInfo rq = reqs[r];
        const int b = budget[lo];
        const int len = b + Sw;
        const int64_t rel = row - offsets[lo];
        const int g = (int)(rel / len), t = (int)(rel - (int64_t)g * len);
        const int pos = t < b ? list_pos[rq.list_off + ((size_t)l * Hkv + g) * rq.cap + t]
                              : rq.n + (t - b);
        const size_t srow = ((size_t)g * T + rq.cu + pos) * cpr + chunk;
        kv[u] = reinterpret_cast<const uint4*>(ptrs.k[l])[srow];
        vv[u] = reinterpret_cast<const uint4*>(ptrs.v[l])[srow];
        dst[u] = row;
        if (pos_out && chunk == 0) pos_out[row] = pos;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (dst[u] >= 0) {
        k_out[(size_t)dst[u] * cpr + chunk] = kv[u];
        v_out[(size_t)dst[u] * cpr + chunk] = vv[u];
      }
    }
  }
}

__global__ void copy_positions(const int32_t* __restrict__ budget, const int32_t* __restrict__ list_pos,
                               const ReqInfo* __restrict__ reqs, int32_t* __restrict__ out,
                               int64_t capacity, int req, int layer, int L, int Hkv, int Sw) {
  const ReqInfo rq = reqs[req];
  const int b = budget[(size_t)req * L + layer];
  const int len = b + Sw;
  const int64_t total = (int64_t)Hkv * len;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total && i < capacity;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int g = (int)(i / len), t = (int)(i - (int64_t)g * len);
    out[i] = t < b ? list_pos[rq.list_off + ((size_t)layer * Hkv + g) * rq.cap + t] : rq.n + (t - b);
  }
}

}  // namespace

int32_t launch_compact(cake_ctx* ctx, int32_t lo, int32_t hi, const LayerPtrs& ptrs, void* k_out,
                       void* v_out, int64_t* row_offsets, int32_t* positions, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  packed_offsets<<<1, 32, 0, st>>>(budget, row_offsets, ctx->n_req, c.n_layers, lo, hi,
                                   c.n_kv_heads, c.window);
  count_launch();
  if (ctx->n_req == 0) return cuda_status(cudaGetLastError());
  const int esize = c.dtype == CAKE_DTYPE_FP32 ? 4 : 2;
  const int cpr = c.head_dim * esize / 16;
  gather_rows<<<ctx->n_sm * 8, GA_THREADS, 0, st>>>(
      ptrs, row_offsets, budget, ctx->list_pos, ctx->d_req, (uint4*)k_out, (uint4*)v_out, positions,
      ctx->n_req, c.n_layers, c.n_kv_heads, c.window, ctx->total_tokens, cpr);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_get_positions(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* out,
                             int64_t capacity, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  copy_positions<<<64, 256, 0, st>>>(budget, ctx->list_pos, ctx->d_req, out, capacity, req, layer,
                                     c.n_layers, c.n_kv_heads, c.window);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
