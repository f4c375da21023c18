// Gather-compaction of the retained K/V rows into the packed varlen cache
// (Eq. 12: K^ = K[D,:], V^ = V[D,:]) and the position getter.
//
// The survivor lists are in bucket order; the packed cache is in ascending token position.
// Positions are distinct integers below n, so the ordering is a bitmap: every retained
// position sets its bit, and the rank of a bit is the number of bits before it.
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

constexpr int POS_THREADS = 1024;

// One CTA per (head, layer in [lo, hi), request): the retained positions of the list in
// ascending order, then the window, written at out[base + g*len ...].  `bitmap` is dynamic
// shared memory when the request's n bits fit, else a slice of global scratch.
__global__ void __launch_bounds__(POS_THREADS)
sorted_positions(const uint2* __restrict__ lists, const int32_t* __restrict__ prefix_all,
                 const ListState* __restrict__ states, const ReqInfo* __restrict__ reqs,
                 const int32_t* __restrict__ budget, const int64_t* __restrict__ offsets,
                 int32_t* __restrict__ out, uint32_t* __restrict__ scratch, int64_t scratch_words,
                 int req0, int lo, int L, int Hkv, int Sw, int smem_words, int64_t capacity) {
  extern __shared__ uint32_t sh_bits[];
  __shared__ int warp_tot[32];
  const int g = blockIdx.x, layer = lo + blockIdx.y, req = req0 + blockIdx.z;
  const ReqInfo rq = reqs[req];
  const size_t lid = ((size_t)req * L + layer) * Hkv + g;
  const int b = budget[(size_t)req * L + layer];
  const int len = b + Sw;
  int32_t* dst = out + (offsets ? offsets[(size_t)req * L + layer] : 0) + (int64_t)g * len;
  // without row offsets the caller gave a capacity: never write past it
  const int64_t room = offsets ? (int64_t)len : capacity - (int64_t)g * len;
  const int words = (rq.n + 31) >> 5;
  uint32_t* bits = sh_bits;
  const bool in_smem = words <= smem_words;
  if (!in_smem) {
    const size_t cta = ((size_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
    bits = scratch + cta * (size_t)scratch_words;
  }
  for (int wi = threadIdx.x; wi < words; wi += POS_THREADS) bits[wi] = 0;
  if (in_smem) __syncthreads(); else { __threadfence_block(); __syncthreads(); }
  const ListState st = states[lid];
  if (st.bucket >= 0 && b > 0) {
    const int32_t* pf = prefix_all + lid * (kBins + 1);
    const uint2* list = lists + rq.list_off + ((size_t)layer * Hkv + g) * rq.n;
    const int start = pf[st.bucket], end = pf[st.bucket + 1];
    for (int i = threadIdx.x; i < end; i += POS_THREADS) {
      const uint2 e = list[i];
      const bool keep = i < start || e.x > st.thr_key || (e.x == st.thr_key && (int32_t)e.y <= st.pos_cut);
      if (keep && e.y < (uint32_t)rq.n) atomicOr(&bits[e.y >> 5], 1u << (e.y & 31));
    }
  }
  __syncthreads();
  // rank of every word, then expand
  const int per = (words + POS_THREADS - 1) / POS_THREADS;
  const int w0 = threadIdx.x * per, w1 = min(words, w0 + per);
  int cnt = 0;
  for (int wi = w0; wi < w1; ++wi) cnt += __popc(bits[wi]);
  // exclusive scan over the block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = warp_tot[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_tot[lane] = winc - w;
  }
  __syncthreads();
  int rank = warp_tot[warp] + inc - cnt;
  for (int wi = w0; wi < w1; ++wi) {
    uint32_t m = bits[wi];
    while (m) {
      const int bit = __ffs(m) - 1;
      m &= m - 1;
      if (rank < b && rank < room) dst[rank] = (wi << 5) + bit;
      ++rank;
    }
  }
  for (int t = threadIdx.x; t < Sw; t += POS_THREADS)
    if (b + t < room) dst[b + t] = rq.n + t;
}

constexpr int GA_THREADS = 256;

// Persistent grid: each warp copies whole rows, `rpp` rows per pass, 16 bytes per lane.
__global__ void __launch_bounds__(GA_THREADS)
gather_rows(LayerPtrs ptrs, const int64_t* __restrict__ offsets, const int32_t* __restrict__ budget,
            const int32_t* __restrict__ pos_packed, const ReqInfo* __restrict__ reqs,
            uint4* __restrict__ k_out, uint4* __restrict__ v_out, int n_req, int L, int Hkv, int Sw,
            int64_t T, int cpr /* 16-byte chunks per row */) {
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
        const int len = budget[lo] + Sw;
        const int64_t rel = row - offsets[lo];
        const int g = (int)(rel / len);
        const int pos = pos_packed[row];
        const size_t srow = ((size_t)g * T + rq.cu + pos) * cpr + chunk;
        kv[u] = reinterpret_cast<const uint4*>(ptrs.k[l])[srow];
        vv[u] = reinterpret_cast<const uint4*>(ptrs.v[l])[srow];
        dst[u] = row;
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

int32_t run_sorted_positions(cake_ctx* ctx, int req0, int n_req, int lo, int hi, const int64_t* offsets,
                             int32_t* out, int64_t capacity, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (n_req <= 0 || hi <= lo) return CAKE_OK;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  int max_n = 0;
  for (int r = req0; r < req0 + n_req; ++r) max_n = ctx->h_req[r].n > max_n ? ctx->h_req[r].n : max_n;
  int need_words = (max_n + 31) / 32;
  int smem_words = need_words < kBitmapSmemWords ? need_words : kBitmapSmemWords;
  static PerDeviceOnce attr;
  if (attr.need(ctx->device)) {
    CAKE_CUDA_TRY(cudaFuncSetAttribute(sorted_positions, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kBitmapSmemWords * 4));
    attr.mark(ctx->device);
  }
  const int64_t ctas = (int64_t)c.n_kv_heads * (hi - lo) * n_req;
  if (need_words > kBitmapSmemWords &&
      (!ctx->d_bitmap || ctas * (int64_t)need_words > ctx->bitmap_words)) return CAKE_ERR_CAPACITY;
  const dim3 grid(c.n_kv_heads, hi - lo, n_req);
  sorted_positions<<<grid, POS_THREADS, (size_t)smem_words * 4, st>>>(
      ctx->d_lists, ctx->d_prefix, ctx->d_lstate, ctx->d_req,
      budget, offsets, out, ctx->d_bitmap, need_words, req0, lo, c.n_layers, c.n_kv_heads, c.window,
      smem_words, capacity);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace

int32_t launch_compact(cake_ctx* ctx, int32_t lo, int32_t hi, const LayerPtrs& ptrs, void* k_out,
                       void* v_out, int64_t* row_offsets, int32_t* positions, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  packed_offsets<<<1, 32, 0, st>>>(budget, row_offsets, ctx->n_req, c.n_layers, lo, hi,
                                   c.n_kv_heads, c.window);
  count_launch();
  if (ctx->n_req == 0 || hi <= lo) return cuda_status(cudaGetLastError());
  // positions in packed row order: into the caller's buffer if there is one
  int32_t* pos = positions ? positions : ctx->d_pos_packed;
  int32_t rc = run_sorted_positions(ctx, 0, ctx->n_req, lo, hi, row_offsets, pos, 0, st);
  if (rc != CAKE_OK) return rc;
  const int esize = c.dtype == CAKE_DTYPE_FP32 ? 4 : 2;
  const int cpr = c.head_dim * esize / 16;
  gather_rows<<<ctx->n_sm * 8, GA_THREADS, 0, st>>>(
      ptrs, row_offsets, budget, pos, ctx->d_req, (uint4*)k_out, (uint4*)v_out, ctx->n_req,
      c.n_layers, c.n_kv_heads, c.window, ctx->total_tokens, cpr);
  count_launch();
  return cuda_status(cudaGetLastError());
}

// Packed row offsets and positions of layers [lo, hi): the first half of a compaction.
int32_t run_packed_positions(cake_ctx* ctx, int32_t lo, int32_t hi, int64_t* row_offsets, int32_t* positions,
                             cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  packed_offsets<<<1, 32, 0, st>>>(budget, row_offsets, ctx->n_req, c.n_layers, lo, hi, c.n_kv_heads,
                                   c.window);
  count_launch();
  if (ctx->n_req == 0 || hi <= lo) return cuda_status(cudaGetLastError());
  return run_sorted_positions(ctx, 0, ctx->n_req, lo, hi, row_offsets, positions, 0, st);
}

// Packed row offsets and positions of every layer into context scratch (decode-time set-up).
int32_t run_sorted_positions_packed(cake_ctx* ctx, const int64_t* offsets_c, int32_t* out, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  int64_t* offsets = const_cast<int64_t*>(offsets_c);
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  packed_offsets<<<1, 32, 0, st>>>(budget, offsets, ctx->n_req, c.n_layers, 0, c.n_layers, c.n_kv_heads,
                                   c.window);
  count_launch();
  return run_sorted_positions(ctx, 0, ctx->n_req, 0, c.n_layers, offsets, out, 0, st);
}

int32_t launch_get_positions(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* out,
                             int64_t capacity, cudaStream_t st) {
  if (capacity < 0) return CAKE_ERR_ARG;
  return run_sorted_positions(ctx, req, 1, layer, layer + 1, nullptr, out, capacity, st);
}

}  // namespace cake
