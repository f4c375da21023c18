// Decode-time eviction with frozen per-layer budgets (Section 5.1 "Implementation Details";
// Appendix "More Implementation Details"; the decode branches of the appendix listing).
//
// After the prefill cascade every (request, layer) keeps len = b + S_w tokens per KV head.  The
// decode cache of a block (request, layer) is laid out [H_kv][cap][d] with cap = len + 1: a head
// owns cap row slots, len of them hold the retained tokens and one is free.  Per generated token
// and layer, cake_decode_step
//   1. writes the new token's K/V row into the head's free slot,
//   2. takes the new query's attention over the head's cap cached keys (softmax over all of
//      them, the columns of the S_w most recent tokens dropped, mean over the group's query heads),
//   3. pools it along ascending token position and updates the stored scores with it,
//   4. evicts the entry that comes last in the order (score descending, position ascending)
//      among the tokens outside the recent window: its slot becomes the free one.
// Rows never move: the order of a head's entries by position is kept as a list of slots.
#include "cake_internal.cuh"

#include <algorithm>
#include <cstdlib>

#include <cooperative_groups.h>

#include <math_constants.h>

namespace cake {
namespace {

constexpr int DEC_THREADS = 512;
constexpr int DEC_CLUSTER = 8;    // CTAs that share a head in the cluster form of the step kernel
constexpr int DEC_CLUSTER_MIN_CAP = 512;   // smaller heads stay on one CTA
constexpr int DEC_ROWS = 4;       // cache rows a half-warp has in flight in the logit loop

__device__ __forceinline__ float key_to_float(uint32_t key) {
  const uint32_t b = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
  return __uint_as_float(b);
}

// Decode row offsets: block (r, l) occupies H_kv * (len + 1) rows.
__global__ void decode_offsets(const int32_t* __restrict__ budget, int64_t* __restrict__ offsets,
                               int n_req, int L, int Hkv, int Sw) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int64_t acc = 0;
  for (int i = 0; i < n_req * L; ++i) {
    offsets[i] = acc;
    acc += (int64_t)Hkv * (budget[i] + Sw + 1);
  }
  offsets[(size_t)n_req * L] = acc;
}

// One CTA per (head, layer, request): positions (ascending, from the packed order), identity
// slot order, and the stored indicator of every survivor, found by binary search of its position.
__global__ void __launch_bounds__(DEC_THREADS)
decode_build(const uint2* __restrict__ lists, const int32_t* __restrict__ prefix_all,
             const ListState* __restrict__ states, const ReqInfo* __restrict__ reqs,
             const int32_t* __restrict__ budget, const int64_t* __restrict__ packed_off,
             const int32_t* __restrict__ pos_packed, const int64_t* __restrict__ dec_off,
             float* __restrict__ score, int32_t* __restrict__ pos, int32_t* __restrict__ order,
             int4* __restrict__ meta, int L, int Hkv, int Sw) {
  const int g = blockIdx.x, layer = blockIdx.y, req = blockIdx.z;
  const ReqInfo rq = reqs[req];
  const int blk = req * L + layer;
  const size_t lid = (size_t)blk * Hkv + g;
  const int b = budget[blk];
  const int len = b + Sw, cap = len + 1;
  const int32_t* src = pos_packed + packed_off[blk] + (int64_t)g * len;
  const int64_t base = dec_off[blk] + (int64_t)g * cap;
  for (int i = threadIdx.x; i < cap; i += DEC_THREADS) {
    pos[base + i] = i < len ? src[i] : -1;
    order[base + i] = i;
    score[base + i] = 0.f;
  }
  if (threadIdx.x == 0) meta[lid] = make_int4(len, len, rq.N, b);
  __syncthreads();
  const ListState st = states[lid];
  if (st.bucket < 0 || b <= 0) return;
  const int32_t* pf = prefix_all + lid * (kBins + 1);
  const uint2* list = lists + rq.list_off + ((size_t)layer * Hkv + g) * rq.n;
  const int start = pf[st.bucket], end = pf[st.bucket + 1];
  for (int i = threadIdx.x; i < end; i += DEC_THREADS) {
    const uint2 e = list[i];
    const bool keep = i < start || e.x > st.thr_key || (e.x == st.thr_key && (int32_t)e.y <= st.pos_cut);
    if (!keep) continue;
    int lo = 0, hi = b - 1;                          // positions of the non-window survivors are sorted
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (src[mid] < (int32_t)e.y) lo = mid + 1; else hi = mid;
    }
    if (src[lo] == (int32_t)e.y) score[base + lo] = key_to_float(e.x);
  }
}

struct DecodeArgs {
  const void* q_new;       // [n_req][H_q][d]
  const void* k_new;       // [n_req][H_kv][d]
  const void* v_new;
  void* k_cache;           // decode cache rows of d elements
  void* v_cache;
  const int64_t* dec_off;
  float* score;
  int32_t* pos;
  int32_t* order;
  int4* meta;              // (len, free slot, next position, frozen budget)
  int32_t* status;
  float* tmp;              // per (head, request) work area for heads beyond the shared-memory plan
  const ReqInfo* reqs;
  int64_t T;               // tokens of the batch
  int n_req;
  int layer, L, Hq, Hkv, d, Sw, kp, pool_mode, update_mode, smem_cap;
  float scale2;
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// A lane's share of a row (up to 32 bytes held as four 8-byte words) as eight floats; elements
// beyond the share are zero because the words beyond it are.
template <typename T> __device__ __forceinline__ void unpack_row(const uint2 (&w)[4], float (&out)[8]);
template <> __device__ __forceinline__ void unpack_row<float>(const uint2 (&w)[4], float (&out)[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) { out[2 * i] = __uint_as_float(w[i].x); out[2 * i + 1] = __uint_as_float(w[i].y); }
}
template <> __device__ __forceinline__ void unpack_row<__nv_bfloat16>(const uint2 (&w)[4], float (&out)[8]) {
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    out[4 * i] = __uint_as_float(w[i].x << 16);     out[4 * i + 1] = __uint_as_float(w[i].x & 0xFFFF0000u);
    out[4 * i + 2] = __uint_as_float(w[i].y << 16); out[4 * i + 3] = __uint_as_float(w[i].y & 0xFFFF0000u);
  }
}

// (value, index) argmin with the tie rule of the eviction: the lowest score goes, among equal
// scores the highest rank (= the highest token position).
__device__ __forceinline__ void worse_of(float& v, int& i, float ov, int oi) {
  if (ov < v || (ov == v && oi > i)) { v = ov; i = oi; }
}

// One CTA per (KV head, request).  Dynamic shared memory: p[G][cap] (logits, then unnormalised
// probabilities by slot) and abar[cap] (group-mean attention by rank).
template <typename T, int G>
__global__ void __launch_bounds__(DEC_THREADS)
decode_step_kernel(const DecodeArgs A) {
  extern __shared__ float sh[];
  __shared__ float red_v[DEC_THREADS / 32];
  __shared__ int red_i[DEC_THREADS / 32];
  __shared__ float s_m[G], s_z[G];
  const int g = blockIdx.x, req = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int blk = req * A.L + A.layer;
  const size_t lid = (size_t)blk * A.Hkv + g;
  const int4 mt = A.meta[lid];
  const int len = mt.x, fre = mt.y, next_pos = mt.z, budget = mt.w;
  const int cap = len + 1;
  const int64_t base = A.dec_off[blk] + (int64_t)g * cap;
  // A head beyond the shared-memory plan works in global memory: its (G + 1) * cap floats lie
  // at the request's token offset of a [H_kv][tokens + requests] area (cap <= N + 1).
  float* p = cap <= A.smem_cap                       // [G][cap]
                 ? sh
                 : A.tmp + (size_t)(G + 1) * ((size_t)g * (size_t)(A.T + A.n_req) + (size_t)A.reqs[req].cu + req);
  float* abar = p + (size_t)G * cap;                 // [cap]
  T* kc = reinterpret_cast<T*>(A.k_cache) + (size_t)base * A.d;
  T* vc = reinterpret_cast<T*>(A.v_cache) + (size_t)base * A.d;
  const T* kn = reinterpret_cast<const T*>(A.k_new) + ((size_t)req * A.Hkv + g) * A.d;
  const T* vn = reinterpret_cast<const T*>(A.v_new) + ((size_t)req * A.Hkv + g) * A.d;
  // 1. the new token takes the free slot and the last rank
  for (int e = threadIdx.x; e < A.d; e += DEC_THREADS) {
    kc[(size_t)fre * A.d + e] = kn[e];
    vc[(size_t)fre * A.d + e] = vn[e];
  }
  if (threadIdx.x == 0) {
    A.order[base + len] = fre;
    A.pos[base + fre] = next_pos;
  }
  // 2. logits of the G query heads against every slot: 16 lanes per row, two rows per warp pass
  const int sub = lane >> 4, l16 = lane & 15;
  const int per = A.d / 16;                          // elements of a row per lane
  float qv[G][8];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int e = 0; e < 8; ++e)
      qv[h][e] = e < per ? to_f32(reinterpret_cast<const T*>(A.q_new)[((size_t)req * A.Hq + g * G + h) * A.d +
                                                                     l16 * per + e]) : 0.f;
  // a lane's share of a row is 8, 16 or 32 bytes: 8-byte loads, DEC_ROWS rows in flight per half-warp
  const int n8 = per * (int)sizeof(T) / 8;
  constexpr int kStep = (DEC_THREADS / 32) * 2;
  for (int s0 = warp * 2; s0 < cap; s0 += kStep * DEC_ROWS) {
    uint2 raw[DEC_ROWS][4];
#pragma unroll
    for (int u = 0; u < DEC_ROWS; ++u) {
      const int s = s0 + u * kStep + sub;
      const T* row = s == fre ? kn : kc + (size_t)s * A.d;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        raw[u][i] = (s < cap && i < n8) ? reinterpret_cast<const uint2*>(row + l16 * per)[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < DEC_ROWS; ++u) {
      const int s = s0 + u * kStep + sub;
      float kv[8];
      unpack_row<T>(raw[u], kv);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fmaf(qv[h][e], kv[e], acc);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (l16 == 0 && s < cap) p[(size_t)h * cap + s] = acc * A.scale2;
      }
    }
  }
  __syncthreads();
  // 3. softmax per head over all cap slots (base 2)
  for (int h = 0; h < G; ++h) {
    float m = -CUDART_INF_F;
#pragma unroll 4
    for (int s = threadIdx.x; s < cap; s += DEC_THREADS) m = fmaxf(m, p[(size_t)h * cap + s]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red_v[warp] = m;
    __syncthreads();
    m = red_v[0];
    for (int w = 1; w < DEC_THREADS / 32; ++w) m = fmaxf(m, red_v[w]);
    __syncthreads();
    float z = 0.f;
#pragma unroll 4
    for (int s = threadIdx.x; s < cap; s += DEC_THREADS) {
      const float e = exp2f(p[(size_t)h * cap + s] - m);
      p[(size_t)h * cap + s] = e;
      z += e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) red_v[warp] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int w = 0; w < DEC_THREADS / 32; ++w) t += red_v[w];
      s_z[h] = t;
      s_m[h] = m;
    }
    __syncthreads();
  }
  // 4. group-mean observed attention by rank (ascending position), pooling, score update
  const int n_obs = cap - A.Sw;                      // entries outside the recent window
  const int n_old = len - A.Sw;                      // of which these already carry a score
#pragma unroll 4
  for (int r = threadIdx.x; r < n_obs; r += DEC_THREADS) {
    const int s = A.order[base + r];
    float a = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h) a += p[(size_t)h * cap + s] / s_z[h];
    abar[r] = a * (1.f / (float)G);
  }
  __syncthreads();
  const int rad = A.kp >> 1;
  float worst = CUDART_INF_F;
  int worst_r = -1;
#pragma unroll 2
  for (int r = threadIdx.x; r < n_obs; r += DEC_THREADS) {
    const int lo = max(0, r - rad), hi = min(n_obs, r + rad + 1);
    float v = abar[lo];
    for (int x = lo + 1; x < hi; ++x) v = A.pool_mode == CAKE_POOL_MAX ? fmaxf(v, abar[x]) : v + abar[x];
    if (A.pool_mode != CAKE_POOL_MAX) v /= (float)A.kp;
    const int s = A.order[base + r];
    float sc = v;
    if (r < n_old) {
      const float old = A.score[base + s];
      sc = A.update_mode == CAKE_DECODE_ADD ? old + v : A.update_mode == CAKE_DECODE_MAX ? fmaxf(old, v) : v;
    }
    A.score[base + s] = sc;
    worse_of(worst, worst_r, sc, r);
  }
  // 5. evict back to the frozen budget: the entry that is last in (score desc, position asc)
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, worst, o);
    const int oi = __shfl_xor_sync(0xffffffffu, worst_r, o);
    if (oi >= 0 && (worst_r < 0 || ov < worst || (ov == worst && oi > worst_r))) { worst = ov; worst_r = oi; }
  }
  __syncthreads();                                   // red_v is free again
  if (lane == 0) { red_v[warp] = worst; red_i[warp] = worst_r; }
  __syncthreads();
  int ev = -1;
  if (n_obs > budget) {
    float bv = CUDART_INF_F;
    for (int w = 0; w < DEC_THREADS / 32; ++w) {
      if (red_i[w] >= 0 && (ev < 0 || red_v[w] < bv || (red_v[w] == bv && red_i[w] > ev))) {
        bv = red_v[w];
        ev = red_i[w];
      }
    }
  }
  if (ev < 0) {                                      // below the budget: the cache would have to grow
    if (threadIdx.x == 0) atomicCAS(A.status, 0, CAKE_ERR_CAPACITY);
    return;
  }
  // ranks after the evicted one move down by one; its slot becomes the free one
  const int ev_slot = A.order[base + ev];
  __syncthreads();
  for (int r0 = ev; r0 < cap - 1; r0 += DEC_THREADS * 4) {       // four batches per round trip
    int nxt[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + u * DEC_THREADS + threadIdx.x;
      nxt[u] = r < cap - 1 ? A.order[base + r + 1] : 0;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + u * DEC_THREADS + threadIdx.x;
      if (r < cap - 1) A.order[base + r] = nxt[u];
    }
    __syncthreads();                                 // the next round reads beyond what this one wrote, but keep rounds apart
  }
  if (threadIdx.x == 0) {
    A.order[base + cap - 1] = ev_slot;
    A.pos[base + ev_slot] = -1;
    A.meta[lid] = make_int4(len, ev_slot, next_pos + 1, budget);
  }
}

// The same step with a head spread over a thread-block cluster of DEC_CLUSTER CTAs: the head's
// slots (logits, softmax) and then its ranks (pooling, score update, list shift) are cut into
// DEC_CLUSTER contiguous parts, the per-head maxima, sums and the eviction candidate are exchanged
// through distributed shared memory, and the group-mean attention passes from slot order to rank
// order through the context's work area.  Every cluster barrier is reached by all CTAs of the
// cluster: what decides the control flow (cap, the evicted rank) is the same in all of them.
// Dynamic shared memory: G * part floats (logits by slot), reused for the pooled window and the
// list shift.
template <typename T, int G>
__global__ void __launch_bounds__(DEC_THREADS)
decode_step_cluster_kernel(const DecodeArgs A) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ float sh[];
  __shared__ float red_v[DEC_THREADS / 32];
  __shared__ int red_i[DEC_THREADS / 32];
  __shared__ float x_m[G], x_z[G];                   // this CTA's partial maximum / sum per head
  __shared__ float x_worst;                          // this CTA's eviction candidate
  __shared__ int x_worst_r;
  __shared__ float s_m[G], s_z[G];
  const int crank = (int)cluster.block_rank();
  const int g = blockIdx.x / DEC_CLUSTER, req = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int blk = req * A.L + A.layer;
  const size_t lid = (size_t)blk * A.Hkv + g;
  const int4 mt = A.meta[lid];
  const int len = mt.x, fre = mt.y, next_pos = mt.z, budget = mt.w;
  const int cap = len + 1;
  const int64_t base = A.dec_off[blk] + (int64_t)g * cap;
  const int part = (cap + DEC_CLUSTER - 1) / DEC_CLUSTER;
  const int s_lo = min(cap, crank * part), s_hi = min(cap, s_lo + part);
  float* p = sh;                                     // [G][part], slot s at s - s_lo
  float* aslot = A.tmp + (size_t)(G + 1) * ((size_t)g * (size_t)(A.T + A.n_req) + (size_t)A.reqs[req].cu + req);
  T* kc = reinterpret_cast<T*>(A.k_cache) + (size_t)base * A.d;
  T* vc = reinterpret_cast<T*>(A.v_cache) + (size_t)base * A.d;
  const T* kn = reinterpret_cast<const T*>(A.k_new) + ((size_t)req * A.Hkv + g) * A.d;
  const T* vn = reinterpret_cast<const T*>(A.v_new) + ((size_t)req * A.Hkv + g) * A.d;
  // 1. the new token takes the free slot and the last rank (first CTA of the cluster)
  if (crank == 0) {
    for (int e = threadIdx.x; e < A.d; e += DEC_THREADS) {
      kc[(size_t)fre * A.d + e] = kn[e];
      vc[(size_t)fre * A.d + e] = vn[e];
    }
    if (threadIdx.x == 0) {
      A.order[base + len] = fre;
      A.pos[base + fre] = next_pos;
    }
  }
  // 2. logits of the G query heads against this CTA's slots
  const int sub = lane >> 4, l16 = lane & 15;
  const int per = A.d / 16;
  float qv[G][8];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int e = 0; e < 8; ++e)
      qv[h][e] = e < per ? to_f32(reinterpret_cast<const T*>(A.q_new)[((size_t)req * A.Hq + g * G + h) * A.d +
                                                                     l16 * per + e]) : 0.f;
  const int n8 = per * (int)sizeof(T) / 8;
  constexpr int kStep = (DEC_THREADS / 32) * 2;
  for (int s0 = s_lo + warp * 2; s0 < s_hi; s0 += kStep * DEC_ROWS) {
    uint2 raw[DEC_ROWS][4];
#pragma unroll
    for (int u = 0; u < DEC_ROWS; ++u) {
      const int s = s0 + u * kStep + sub;
      const T* row = s == fre ? kn : kc + (size_t)s * A.d;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        raw[u][i] = (s < s_hi && i < n8) ? reinterpret_cast<const uint2*>(row + l16 * per)[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < DEC_ROWS; ++u) {
      const int s = s0 + u * kStep + sub;
      float kv[8];
      unpack_row<T>(raw[u], kv);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fmaf(qv[h][e], kv[e], acc);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (l16 == 0 && s < s_hi) p[(size_t)h * part + (s - s_lo)] = acc * A.scale2;
      }
    }
  }
  __syncthreads();
  // 3. softmax per head over all cap slots (base 2): partial maxima, then partial sums, each
  //    combined over the cluster in rank order
  const int n_loc = s_hi - s_lo;
  for (int h = 0; h < G; ++h) {
    float m = -CUDART_INF_F;
    for (int i = threadIdx.x; i < n_loc; i += DEC_THREADS) m = fmaxf(m, p[(size_t)h * part + i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red_v[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = red_v[0];
      for (int w = 1; w < DEC_THREADS / 32; ++w) t = fmaxf(t, red_v[w]);
      x_m[h] = t;
    }
    __syncthreads();
  }
  cluster.sync();
  if (threadIdx.x < G) {
    float t = -CUDART_INF_F;
    for (int c = 0; c < DEC_CLUSTER; ++c) t = fmaxf(t, *cluster.map_shared_rank(&x_m[threadIdx.x], c));
    s_m[threadIdx.x] = t;
  }
  __syncthreads();
  for (int h = 0; h < G; ++h) {
    const float m = s_m[h];
    float z = 0.f;
    for (int i = threadIdx.x; i < n_loc; i += DEC_THREADS) {
      const float e = exp2f(p[(size_t)h * part + i] - m);
      p[(size_t)h * part + i] = e;
      z += e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) red_v[warp] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int w = 0; w < DEC_THREADS / 32; ++w) t += red_v[w];
      x_z[h] = t;
    }
    __syncthreads();
  }
  cluster.sync();
  if (threadIdx.x < G) {
    float t = 0.f;
    for (int c = 0; c < DEC_CLUSTER; ++c) t += *cluster.map_shared_rank(&x_z[threadIdx.x], c);
    s_z[threadIdx.x] = t;
  }
  __syncthreads();
  // 4. group-mean attention of this CTA's slots into the work area (by slot)
  {
    float inv_z[G];
#pragma unroll
    for (int h = 0; h < G; ++h) inv_z[h] = s_z[h];
    for (int i = threadIdx.x; i < n_loc; i += DEC_THREADS) {
      float a = 0.f;
#pragma unroll
      for (int h = 0; h < G; ++h) a += p[(size_t)h * part + i] / inv_z[h];
      aslot[s_lo + i] = a * (1.f / (float)G);
    }
  }
  cluster.sync();                                    // every slot's value is written; sh is free
  // 5. this CTA's ranks: pooling along the rank order, score update, eviction candidate
  const int n_obs = cap - A.Sw;                      // entries outside the recent window
  const int n_old = len - A.Sw;                      // of which these already carry a score
  const int rad = A.kp >> 1;
  const int rpart = (n_obs + DEC_CLUSTER - 1) / DEC_CLUSTER;
  const int r_lo = min(n_obs, crank * rpart), r_hi = min(n_obs, r_lo + rpart);
  const int w_lo = max(0, r_lo - rad), w_hi = min(n_obs, r_hi + rad);
  float* abar = sh;                                  // ranks w_lo .. w_hi - 1
#pragma unroll 4
  for (int i = threadIdx.x; i < w_hi - w_lo; i += DEC_THREADS) abar[i] = aslot[A.order[base + w_lo + i]];
  __syncthreads();
  float worst = CUDART_INF_F;
  int worst_r = -1;
#pragma unroll 2
  for (int r = r_lo + threadIdx.x; r < r_hi; r += DEC_THREADS) {
    const int lo = max(0, r - rad), hi = min(n_obs, r + rad + 1);
    float v = abar[lo - w_lo];
    for (int x = lo + 1; x < hi; ++x) v = A.pool_mode == CAKE_POOL_MAX ? fmaxf(v, abar[x - w_lo]) : v + abar[x - w_lo];
    if (A.pool_mode != CAKE_POOL_MAX) v /= (float)A.kp;
    const int s = A.order[base + r];
    float sc = v;
    if (r < n_old) {
      const float old = A.score[base + s];
      sc = A.update_mode == CAKE_DECODE_ADD ? old + v : A.update_mode == CAKE_DECODE_MAX ? fmaxf(old, v) : v;
    }
    A.score[base + s] = sc;
    worse_of(worst, worst_r, sc, r);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, worst, o);
    const int oi = __shfl_xor_sync(0xffffffffu, worst_r, o);
    if (oi >= 0 && (worst_r < 0 || ov < worst || (ov == worst && oi > worst_r))) { worst = ov; worst_r = oi; }
  }
  if (lane == 0) { red_v[warp] = worst; red_i[warp] = worst_r; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float bv = CUDART_INF_F;
    int bi = -1;
    for (int w = 0; w < DEC_THREADS / 32; ++w)
      if (red_i[w] >= 0 && (bi < 0 || red_v[w] < bv || (red_v[w] == bv && red_i[w] > bi))) { bv = red_v[w]; bi = red_i[w]; }
    x_worst = bv;
    x_worst_r = bi;
  }
  cluster.sync();
  int ev = -1;
  if (n_obs > budget) {
    float bv = CUDART_INF_F;
    for (int c = 0; c < DEC_CLUSTER; ++c) {
      const float cv = *cluster.map_shared_rank(&x_worst, c);
      const int ci = *cluster.map_shared_rank(&x_worst_r, c);
      if (ci >= 0 && (ev < 0 || cv < bv || (cv == bv && ci > ev))) { bv = cv; ev = ci; }
    }
  }
  if (ev < 0) {                                      // below the budget: the cache would have to grow
    if (crank == 0 && threadIdx.x == 0) atomicCAS(A.status, 0, CAKE_ERR_CAPACITY);
    cluster.sync();                                  // nobody leaves while its candidate may still be read
    return;
  }
  // 6. ranks after the evicted one move down by one; its slot becomes the free one.  Every CTA
  //    reads the successors of its part of the list, the cluster meets, then it writes them.
  const int ev_slot = A.order[base + ev];
  const int m_lo = max(ev, min(cap - 1, crank * part)), m_hi = max(m_lo, min(cap - 1, crank * part + part));
  int* nxt = reinterpret_cast<int*>(sh);
#pragma unroll 4
  for (int i = threadIdx.x; i < m_hi - m_lo; i += DEC_THREADS) nxt[i] = A.order[base + m_lo + i + 1];
  cluster.sync();
#pragma unroll 4
  for (int i = threadIdx.x; i < m_hi - m_lo; i += DEC_THREADS) A.order[base + m_lo + i] = nxt[i];
  if (crank == 0 && threadIdx.x == 0) {
    A.order[base + cap - 1] = ev_slot;
    A.pos[base + ev_slot] = -1;
    A.meta[lid] = make_int4(len, ev_slot, next_pos + 1, budget);
  }
}

// Entries of one (request, layer) in ascending position: positions, scores (window entries 0),
// slots.  One CTA per head.
__global__ void decode_read_state(const int64_t* __restrict__ dec_off, const float* __restrict__ score,
                                  const int32_t* __restrict__ pos, const int32_t* __restrict__ order,
                                  const int4* __restrict__ meta, int32_t* __restrict__ pos_out,
                                  float* __restrict__ score_out, int32_t* __restrict__ slot_out,
                                  int blk, int Hkv, int Sw) {
  const int g = blockIdx.x;
  const int len = meta[(size_t)blk * Hkv + g].x;
  const int64_t base = dec_off[blk] + (int64_t)g * (len + 1);
  for (int r = threadIdx.x; r < len; r += blockDim.x) {
    const int s = order[base + r];
    if (pos_out) pos_out[(size_t)g * len + r] = pos[base + s];
    if (slot_out) slot_out[(size_t)g * len + r] = s;
    if (score_out) score_out[(size_t)g * len + r] = r < len - Sw ? score[base + s] : 0.f;
  }
}

// Rows of the packed order into the decode layout (one spare row per head).
__global__ void __launch_bounds__(256)
decode_gather(LayerPtrs ptrs, const int64_t* __restrict__ packed_off, const int64_t* __restrict__ dec_off,
              const int32_t* __restrict__ budget, const int32_t* __restrict__ pos_packed,
              const ReqInfo* __restrict__ reqs, uint4* __restrict__ k_out, uint4* __restrict__ v_out,
              int n_req, int L, int Hkv, int Sw, int64_t T, int cpr) {
  const int64_t total = packed_off[(size_t)n_req * L];
  const int nblk = n_req * L;
  const int64_t n_chunks = total * cpr;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_chunks;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / cpr;
    const int chunk = (int)(i - row * cpr);
    int lo = 0, hi = nblk - 1;                       // last block with offset <= row
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (packed_off[mid] <= row) lo = mid; else hi = mid - 1;
    }
    const int r = lo / L, l = lo - r * L;
    const int len = budget[lo] + Sw;
    const int64_t rel = row - packed_off[lo];
    const int g = (int)(rel / len);
    const int idx = (int)(rel - (int64_t)g * len);
    const size_t srow = ((size_t)g * T + reqs[r].cu + pos_packed[row]) * cpr + chunk;
    const size_t drow = (size_t)(dec_off[lo] + (int64_t)g * (len + 1) + idx) * cpr + chunk;
    k_out[drow] = reinterpret_cast<const uint4*>(ptrs.k[l])[srow];
    v_out[drow] = reinterpret_cast<const uint4*>(ptrs.v[l])[srow];
  }
}

template <typename T, int G>
cudaError_t launch_step_cluster_g(dim3 grid, size_t smem, cudaStream_t st, const DecodeArgs& A) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid.x * DEC_CLUSTER, grid.y, 1);
  cfg.blockDim = dim3(DEC_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = DEC_CLUSTER;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_step_cluster_kernel<T, G>, A);
}

template <typename T>
cudaError_t launch_step_cluster(int device, int G, dim3 grid, size_t smem, cudaStream_t st, const DecodeArgs& A) {
  static PerDeviceOnce attr;
  if (attr.need(device)) {
    cudaError_t e = cudaSuccess;
#define CAKE_DEC_ATTR(GG) \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_step_cluster_kernel<T, GG>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
    CAKE_DEC_ATTR(1); CAKE_DEC_ATTR(2); CAKE_DEC_ATTR(4); CAKE_DEC_ATTR(8);
#undef CAKE_DEC_ATTR
    if (e != cudaSuccess) return e;
    attr.mark(device);
  }
  switch (G) {
    case 1: return launch_step_cluster_g<T, 1>(grid, smem, st, A);
    case 2: return launch_step_cluster_g<T, 2>(grid, smem, st, A);
    case 4: return launch_step_cluster_g<T, 4>(grid, smem, st, A);
    case 8: return launch_step_cluster_g<T, 8>(grid, smem, st, A);
    default: return cudaErrorInvalidValue;
  }
}

template <typename T>
cudaError_t launch_step(int device, int G, dim3 grid, size_t smem, cudaStream_t st, const DecodeArgs& A) {
  static PerDeviceOnce attr;
  if (attr.need(device)) {
    cudaError_t e = cudaSuccess;
#define CAKE_DEC_ATTR(GG) \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_step_kernel<T, GG>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
    CAKE_DEC_ATTR(1); CAKE_DEC_ATTR(2); CAKE_DEC_ATTR(4); CAKE_DEC_ATTR(8);
#undef CAKE_DEC_ATTR
    if (e != cudaSuccess) return e;
    attr.mark(device);
  }
  switch (G) {
    case 1: decode_step_kernel<T, 1><<<grid, DEC_THREADS, smem, st>>>(A); break;
    case 2: decode_step_kernel<T, 2><<<grid, DEC_THREADS, smem, st>>>(A); break;
    case 4: decode_step_kernel<T, 4><<<grid, DEC_THREADS, smem, st>>>(A); break;
    case 8: decode_step_kernel<T, 8><<<grid, DEC_THREADS, smem, st>>>(A); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

int32_t run_sorted_positions_packed(cake_ctx* ctx, const int64_t* offsets, int32_t* out, cudaStream_t st);

int32_t launch_decode_begin(cake_ctx* ctx, const LayerPtrs& ptrs, void* k_cache, void* v_cache,
                            int64_t* row_offsets, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  const int32_t* budget = ctx->d_budget[(ctx->n_evicted - 1) & 1];
  decode_offsets<<<1, 32, 0, st>>>(budget, ctx->d_dec_off, ctx->n_req, c.n_layers, c.n_kv_heads, c.window);
  count_launch();
  if (row_offsets)
    CAKE_CUDA_TRY(cudaMemcpyAsync(row_offsets, ctx->d_dec_off, sizeof(int64_t) * (ctx->n_req * c.n_layers + 1),
                                  cudaMemcpyDeviceToDevice, st));
  if (ctx->n_req == 0) return cuda_status(cudaGetLastError());
  // positions in packed order (context scratch), then the decode state and the rows
  int32_t rc = run_sorted_positions_packed(ctx, ctx->d_dec_packed_off, ctx->d_pos_packed, st);
  if (rc != CAKE_OK) return rc;
  const dim3 grid(c.n_kv_heads, c.n_layers, ctx->n_req);
  decode_build<<<grid, DEC_THREADS, 0, st>>>(ctx->d_lists, ctx->d_prefix, ctx->d_lstate, ctx->d_req, budget,
                                             ctx->d_dec_packed_off, ctx->d_pos_packed, ctx->d_dec_off,
                                             ctx->d_dec_score, ctx->d_dec_pos, ctx->d_dec_order,
                                             ctx->d_dec_meta, c.n_layers, c.n_kv_heads, c.window);
  count_launch();
  const int esize = c.dtype == CAKE_DTYPE_FP32 ? 4 : 2;
  const int cpr = c.head_dim * esize / 16;
  decode_gather<<<ctx->n_sm * 8, 256, 0, st>>>(ptrs, ctx->d_dec_packed_off, ctx->d_dec_off, budget,
                                               ctx->d_pos_packed, ctx->d_req, (uint4*)k_cache, (uint4*)v_cache,
                                               ctx->n_req, c.n_layers, c.n_kv_heads, c.window,
                                               ctx->total_tokens, cpr);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int32_t launch_decode_step(cake_ctx* ctx, int32_t layer, const void* q_new, const void* k_new,
                           const void* v_new, void* k_cache, void* v_cache, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_req == 0) return CAKE_OK;
  const int G = c.n_q_heads / c.n_kv_heads;
  DecodeArgs A;
  A.q_new = q_new; A.k_new = k_new; A.v_new = v_new; A.k_cache = k_cache; A.v_cache = v_cache;
  A.dec_off = ctx->d_dec_off; A.score = ctx->d_dec_score; A.pos = ctx->d_dec_pos;
  A.order = ctx->d_dec_order; A.meta = ctx->d_dec_meta; A.status = ctx->d_status;
  A.layer = layer; A.L = c.n_layers; A.Hq = c.n_q_heads; A.Hkv = c.n_kv_heads; A.d = c.head_dim;
  A.Sw = c.window; A.kp = c.pool_kernel; A.pool_mode = c.pool_mode; A.update_mode = ctx->dec_update_mode;
  A.scale2 = 1.4426950408889634f / sqrtf((float)c.head_dim);
  // shared memory: (G + 1) floats per slot, sized for the largest head of the batch up to the
  // 200 KB the kernel may take; larger heads use the context's work area in global memory
  const int64_t limit = (200 * 1024) / ((int64_t)(G + 1) * (int64_t)sizeof(float));
  const int64_t cap = std::min<int64_t>(ctx->dec_max_cap, limit);
  const size_t smem = (size_t)(G + 1) * cap * sizeof(float);
  A.smem_cap = (int)cap;
  A.tmp = ctx->d_dec_tmp; A.reqs = ctx->d_req; A.T = ctx->total_tokens; A.n_req = ctx->n_req;
  const dim3 grid(c.n_kv_heads, ctx->n_req);
  // Large heads are spread over a cluster of DEC_CLUSTER CTAs each (CAKE_DECODE_CLUSTER=0 keeps
  // every head on one CTA): G floats per slot of a CTA's part, reused for the pooled window.
  const int64_t part = (ctx->dec_max_cap + DEC_CLUSTER - 1) / DEC_CLUSTER;
  const size_t smem_cl = ((size_t)G * part + (size_t)c.pool_kernel + 8) * sizeof(float);
  const char* env = getenv("CAKE_DECODE_CLUSTER");
  const bool use_cluster = ctx->dec_max_cap >= DEC_CLUSTER_MIN_CAP && smem_cl <= 200 * 1024 &&
                           !(env && env[0] == '0');
  cudaError_t e;
  if (use_cluster)
    e = c.dtype == CAKE_DTYPE_FP32 ? launch_step_cluster<float>(ctx->device, G, grid, smem_cl, st, A)
                                   : launch_step_cluster<__nv_bfloat16>(ctx->device, G, grid, smem_cl, st, A);
  else
    e = c.dtype == CAKE_DTYPE_FP32 ? launch_step<float>(ctx->device, G, grid, smem, st, A)
                                   : launch_step<__nv_bfloat16>(ctx->device, G, grid, smem, st, A);
  count_launch();
  return cuda_status(e);
}

int32_t launch_decode_read(cake_ctx* ctx, int32_t req, int32_t layer, int32_t* positions, float* scores,
                           int32_t* slots, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  decode_read_state<<<c.n_kv_heads, 256, 0, st>>>(ctx->d_dec_off, ctx->d_dec_score, ctx->d_dec_pos,
                                                  ctx->d_dec_order, ctx->d_dec_meta, positions, scores, slots,
                                                  req * c.n_layers + layer, c.n_kv_heads, c.window);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
