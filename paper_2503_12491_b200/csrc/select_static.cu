// A stand-alone per-head top-k selection that allocates nothing: the entry point for
// callers that must not touch the device allocator.  Its scratch (two bitmaps per head) lives
// in a fixed array inside the library instead of in memory obtained from cudaMalloc.
#include "cake_internal.cuh"

namespace cake {
namespace {

constexpr int SEL_THREADS = 1024;
constexpr int kSelMaxWords = 32768;            // 32-bit bitmap words: heads * ceil(n/32) at most

// Scratch shared by every call in the process: [2][kSelMaxWords] words = 256 KB per GPU that
// loads the library.  Half 0: keys above the threshold; half 1: keys equal to it.
static __device__ __align__(256) uint32_t g_select_scratch[2 * kSelMaxWords];

// Order-preserving integer image of a float; -0 and +0 compare equal, as they do as floats.
__device__ inline uint32_t sel_key(float v) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive scan of two counters packed as (hi: a, lo: b) over the block.
__device__ inline unsigned long long sel_scan(unsigned long long v, unsigned long long* warp_tot) {
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
    const unsigned long long w = warp_tot[lane];
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_tot[lane] = winc - w;
  }
  __syncthreads();
  return warp_tot[warp] + inc - v;
}

// One CTA per head: keeps the `keep` entries that come first in the order (value descending,
// position ascending) -- the TopK of Eq. 12 -- and writes their positions in ascending order.
__global__ void __launch_bounds__(SEL_THREADS)
select_positions_static(const float* __restrict__ values, int n, int keep,
                        int32_t* __restrict__ out, uint32_t* __restrict__ scratch, int words) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_krem;
  __shared__ unsigned long long warp_tot[32];
  const int head = blockIdx.x;
  const float* v = values + (size_t)head * n;
  uint32_t* gt = scratch + (size_t)head * words;
  uint32_t* eq = scratch + kSelMaxWords + (size_t)head * words;
  int32_t* dst = out + (size_t)head * keep;
  // the array keeps whatever the previous call left in it
  for (int w = threadIdx.x; w < words; w += SEL_THREADS) { gt[w] = 0; eq[w] = 0; }
  // radix select of the keep-th largest key, 8 bits per pass from the top
  uint32_t prefix = 0, mask = 0, krem = (uint32_t)keep;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = threadIdx.x; b < 256; b += SEL_THREADS) hist[b] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
      const uint32_t key = sel_key(v[j]);
      if ((key & mask) == prefix) {
        atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
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
  const uint32_t thr = prefix;        // key of the keep-th largest entry
  const uint32_t need_eq = krem;      // entries equal to it that are kept: the lowest positions
  for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
    const uint32_t key = sel_key(v[j]);
    if (key > thr) atomicOr(&gt[j >> 5], 1u << (j & 31));
    else if (key == thr) atomicOr(&eq[j >> 5], 1u << (j & 31));
  }
  __threadfence_block();
  __syncthreads();
  // ranks: every thread owns a run of words
  const int per = (words + SEL_THREADS - 1) / SEL_THREADS;
  const int w0 = min(words, (int)threadIdx.x * per), w1 = min(words, w0 + per);
  uint32_t cg = 0, ce = 0;
  for (int w = w0; w < w1; ++w) { cg += __popc(gt[w]); ce += __popc(eq[w]); }
  const unsigned long long ex = sel_scan(((unsigned long long)cg << 32) | ce, warp_tot);
  uint32_t g_before = (uint32_t)(ex >> 32), e_before = (uint32_t)(ex & 0xffffffffu);
  for (int w = w0; w < w1; ++w) {
    const uint32_t mg = gt[w], me = eq[w];
    uint32_t m = mg | me;
    while (m) {
      const int bit = __ffs(m) - 1;
      m &= m - 1;
      if ((mg >> bit) & 1u) {
        dst[g_before + min(e_before, need_eq)] = (w << 5) + bit;
        ++g_before;
      } else {
        if (e_before < need_eq) dst[g_before + e_before] = (w << 5) + bit;
        ++e_before;
      }
    }
  }
}

constexpr int kMaxDevices = 64;
uint32_t* g_scratch_ptr[kMaxDevices];     // device address of the scratch, per device ordinal

}  // namespace
}  // namespace cake

extern "C" int32_t cake_select_positions_static(const float* values, int32_t n_heads, int32_t n,
                                                int32_t keep, int32_t* positions_out, void* stream) {
  using namespace cake;
  if (n_heads < 0 || n < 0 || keep < 0 || keep > n) return CAKE_ERR_ARG;
  if (n_heads == 0 || keep == 0) return CAKE_OK;
  if (!values || !positions_out) return CAKE_ERR_ARG;
  const int words = (n + 31) / 32;
  if ((int64_t)n_heads * words > kSelMaxWords) return CAKE_ERR_CAPACITY;
  int dev = -1;
  CAKE_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return CAKE_ERR_ARG;
  if (!g_scratch_ptr[dev]) {
    // In host code the array's name is only a handle; the kernel needs its device address.
    uint32_t* p = nullptr;
    CAKE_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_select_scratch));
    g_scratch_ptr[dev] = p;
  }
  select_positions_static<<<n_heads, SEL_THREADS, 0, (cudaStream_t)stream>>>(
      values, n, keep, positions_out, g_scratch_ptr[dev], words);
  count_launch();
  return cuda_status(cudaGetLastError());
}
