// Window-score kernels for bf16 inputs on the sm_100a tensor cores.
//
// Both passes stream K tiles of 128 keys through shared memory with TMA
// (no multicast), multiply them against the resident window queries with
// tcgen05.mma (bf16 operands, fp32 accumulators in tensor memory) and reduce
// the accumulator tile on chip; the S_w x N score matrix never reaches HBM.
//
//   pass A (rows)   D[row][key]  = Q K^T : one thread owns one window row and
//                   keeps its running max / sum (softmax denominator, Eq. 2) and
//                   sum e*log2(e) (row entropy, Eq. 4).
//   pass B (cols)   D[key][row]  = K Q^T : one thread owns one key and reduces its
//                   normalised column over the window rows: group-mean attention,
//                   Mean + gamma Var (Eq. 11) and the per-head Var (Eq. 5).
//
// Warp roles in a CTA of 320 threads: warp 0 issues TMA loads, warp 1 owns the
// tensor-memory allocation and issues the MMAs, warps 2..9 are two groups of
// four "statistics" warps that take alternate accumulator tiles.  Every wait on
// an mbarrier is bounded; a timed-out wait raises CAKE_ERR_TIMEOUT and the CTA
// drains and exits.
#include "cake_internal.cuh"

#include <cuda.h>
#include <math_constants.h>

namespace cake {
namespace {

constexpr int TILE = 128;            // keys per tile
constexpr int STAGES = 4;            // K tiles in flight
constexpr int NBUF = 4;              // accumulator buffers (4 x 128 of the 512 TMEM columns)
constexpr int TC_THREADS = 320;
constexpr int SLAB_BYTES = TILE * 128;   // one 64-element slab of a 128-row tile
constexpr long long kSpinLimit = 4000000000ll;   // cycles (~2 s) before a wait gives up
constexpr float kLog2e = 1.4426950408889634f;

struct TcParams {
  const TcSegment* segs;
  const int32_t* cta_seg;       // [n_cta + 1]
  const ReqInfo* reqs;
  float* lse2;                  // [req][H_kv][128] in tile row order r' = i*G + h
  float4* rowpart;              // pass A out: [segment][128] (m, z_all, z_win, w)
  float* raw;                   // pass B out: [H_kv][T]
  float* colpart;               // pass B out: [segment][G][2]
  int32_t* status;
  int64_t T;
  int Hkv, G, Sw, rows, d;
  float scale2, gamma, bessel;
};

// ------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.b32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false (and the sticky status set) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kSpinLimit) {
      atomicCAS(status, 0, CAKE_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0,
                                            int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void named_bar(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)(1024u >> 4) << 32;                 // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                            // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct Smem {
  uint8_t* q;          // 2 slabs x 128 rows x 128 B
  uint8_t* k;          // STAGES x (2 slabs x 128 rows x 128 B)
  uint64_t* full;      // [STAGES]
  uint64_t* empty;     // [STAGES]
  uint64_t* acc_full;  // [NBUF]
  uint64_t* acc_empty; // [NBUF]
  uint64_t* q_full;
  uint64_t* q_empty;
  uint32_t* tmem_holder;
  float* lse;          // [128]
  float* xchg;         // [128 * 4]
};

constexpr size_t kSmemBytes = 1024 /*align*/ + 2 * SLAB_BYTES + (size_t)STAGES * 2 * SLAB_BYTES + 256 +
                              128 * 4 + 128 * 16 + 64;

__device__ __forceinline__ Smem carve(uint8_t* base) {
  Smem s;
  uint8_t* p = (uint8_t*)(((uintptr_t)base + 1023) & ~(uintptr_t)1023);
  s.q = p;                    p += 2 * SLAB_BYTES;
  s.k = p;                    p += (size_t)STAGES * 2 * SLAB_BYTES;
  s.full = (uint64_t*)p;      p += 8 * STAGES;
  s.empty = (uint64_t*)p;     p += 8 * STAGES;
  s.acc_full = (uint64_t*)p;  p += 8 * NBUF;
  s.acc_empty = (uint64_t*)p; p += 8 * NBUF;
  s.q_full = (uint64_t*)p;    p += 8;
  s.q_empty = (uint64_t*)p;   p += 8;
  s.tmem_holder = (uint32_t*)p; p += 16;
  p = (uint8_t*)(((uintptr_t)p + 15) & ~(uintptr_t)15);
  s.lse = (float*)p;          p += 128 * 4;
  s.xchg = (float*)p;
  return s;
}

// ------------------------------------------------------------------ kernel
template <bool kCols, bool kEntropy>
__global__ void __launch_bounds__(TC_THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const TcParams P) {
  extern __shared__ uint8_t smem_raw[];
  const Smem S = carve(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_slab = P.d / 64;
  const uint32_t stage_bytes = (uint32_t)(TILE * P.d * 2);
  const int rows_pad = (P.rows + 15) & ~15;
  const int seg_lo = P.cta_seg[blockIdx.x], seg_hi = P.cta_seg[blockIdx.x + 1];

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&S.full[i], 1); mbar_init(&S.empty[i], 1); }
    for (int i = 0; i < NBUF; ++i) { mbar_init(&S.acc_full[i], 1); mbar_init(&S.acc_empty[i], 128); }
    mbar_init(S.q_full, 1);
    mbar_init(S.q_empty, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of the query tile that TMA never writes must read as zero
  for (int i = threadIdx.x; i < 2 * SLAB_BYTES / 16; i += TC_THREADS)
    reinterpret_cast<uint4*>(S.q)[i] = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(S.tmem_holder)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *S.tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&k_map) : "memory");
      uint32_t t = 0, qn = 0;
      bool ok = true;
      for (int sg = seg_lo; sg < seg_hi && ok; ++sg) {
        const TcSegment seg = P.segs[sg];
        const ReqInfo rq = P.reqs[seg.req];
        const int nkeys = kCols ? min(seg.nkeys, rq.n - seg.key0) : seg.nkeys;
        if (nkeys <= 0) continue;
        // previous segment's MMAs must be done with the query tile
        ok = mbar_wait(S.q_empty, (qn & 1) ^ 1, P.status);
        ++qn;
        if (!ok) break;
        mbar_expect_tx(S.q_full, (uint32_t)(P.rows * P.d * 2));
        for (int sl = 0; sl < n_slab; ++sl)
          tma_load_4d(S.q + sl * SLAB_BYTES, &q_map, S.q_full, sl * 64, seg.g * P.G, 0, seg.req);
        const int64_t row0 = (int64_t)seg.g * P.T + rq.cu + seg.key0;
        const int ntiles = (nkeys + TILE - 1) / TILE;
        for (int it = 0; it < ntiles; ++it, ++t) {
          const int s = t % STAGES;
          ok = mbar_wait(&S.empty[s], ((t / STAGES) & 1) ^ 1, P.status);
          if (!ok) break;
          mbar_expect_tx(&S.full[s], stage_bytes);
          uint8_t* dst = S.k + (size_t)s * 2 * SLAB_BYTES;
          for (int sl = 0; sl < n_slab; ++sl)
            tma_load_2d(dst + sl * SLAB_BYTES, &k_map, &S.full[s], sl * 64, (int)(row0 + it * TILE));
        }
      }
      // do not leave the CTA while a bulk copy may still be writing its shared memory
      const uint32_t issued = t;
      for (uint32_t u = issued > STAGES ? issued - STAGES : 0; u < issued; ++u)
        mbar_wait(&S.full[u % STAGES], (u / STAGES) & 1, P.status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = kCols ? instr_desc(128, rows_pad) : instr_desc(128, TILE);
      uint32_t t = 0, qn = 0;
      bool ok = true;
      for (int sg = seg_lo; sg < seg_hi && ok; ++sg) {
        const TcSegment seg = P.segs[sg];
        const ReqInfo rq = P.reqs[seg.req];
        const int nkeys = kCols ? min(seg.nkeys, rq.n - seg.key0) : seg.nkeys;
        if (nkeys <= 0) continue;
        ok = mbar_wait(S.q_full, qn & 1, P.status);
        ++qn;
        if (!ok) break;
        const int ntiles = (nkeys + TILE - 1) / TILE;
        for (int it = 0; it < ntiles; ++it, ++t) {
          const int s = t % STAGES, b = t % NBUF;
          ok = mbar_wait(&S.acc_empty[b], ((t / NBUF) & 1) ^ 1, P.status);
          if (!ok) break;
          ok = mbar_wait(&S.full[s], (t / STAGES) & 1, P.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t kaddr = smem_u32(S.k + (size_t)s * 2 * SLAB_BYTES);
          const uint32_t qaddr = smem_u32(S.q);
          const uint32_t tmem_d = tmem_base + (uint32_t)(b * 128);
          for (int sl = 0; sl < n_slab; ++sl) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t kd = smem_desc(kaddr + sl * SLAB_BYTES + ks * 32);
              const uint64_t qd = smem_desc(qaddr + sl * SLAB_BYTES + ks * 32);
              if (kCols) umma_bf16(tmem_d, kd, qd, idesc, (sl | ks) != 0);
              else       umma_bf16(tmem_d, qd, kd, idesc, (sl | ks) != 0);
            }
          }
          umma_commit(&S.empty[s]);
          umma_commit(&S.acc_full[b]);
        }
        umma_commit(S.q_empty);        // query tile free once every MMA of the segment has run
      }
    }
  } else {
    // ------------------------------------------------ statistics warps
    const int wg = (warp - 2) >> 2;                 // 0 or 1: takes tiles of matching parity
    const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
    const int lane_row = quad * 32 + lane;          // accumulator lane (row in pass A, key in pass B)
    const int sthread = threadIdx.x - 64;           // 0..255 among the statistics threads
    uint32_t t = 0;
    bool ok = true;
    for (int sg = seg_lo; sg < seg_hi; ++sg) {
      const TcSegment seg = P.segs[sg];
      const ReqInfo rq = P.reqs[seg.req];
      const int nkeys = kCols ? min(seg.nkeys, rq.n - seg.key0) : seg.nkeys;
      const int ntiles = nkeys > 0 ? (nkeys + TILE - 1) / TILE : 0;
      if (kCols) {
        // ---------------- pass B: thread = key, columns = rows r' = i*G + h
        named_bar(1, 256);                          // previous segment done with S.lse / S.xchg
        if (sthread < 128)
          S.lse[sthread] = sthread < P.rows
              ? P.lse2[((size_t)seg.req * P.Hkv + seg.g) * 128 + sthread] : 0.f;
        named_bar(1, 256);
        float vacc[8], hs[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) { vacc[h] = 0.f; hs[h] = 0.f; }
        const float inv_sw = 1.f / (float)P.Sw, inv_g = 1.f / (float)P.G;
        for (int it = 0; it < ntiles; ++it, ++t) {
          if ((int)(t & 1) != wg) continue;
          const int b = t % NBUF;
          if (ok) ok = mbar_wait(&S.acc_full[b], (t / NBUF) & 1, P.status);
          if (!ok) continue;
          tc_fence_after();
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * 128);
          float s1[8], s2[8], a1 = 0.f, a2 = 0.f, hkeep[8];
#pragma unroll
          for (int h = 0; h < 8; ++h) { s1[h] = 0.f; s2[h] = 0.f; hkeep[h] = hs[h]; }
          for (int c0 = 0; c0 < P.rows; c0 += 32) {
            float v[32];
            tmem_ld32(taddr + c0, v);
            // 32 columns = 32/G window rows x G heads
            if (P.G == 4) {
#pragma unroll
              for (int ii = 0; ii < 8; ++ii) {
                const float4 l4 = *reinterpret_cast<const float4*>(&S.lse[c0 + ii * 4]);
                const float t0 = fmaf(v[ii * 4 + 0], P.scale2, -l4.x);
                const float t1 = fmaf(v[ii * 4 + 1], P.scale2, -l4.y);
                const float t2 = fmaf(v[ii * 4 + 2], P.scale2, -l4.z);
                const float t3 = fmaf(v[ii * 4 + 3], P.scale2, -l4.w);
                const float p0 = ex2(t0), p1 = ex2(t1), p2 = ex2(t2), p3 = ex2(t3);
                if (kEntropy) {
                  hs[0] = fmaf(p0, t0, hs[0]); hs[1] = fmaf(p1, t1, hs[1]);
                  hs[2] = fmaf(p2, t2, hs[2]); hs[3] = fmaf(p3, t3, hs[3]);
                }
                s1[0] += p0; s2[0] = fmaf(p0, p0, s2[0]);
                s1[1] += p1; s2[1] = fmaf(p1, p1, s2[1]);
                s1[2] += p2; s2[2] = fmaf(p2, p2, s2[2]);
                s1[3] += p3; s2[3] = fmaf(p3, p3, s2[3]);
                const float a = ((p0 + p1) + (p2 + p3)) * inv_g;
                a1 += a; a2 = fmaf(a, a, a2);
              }
            } else {
              // generic group size (1, 2 or 8): column c = i*G + h
              for (int e = 0; e < 32; e += P.G) {
                float a = 0.f;
                for (int h = 0; h < P.G; ++h) {
                  const float tt = fmaf(v[e + h], P.scale2, -S.lse[c0 + e + h]);
                  const float p = ex2(tt);
#pragma unroll
                  for (int hh = 0; hh < 8; ++hh)
                    if (hh == h) {
                      s1[hh] += p; s2[hh] = fmaf(p, p, s2[hh]);
                      if (kEntropy) hs[hh] = fmaf(p, tt, hs[hh]);
                    }
                  a += p;
                }
                a *= inv_g;
                a1 += a; a2 = fmaf(a, a, a2);
              }
            }
          }
          tc_fence_before();
          mbar_arrive(&S.acc_empty[b]);
          const int j = seg.key0 + it * TILE + lane_row;          // key index inside the request
          if (j < rq.n && it * TILE + lane_row < nkeys) {
            const float mean = a1 * inv_sw;
            const float var = fmaxf(a2 * inv_sw - mean * mean, 0.f) * P.bessel;
            P.raw[(size_t)seg.g * P.T + rq.cu + j] = fmaf(P.gamma, var, mean);
#pragma unroll
            for (int h = 0; h < 8; ++h) {
              const float mh = s1[h] * inv_sw;
              vacc[h] += fmaxf(s2[h] * inv_sw - mh * mh, 0.f) * P.bessel;
            }
          } else {
#pragma unroll
            for (int h = 0; h < 8; ++h) hs[h] = hkeep[h];      // key outside the observed range
          }
        }
        // fixed-order reduction of vacc over the 256 statistics threads
        named_bar(1, 256);
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          float x = vacc[h], y = hs[h];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            x += __shfl_xor_sync(0xffffffffu, x, o);
            y += __shfl_xor_sync(0xffffffffu, y, o);
          }
          if (lane == 0) { S.xchg[(warp - 2) * 16 + h] = x; S.xchg[(warp - 2) * 16 + 8 + h] = y; }
        }
        named_bar(1, 256);
        if (sthread < P.G) {
          float acc = 0.f, hacc = 0.f;
          for (int w2 = 0; w2 < 8; ++w2) {
            acc += S.xchg[w2 * 16 + sthread];
            hacc += S.xchg[w2 * 16 + 8 + sthread];
          }
          P.colpart[((size_t)sg * P.G + sthread) * 2 + 0] = hacc;
          P.colpart[((size_t)sg * P.G + sthread) * 2 + 1] = acc;
        }
      } else {
        // ---------------- pass A: thread = window row r' = i*G + h, columns = keys
        const int i_row = lane_row / P.G;
        const int last = rq.n + i_row;                 // last key this row may attend to
        float m = -CUDART_INF_F, z = 0.f, zwin = 0.f, w = 0.f;
        for (int it = 0; it < ntiles; ++it, ++t) {
          if ((int)(t & 1) != wg) continue;
          const int b = t % NBUF;
          if (ok) ok = mbar_wait(&S.acc_full[b], (t / NBUF) & 1, P.status);
          if (!ok) continue;
          tc_fence_after();
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * 128);
          const int key0 = seg.key0 + it * TILE;
          const bool interior = key0 + TILE <= rq.n && it * TILE + TILE <= nkeys;
#pragma unroll 1
          for (int c0 = 0; c0 < TILE; c0 += 32) {
            float v[32];
            tmem_ld32(taddr + c0, v);
            if (interior) {
              float cm = v[0];
#pragma unroll
              for (int e = 1; e < 32; ++e) cm = fmaxf(cm, v[e]);
              const float mn = fmaxf(m, cm * P.scale2);
              const float f = ex2(m - mn);                     // 0 on the first chunk
              const float dm = (m == -CUDART_INF_F) ? 0.f : (m - mn);
              w = f * fmaf(dm, z - zwin, w);
              z *= f; zwin *= f;
              m = mn;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float tt = fmaf(v[e], P.scale2, -m);
                const float ee = ex2(tt);
                z += ee;
                w = fmaf(ee, tt, w);
              }
            } else {
              float cm = -CUDART_INF_F;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int j = key0 + c0 + e;
                const bool vis = (it * TILE + c0 + e < nkeys) && j <= last;
                cm = vis ? fmaxf(cm, v[e]) : cm;
              }
              if (cm != -CUDART_INF_F) {
                const float mn = fmaxf(m, cm * P.scale2);
                const float f = ex2(m - mn);
                const float dm = (m == -CUDART_INF_F) ? 0.f : (m - mn);
                w = f * fmaf(dm, z - zwin, w);
                z *= f; zwin *= f;
                m = mn;
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  const int j = key0 + c0 + e;
                  const bool vis = (it * TILE + c0 + e < nkeys) && j <= last;
                  const bool obs = j < rq.n;
                  const float tt = fmaf(v[e], P.scale2, -m);
                  const float ee = vis ? ex2(tt) : 0.f;
                  z += ee;
                  zwin += obs ? 0.f : ee;
                  w = (vis && obs) ? fmaf(ee, tt, w) : w;
                }
              }
            }
          }
          tc_fence_before();
          mbar_arrive(&S.acc_empty[b]);
        }
        // merge the two groups' partial rows, group 0 writes
        named_bar(1, 256);
        if (wg == 1) {
          reinterpret_cast<float4*>(S.xchg)[lane_row] = make_float4(m, z, zwin, w);
        }
        named_bar(1, 256);
        if (wg == 0) {
          const float4 o = reinterpret_cast<const float4*>(S.xchg)[lane_row];
          float mn = fmaxf(m, o.x);
          float4 outv = make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);
          if (mn != -CUDART_INF_F) {
            const float fa = (m == -CUDART_INF_F) ? 0.f : ex2(m - mn);
            const float fb = (o.x == -CUDART_INF_F) ? 0.f : ex2(o.x - mn);
            const float da = (m == -CUDART_INF_F) ? 0.f : (m - mn);
            const float db = (o.x == -CUDART_INF_F) ? 0.f : (o.x - mn);
            outv.x = mn;
            outv.y = z * fa + o.y * fb;
            outv.z = zwin * fa + o.z * fb;
            outv.w = fa * fmaf(da, z - zwin, w) + fb * fmaf(db, o.y - o.z, o.w);
          }
          P.rowpart[(size_t)sg * 128 + lane_row] = outv;
        }
      }
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512)
                 : "memory");
  }
}

// Merge the row partials of every (request, KV head): lse2 per row and the
// entropy per query head.  Rows are in tile order r' = i*G + h.
__global__ void tc_rowstats_combine(const float4* __restrict__ rowpart,
                                    const int32_t* __restrict__ pair_seg,
                                    float* __restrict__ lse2, double* __restrict__ hhead, int Hkv,
                                    int G, int rows, int Hq) {
  __shared__ float hrow[128];
  const int req = blockIdx.x, g = blockIdx.y, r = threadIdx.x;
  const int pair = req * Hkv + g;
  float m = -CUDART_INF_F, z = 0.f, zw = 0.f, w = 0.f;
  for (int sg = pair_seg[pair]; sg < pair_seg[pair + 1]; ++sg) {
    const float4 p = rowpart[(size_t)sg * 128 + r];
    if (p.x == -CUDART_INF_F) continue;
    const float mn = fmaxf(m, p.x);
    const float fa = (m == -CUDART_INF_F) ? 0.f : exp2f(m - mn);
    const float fb = exp2f(p.x - mn);
    const float da = (m == -CUDART_INF_F) ? 0.f : (m - mn);
    const float db = p.x - mn;
    w = fa * fmaf(da, z - zw, w) + fb * fmaf(db, p.y - p.z, p.w);
    z = z * fa + p.y * fb;
    zw = zw * fa + p.z * fb;
    m = mn;
  }
  float h = 0.f;
  if (r < rows) {
    const float lz = log2f(z);
    lse2[(size_t)pair * 128 + r] = m + lz;
    // sum_j p log2 p = (w - log2(z) * z_obs) / z
    h = (w - lz * (z - zw)) / z;
  }
  hrow[r] = h;
  __syncthreads();
  if (r < G) {                                  // head h = rows r, r+G, r+2G, ...
    double acc = 0.0;
    for (int i = r; i < rows; i += G) acc += (double)hrow[i];
    hhead[(size_t)req * Hq + g * G + r] = -0.6931471805599453 * acc;
  }
}

// External natural-log LSE [req][H_q][S_w] -> base-2, tile row order.
__global__ void tc_lse_permute(const float* __restrict__ lse, float* __restrict__ lse2, int Hkv, int G,
                               int Sw) {
  const int req = blockIdx.x, g = blockIdx.y, r = threadIdx.x;
  if (r >= G * Sw) return;
  const int i = r / G, h = r - i * G;
  lse2[((size_t)req * Hkv + g) * 128 + r] =
      lse[((size_t)req * Hkv * G + g * G + h) * Sw + i] * kLog2e;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

}  // namespace

bool tc_path_supported(const cake_config& c) {
  const int G = c.n_q_heads / c.n_kv_heads;
  const int rows = G * c.window;
  return c.dtype == CAKE_DTYPE_BF16 && (c.head_dim == 64 || c.head_dim == 128) && rows % 32 == 0 &&
         rows <= 128 && (G == 1 || G == 2 || G == 4 || G == 8) && c.window <= 256;
}

int32_t launch_score_tc(cake_ctx* ctx, const void* q_win, const void* k, const float* lse,
                        cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_tc_segs == 0) return CAKE_OK;
  if ((int64_t)c.n_kv_heads * ctx->total_tokens >= ((int64_t)1 << 31)) return CAKE_ERR_ARG;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return CAKE_ERR_CUDA;
  const int G = c.n_q_heads / c.n_kv_heads;
  CUtensorMap qmap, kmap;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)c.head_dim, (cuuint64_t)c.n_kv_heads * ctx->total_tokens};
    const cuuint64_t strides[1] = {(cuuint64_t)c.head_dim * 2};
    const cuuint32_t box[2] = {64, TILE};
    const cuuint32_t es[2] = {1, 1};
    if (enc(&kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(k), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return CAKE_ERR_CUDA;
  }
  {
    // [req][head][i][d] viewed as (d, head, i, req) so that a box lands as rows r' = i*G + h
    const cuuint64_t dims[4] = {(cuuint64_t)c.head_dim, (cuuint64_t)c.n_q_heads, (cuuint64_t)c.window,
                                (cuuint64_t)ctx->n_req};
    const cuuint64_t strides[3] = {(cuuint64_t)c.window * c.head_dim * 2, (cuuint64_t)c.head_dim * 2,
                                   (cuuint64_t)c.n_q_heads * c.window * c.head_dim * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)c.window, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    if (enc(&qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q_win), dims, strides, box,
            es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return CAKE_ERR_CUDA;
  }
  static bool attr_done = false;
  if (!attr_done) {
    CAKE_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<false, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    CAKE_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<true, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    CAKE_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<true, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    attr_done = true;
  }
  TcParams P;
  P.segs = ctx->d_tc_segs;
  P.cta_seg = ctx->d_tc_cta_seg;
  P.reqs = ctx->d_req;
  P.lse2 = ctx->d_lse2_tc;
  P.rowpart = ctx->d_tc_rowpart;
  P.raw = ctx->d_raw;
  P.colpart = ctx->d_colpart;
  P.status = ctx->d_status;
  P.T = ctx->total_tokens;
  P.Hkv = c.n_kv_heads; P.G = G; P.Sw = c.window; P.rows = ctx->rows; P.d = c.head_dim;
  P.scale2 = kLog2e / sqrtf((float)c.head_dim);
  P.gamma = c.gamma;
  P.bessel = c.var_ddof ? (float)c.window / (float)(c.window - 1) : 1.f;

  const dim3 pairs(ctx->n_req, c.n_kv_heads);
  int sp = prof_begin(ctx, CAKE_PROF_SCORE_ROWS, st);
  if (lse) {
    tc_lse_permute<<<pairs, 128, 0, st>>>(lse, ctx->d_lse2_tc, c.n_kv_heads, G, c.window);
    CAKE_CUDA_TRY(cudaMemsetAsync(ctx->d_hhead, 0, sizeof(double) * ctx->n_req * c.n_q_heads, st));
    count_launch();
    ctx->hhead_from_rows = false;
  } else {
    score_tc_kernel<false, false><<<ctx->n_tc_ctas, TC_THREADS, kSmemBytes, st>>>(qmap, kmap, P);
    tc_rowstats_combine<<<pairs, 128, 0, st>>>(ctx->d_tc_rowpart, ctx->d_tc_pair_seg, ctx->d_lse2_tc,
                                               ctx->d_hhead, c.n_kv_heads, G, ctx->rows, c.n_q_heads);
    count_launch(2);
    ctx->hhead_from_rows = true;
  }
  prof_end(ctx, sp, st);
  sp = prof_begin(ctx, CAKE_PROF_SCORE_COLS, st);
  if (lse) score_tc_kernel<true, true><<<ctx->n_tc_ctas, TC_THREADS, kSmemBytes, st>>>(qmap, kmap, P);
  else     score_tc_kernel<true, false><<<ctx->n_tc_ctas, TC_THREADS, kSmemBytes, st>>>(qmap, kmap, P);
  count_launch();
  prof_end(ctx, sp, st);
  return cuda_status(cudaGetLastError());
}

}  // namespace cake
