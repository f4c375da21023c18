// Window-score kernel for bf16 inputs on the sm_100a tensor cores: one persistent
// launch per layer runs both passes over the keys.
//
//   pass A (rows)   D[row][key]  = Q K^T : one thread owns one window row and keeps
//                   its running max / sum (softmax denominator, Eq. 2) and
//                   sum e*log2(e) (row entropy, Eq. 4).
//   pass B (cols)   D[key][row]  = K Q^T : one thread owns one key and reduces its
//                   normalised column over the window rows: group-mean attention,
//                   Mean + gamma Var (Eq. 11) and the per-head Var (Eq. 5).
//
// K tiles of 128 keys stream through shared memory with TMA (no multicast), are
// multiplied against the resident window queries with tcgen05.mma (bf16 operands,
// fp32 accumulators in tensor memory) and reduced on chip; the S_w x N score matrix
// never reaches HBM.
//
// Schedule.  The (request, KV head) pairs of a layer are grouped into waves of at
// most kWaveBytes of K.  Every CTA owns the same slice of a wave in both passes and runs
//     A(wave 0), A(wave 1), B(wave 0), A(wave 2), B(wave 1), ... , B(last wave)
// so pass B re-reads a wave's K from L2 shortly after pass A brought it in, and DRAM
// sees K once.  Pass B of a pair needs the pair's softmax denominators, i.e. every
// CTA's pass-A partial rows.  The merge is spread over the grid by rows: the merger warp
// of CTA (pair * rows + r) % grid waits until all partials of the pair are delivered, loads
// row r's partials in a single round trip, merges them and counts the row as done.  The pass A
// of the next wave sits between a pair's pass A and its pass B, so pass B's wait on
// that count is normally already satisfied.
//
// Warp roles in a CTA of 512 threads: warps 0..11 are "statistics" warps in three groups of
// four (a group takes every third accumulator tile, a warp owns 32 of its TMEM lanes, works
// alone and writes its own partial results), warp 12 issues TMA loads, warp 13 owns the
// tensor-memory allocation and issues the MMAs (both as converged warps with an elected lane),
// warp 14 publishes this CTA's finished pass-A ops to the grid and merges rows, warp 15 stages
// the denominators of the next pass-B op in shared memory.  Every wait
// (mbarrier or flag) is bounded; a timed-out wait raises CAKE_ERR_TIMEOUT and the CTA
// drains and exits.
#include "cake_internal.cuh"

#include <cuda.h>
#include <math_constants.h>

#include <algorithm>
#include <cstring>
#include <vector>

namespace cake {
namespace {

constexpr int TILE = 128;            // keys per tile
constexpr int STAGES = 4;            // K tiles in flight
constexpr int NBUF = 3;              // accumulator buffers: 3 x 128 of the 512 TMEM columns
constexpr int TMEM_Q_COL = NBUF * 128;   // + 64 columns: the window queries as pass A's A operand
constexpr int NWG = kScoreGroups;    // statistics warp groups
static_assert(NWG == NBUF, "one accumulator buffer per statistics group");
static_assert(NWG * 4 <= 16, "a_done holds one counter per statistics warp");
constexpr int STAT_THREADS = NWG * 128;
constexpr int TC_THREADS = STAT_THREADS + 128;  // + TMA, MMA, row-merger and denominator warps
constexpr int WARP_TMA = NWG * 4, WARP_MMA = NWG * 4 + 1, WARP_MERGE = NWG * 4 + 2,
              WARP_LSE = NWG * 4 + 3;
constexpr int NSTATW = NWG * 4;      // statistics warps
constexpr int SLAB_BYTES = TILE * 128;   // one 64-element slab of a 128-row tile
constexpr long long kSpinLimit = 4000000000ll;   // default cycles (~2 s) before a wait gives up
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kChunkSumMax = 65536.f;   // a pass-A chunk sum beyond this moves the row's reference
constexpr int64_t kWaveBytes = 32ll << 20;
constexpr int kWaveDepth = 1;         // pass B of a wave follows pass A of the wave this far ahead

struct TcParams {
  const ScoreOp* ops;
  const int32_t* cta_op;        // [n_cta + 1]
  const ReqInfo* reqs;
  const int32_t* pair_aseg;     // [pairs + 1] pass-A segment ranges per pair
  uint32_t* pair_cnt;           // [pairs] delivered pass-A partials (monotonic over layers)
  uint32_t* pair_done;          // [pairs] merged rows (monotonic over layers); null = pass B only
  float* lse2;                  // [pair][128] in tile row order r' = i*G + h
  const float* lse_ext;         // caller's natural-log LSE [req][H_q][S_w], or null
  float4* rowpart;              // pass A out: [A-segment][group][128] (m, z_all, z_win, w)
  float* raw;                   // pass B out: [H_kv][T]
  float* colpart;               // pass B out: [B-segment][statistics warp][G][2]
  float* hrow;                  // [pair][128] sum_j p log2 p of every window row
  int32_t* status;
  int64_t T;
  uint32_t epoch;
  long long spin_limit;         // cycles after which a wait gives up and raises CAKE_ERR_TIMEOUT
  int n_pairs;
  int Hkv, Hq, Sw, rows, d;
  float scale2, inv_scale2, gamma, bessel;
  int ind_mode;                 // CAKE_IND_*
  int merge_ways;               // rows the merger warp merges side by side: 1, or 2 to 32 when pairs are short
};

// ------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{\n.reg .pred e;\nelect.sync _|e, 0xffffffff;\n"
               "@e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n}" ::"r"(smem_u32(bar)),
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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int32_t* status,
                                          long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) {
      atomicCAS(status, 0, CAKE_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}
// 3-D tiled TMA load with an L2 eviction-priority hint: a whole key tile (both 64-element slabs)
// in one copy.
__device__ __forceinline__ void tma_load_3d_hint(void* dst, const CUtensorMap* map, uint64_t* bar,
                                                 int c0, int c1, int c2, uint64_t policy) {
  asm volatile(
      "{\n.reg .pred e;\nelect.sync _|e, 0xffffffff;\n"
      "@e cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5}], [%2], %6;\n}"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "{\n.reg .pred e;\nelect.sync _|e, 0xffffffff;\n"
      "@e cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n}"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// The MMA and TMA warps run converged, all 32 lanes executing the same loop, and one elected lane
// issues each asynchronous instruction.  Issued from inside a one-lane branch the operands of
// every tcgen05.mma are moved to uniform registers one by one and an M128 x N128 x K16 MMA costs
// about 70 cycles to issue, more than the 64 cycles it takes to execute; from a converged warp
// the descriptor arithmetic stays in the uniform datapath and the tensor pipe sets the pace.
// Descriptors differ only in the 14-bit address field of their low word, the high word (stride,
// version, swizzle) is a constant, and the accumulate flag is an immediate.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // SBO, version 1, SWIZZLE_128B
template <int kAcc>
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
  asm volatile(
      "{\n.reg .pred p, e;\n.reg .b64 da, db;\nsetp.ne.b32 p, %4, 0;\nelect.sync _|e, 0xffffffff;\n"
      "mov.b64 da, {%1, %5};\nmov.b64 db, {%2, %5};\n"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}"
      ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "n"(kAcc), "r"(kDescHi)
      : "memory");
}
template <int kAcc>
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_lo, uint32_t idesc) {
  asm volatile(
      "{\n.reg .pred p, e;\n.reg .b64 db;\nsetp.ne.b32 p, %4, 0;\nelect.sync _|e, 0xffffffff;\n"
      "mov.b64 db, {%2, %5};\n"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n}"
      ::"r"(tmem_d), "r"(tmem_a), "r"(b_lo), "r"(idesc), "n"(kAcc), "r"(kDescHi)
      : "memory");
}
// The same with an explicit high descriptor word: operands that are not in the 128-byte swizzle.
template <int kAcc>
__device__ __forceinline__ void umma_ss_hi(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                           uint32_t hi) {
  asm volatile(
      "{\n.reg .pred p, e;\n.reg .b64 da, db;\nsetp.ne.b32 p, %4, 0;\nelect.sync _|e, 0xffffffff;\n"
      "mov.b64 da, {%1, %5};\nmov.b64 db, {%2, %5};\n"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}"
      ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "n"(kAcc), "r"(hi)
      : "memory");
}
// Pass B folds the rows' log-sum-exps into the contraction: one more K = 16 step whose key-side
// operand holds 1 in its first three columns and whose row-side operand holds -lse / scale split
// into three bf16 terms, so the accumulator is (q.k - lse/scale) and the statistics warps neither
// load nor subtract anything per logit.  These two operands are 128 rows x 16 bf16 in the
// K-major layout without swizzle: 8-row x 16-byte core matrices, the two core matrices of a row
// group 128 bytes apart (leading-dimension offset), row groups 256 bytes apart (stride offset).
constexpr uint32_t kExtBytes = 128 * 32;
constexpr uint32_t kExtDescHi = (256u >> 4) | (1u << 14);            // SBO, version 1, no swizzle
constexpr uint32_t kExtDescLoLbo = (128u >> 4) << 16;                // LBO field of the low word
__device__ __forceinline__ uint32_t ext_row_offset(int r) { return (uint32_t)((r >> 3) * 256 + (r & 7) * 16); }

// Copies 128 rows x 32 bytes (one K = 16 slice of a K-major operand) from shared to tensor memory.
__device__ __forceinline__ void tmem_cp_128x256b(uint32_t tmem_dst, uint64_t sdesc) {
  asm volatile("{\n.reg .pred e;\nelect.sync _|e, 0xffffffff;\n@e tcgen05.cp.cta_group::1.128x256b [%0], %1;\n}"
               ::"r"(tmem_dst), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("{\n.reg .pred e;\nelect.sync _|e, 0xffffffff;\n"
               "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}"
               ::"r"(smem_u32(bar)) : "memory");
}
// Starts the load of 32 consecutive fp32 columns of this thread's TMEM lane; the registers
// are valid only after tmem_ld_wait on the same array.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
// Waits for the thread's outstanding TMEM loads.  The registers pass through the statement so
// that no use of them can be scheduled before it.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two fp32 values in one 64-bit register and the packed fp32x2 arithmetic on them: one
// instruction issue for two FMAs or adds.  The statistics loops are bound by issue slots, not by
// the FMA pipe, so halving their FFMA/FADD count matters although the pipe rate is the same.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
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

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Counters in shared memory that only grow, each written by one warp: a wait for "at least v"
// cannot mistake one round for another, whoever waits and however late.
__device__ __forceinline__ void smem_store_release(uint32_t* c, uint32_t v) {
  asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(c)), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t smem_count_acquire(const uint32_t* c) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(c)) : "memory");
  return v;
}

struct Smem {
  uint8_t* q;          // 2 buffers x (2 slabs x 128 rows x 128 B)
  uint8_t* k;          // STAGES x (2 slabs x 128 rows x 128 B)
  uint64_t* full;      // [STAGES]
  uint64_t* empty;     // [STAGES]
  uint64_t* acc_full;  // [NBUF]
  uint64_t* acc_empty; // [NBUF]
  uint64_t* q_full;    // [2]
  uint64_t* q_empty;   // [2]
  uint64_t* lse_full;  // [2]
  uint64_t* lse_free;  // [2]
  uint32_t* tmem_holder;
  uint32_t* a_done;    // [NSTATW] pass-A ops whose partial rows each statistics warp has written
  uint8_t* ext_a;      // the constant key-side operand of the extra K step of pass B
  uint8_t* ext_b;      // [2] its row-side operand: -lse/scale of the current / next pass-B op
  ScoreOp* ops;        // [kSmemOps] the first ops of this CTA's program
};

constexpr size_t kQBytes = 2 * SLAB_BYTES;
constexpr int kSmemOps = 128;        // ops of a CTA's program kept in shared memory
constexpr size_t kSmemBytes = 1024 /*align*/ + 2 * kQBytes + (size_t)STAGES * 2 * SLAB_BYTES + 320 +
                              128 + 3 * kExtBytes + kSmemOps * sizeof(ScoreOp) + 64;

__device__ __forceinline__ Smem carve(uint8_t* base) {
  Smem s;
  uint8_t* p = (uint8_t*)(((uintptr_t)base + 1023) & ~(uintptr_t)1023);
  s.q = p;                    p += 2 * kQBytes;
  s.k = p;                    p += (size_t)STAGES * 2 * SLAB_BYTES;
  s.full = (uint64_t*)p;      p += 8 * STAGES;
  s.empty = (uint64_t*)p;     p += 8 * STAGES;
  s.acc_full = (uint64_t*)p;  p += 8 * NBUF;
  s.acc_empty = (uint64_t*)p; p += 8 * NBUF;
  s.q_full = (uint64_t*)p;    p += 16;
  s.q_empty = (uint64_t*)p;   p += 16;
  s.lse_full = (uint64_t*)p;  p += 16;
  s.lse_free = (uint64_t*)p;  p += 16;
  s.tmem_holder = (uint32_t*)p; p += 8;
  s.a_done = (uint32_t*)p;    p += 4 * 16;
  p = (uint8_t*)(((uintptr_t)p + 15) & ~(uintptr_t)15);
  p = (uint8_t*)(((uintptr_t)p + 127) & ~(uintptr_t)127);
  s.ext_a = p;                p += kExtBytes;
  s.ext_b = p;                p += 2 * kExtBytes;
  s.ops = (ScoreOp*)p;
  return s;
}

// Merge of two partial softmax rows (m, z_all, z_win, w) with base-2 exponents;
// w = sum over observed keys of e * (logit2 - m).
__device__ __forceinline__ float4 merge_rows(float4 a, float4 b) {
  if (b.x == -CUDART_INF_F) return a;
  if (a.x == -CUDART_INF_F) return b;
  const float mn = fmaxf(a.x, b.x);
  const float fa = exp2f(a.x - mn), fb = exp2f(b.x - mn);
  float4 o;
  o.x = mn;
  o.y = a.y * fa + b.y * fb;
  o.z = a.z * fa + b.z * fb;
  o.w = fa * fmaf(a.x - mn, a.y - a.z, a.w) + fb * fmaf(b.x - mn, b.y - b.z, b.w);
  return o;
}

// ------------------------------------------------------------------ kernel
template <int G, bool kEntropyB>
__global__ void __launch_bounds__(TC_THREADS, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                   const TcParams P) {
  extern __shared__ uint8_t smem_raw[];
  const Smem S = carve(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_slab = P.d / 64;
  const uint32_t stage_bytes = (uint32_t)(TILE * P.d * 2);
  const int rows_pad = (P.rows + 15) & ~15;
  const int op_lo = P.cta_op[blockIdx.x], op_hi = P.cta_op[blockIdx.x + 1];

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&S.full[i], 1); mbar_init(&S.empty[i], 1); }
    for (int i = 0; i < NBUF; ++i) { mbar_init(&S.acc_full[i], 1); mbar_init(&S.acc_empty[i], 4); }
    for (int i = 0; i < 2; ++i) { mbar_init(&S.q_full[i], 1); mbar_init(&S.q_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&S.lse_full[i], 1); mbar_init(&S.lse_free[i], 1); }
    for (int i = 0; i < NSTATW; ++i) S.a_done[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the program of this CTA: a global read per op would put an L2 round trip on every op
  for (int i = threadIdx.x; i < min(op_hi - op_lo, kSmemOps); i += TC_THREADS) S.ops[i] = P.ops[op_lo + i];
  auto get_op = [&](int oi) -> ScoreOp {
    return oi - op_lo < kSmemOps ? S.ops[oi - op_lo] : P.ops[oi];
  };
  // rows of the query tiles that TMA never writes must read as zero
  for (int i = threadIdx.x; i < (int)(2 * kQBytes / 16); i += TC_THREADS)
    reinterpret_cast<uint4*>(S.q)[i] = make_uint4(0, 0, 0, 0);
  // operands of the extra K step: zero, then ones in the first three columns of the key side
  for (int i = threadIdx.x; i < (int)(3 * kExtBytes / 16); i += TC_THREADS)
    reinterpret_cast<uint4*>(S.ext_a)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (threadIdx.x < 128)
    *reinterpret_cast<uint2*>(S.ext_a + ext_row_offset(threadIdx.x)) = make_uint2(0x3F803F80u, 0x00003F80u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == WARP_MMA) {
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

  if (warp == WARP_TMA) {
    // ------------------------------------------------ TMA producer (converged warp, elected lane issues)
    {
      if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&k_map) : "memory");
      }
      __syncwarp();
      // pass A's tiles are read again by pass B: keep them in L2; pass B's read is the last
      const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
      uint32_t t = 0, qn = 0;
      bool ok = true;
      for (int oi = op_lo; oi < op_hi && ok; ++oi) {
        const ScoreOp op = get_op(oi);
        if (op.nkeys <= 0) continue;
        const uint64_t pol = (op.phase || !P.pair_done) ? drop : keep;
        const int qb = qn & 1;
        // the MMAs of the op that used this query buffer two ops ago must be done
        ok = mbar_wait(&S.q_empty[qb], ((qn >> 1) & 1) ^ 1, P.status, P.spin_limit);
        ++qn;
        if (!ok) break;
        mbar_expect_tx(&S.q_full[qb], (uint32_t)(P.rows * P.d * 2));
        for (int sl = 0; sl < n_slab; ++sl)
          tma_load_4d(S.q + qb * kQBytes + sl * SLAB_BYTES, &q_map, &S.q_full[qb], sl * 64, op.g * G,
                      0, op.req);
        const int64_t row0 = op.base + op.key0;
        const int ntiles = (op.nkeys + TILE - 1) / TILE;
        for (int it = 0; it < ntiles; ++it, ++t) {
          const int s = t % STAGES;
          ok = mbar_wait(&S.empty[s], ((t / STAGES) & 1) ^ 1, P.status, P.spin_limit);
          if (!ok) break;
          mbar_expect_tx(&S.full[s], stage_bytes);
          uint8_t* dst = S.k + (size_t)s * 2 * SLAB_BYTES;
          // the map's dimensions are (64 elements, key rows, slabs): the box lands slab by slab
          tma_load_3d_hint(dst, &k_map, &S.full[s], 0, (int)(row0 + it * TILE), 0, pol);
        }
      }
      // do not leave the CTA while a bulk copy may still be writing its shared memory
      const uint32_t issued = t;
      for (uint32_t u = issued > STAGES ? issued - STAGES : 0; u < issued; ++u)
        mbar_wait(&S.full[u % STAGES], (u / STAGES) & 1, P.status, P.spin_limit);
      for (uint32_t u = qn > 2 ? qn - 2 : 0; u < qn; ++u)
        mbar_wait(&S.q_full[u & 1], (u >> 1) & 1, P.status, P.spin_limit);
    }
  } else if (warp == WARP_MMA) {
    // ------------------------------------------------ MMA issuer (converged warp, elected lane issues)
    {
      uint32_t t = 0, qn = 0, kbm = 0;
      const uint32_t k_lo0 = (smem_u32(S.k) & 0x3FFFFu) >> 4;
      const uint32_t ext_a_lo = ((smem_u32(S.ext_a) & 0x3FFFFu) >> 4) | kExtDescLoLbo;
      bool ok = true;
      for (int oi = op_lo; oi < op_hi && ok; ++oi) {
        const ScoreOp op = get_op(oi);
        if (op.nkeys <= 0) continue;
        const uint32_t idesc = op.phase ? instr_desc(128, rows_pad) : instr_desc(128, TILE);
        const int eslot = kbm & 1;
        const uint32_t ext_b_lo = ((smem_u32(S.ext_b + eslot * kExtBytes) & 0x3FFFFu) >> 4) | kExtDescLoLbo;
        const int qb = qn & 1;
        ok = mbar_wait(&S.q_full[qb], (qn >> 1) & 1, P.status, P.spin_limit);
        ++qn;
        if (!ok) break;
        const uint32_t qaddr = smem_u32(S.q + qb * kQBytes);
        const uint32_t q_lo = (qaddr & 0x3FFFFu) >> 4;      // address field of the descriptors
        const uint32_t tmem_q = tmem_base + (uint32_t)TMEM_Q_COL;
        if (!op.phase) {
          // pass A multiplies every key tile by the same queries: hold them in tensor memory, so
          // that an MMA reads only the key tile from shared memory.  The copies run in issue
          // order behind the previous op's MMAs and ahead of this op's.
          tc_fence_after();
          for (int sl = 0; sl < n_slab; ++sl)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              tmem_cp_128x256b(tmem_q + (uint32_t)((sl * 4 + ks) * 8),
                               smem_desc(qaddr + sl * SLAB_BYTES + ks * 32));
        }
        if (op.phase) {
          // the rows' -lse/scale operand of this op (written by the denominator warp)
          ok = mbar_wait(&S.lse_full[eslot], (kbm >> 1) & 1, P.status, P.spin_limit);
          if (!ok) break;
        }
        const int ntiles = (op.nkeys + TILE - 1) / TILE;
        for (int it = 0; it < ntiles; ++it, ++t) {
          const int s = t % STAGES, b = t % NBUF;
          ok = mbar_wait(&S.acc_empty[b], ((t / NBUF) & 1) ^ 1, P.status, P.spin_limit);
          if (!ok) break;
          ok = mbar_wait(&S.full[s], (t / STAGES) & 1, P.status, P.spin_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + (uint32_t)s * (uint32_t)((2 * SLAB_BYTES) >> 4);
          const uint32_t tmem_d = tmem_base + (uint32_t)(b * 128);
          if (op.phase) {
            // D[key][row] = K Q^T
            umma_ss<0>(tmem_d, k_lo, q_lo, idesc);
            umma_ss<1>(tmem_d, k_lo + 2, q_lo + 2, idesc);
            umma_ss<1>(tmem_d, k_lo + 4, q_lo + 4, idesc);
            umma_ss<1>(tmem_d, k_lo + 6, q_lo + 6, idesc);
            if (n_slab == 2) {
              constexpr uint32_t o = SLAB_BYTES >> 4;
              umma_ss<1>(tmem_d, k_lo + o, q_lo + o, idesc);
              umma_ss<1>(tmem_d, k_lo + o + 2, q_lo + o + 2, idesc);
              umma_ss<1>(tmem_d, k_lo + o + 4, q_lo + o + 4, idesc);
              umma_ss<1>(tmem_d, k_lo + o + 6, q_lo + o + 6, idesc);
            }
            umma_ss_hi<1>(tmem_d, ext_a_lo, ext_b_lo, idesc, kExtDescHi);      // ... - lse/scale
          } else {
            // D[row][key] = Q K^T, queries from tensor memory
            umma_ts<0>(tmem_d, tmem_q, k_lo, idesc);
            umma_ts<1>(tmem_d, tmem_q + 8, k_lo + 2, idesc);
            umma_ts<1>(tmem_d, tmem_q + 16, k_lo + 4, idesc);
            umma_ts<1>(tmem_d, tmem_q + 24, k_lo + 6, idesc);
            if (n_slab == 2) {
              constexpr uint32_t o = SLAB_BYTES >> 4;
              umma_ts<1>(tmem_d, tmem_q + 32, k_lo + o, idesc);
              umma_ts<1>(tmem_d, tmem_q + 40, k_lo + o + 2, idesc);
              umma_ts<1>(tmem_d, tmem_q + 48, k_lo + o + 4, idesc);
              umma_ts<1>(tmem_d, tmem_q + 56, k_lo + o + 6, idesc);
            }
          }
          umma_commit(&S.empty[s]);
          umma_commit(&S.acc_full[b]);
        }
        umma_commit(&S.q_empty[qb]);     // query buffer free once every MMA of the op has run
        if (op.phase) {
          umma_commit(&S.lse_free[eslot]);   // and so is the op's -lse/scale operand
          ++kbm;
        }
      }
    }
  } else if (warp == WARP_MERGE) {
    // ------------------------------------------------ row merger
    // Every (pair, row) is merged by one CTA of the grid: once all partials of the pair have
    // been delivered, the warp loads the row's partials in one round trip, merges them in a
    // fixed order and publishes the row's base-2 log-sum-exp and entropy term.
    if (P.pair_done) {
      bool ok = true;
      // Publishes, in program order, every pass-A op of this CTA whose twelve partial row sets
      // are written: one fence, then the op's count goes to its pair.
      int pub_oi = op_lo;
      uint32_t pub = 0;
      auto publish = [&]() -> bool {               // true once every pass-A op is published
        while (pub_oi < op_hi) {
          const ScoreOp o = get_op(pub_oi);
          if (o.nkeys <= 0 || o.phase) { ++pub_oi; continue; }
          // every statistics warp counts its own finished pass-A ops: a warp whose group has
          // no tile in an op runs ahead of the others, so a single shared count of arrivals
          // could be reached before the slowest warp has written this op's rows
          const uint32_t mine = lane < NSTATW ? smem_count_acquire(&S.a_done[lane]) : 0xFFFFFFFFu;
          if (!__all_sync(0xffffffffu, mine >= pub + 1u)) return false;
          __threadfence();
          if (lane == 0) atomicAdd(&P.pair_cnt[o.req * P.Hkv + o.g], (uint32_t)NSTATW);
          ++pub;
          ++pub_oi;
        }
        return true;
      };
      if (P.merge_ways > 1) {
        // Short pairs (a ragged batch, MHA): a wave holds several pairs whose rows have few
        // partials each, so the rows of `ways` (2 to 32) consecutive pairs are merged side by side,
        // by 32 / ways lanes each, and the wave's denominators are ready that much sooner.
        const int ways = P.merge_ways, lpr = 32 / ways;         // lanes per row
        const int sub = lane / lpr, l8 = lane % lpr;
        for (int p0 = 0; p0 < P.n_pairs && ok; p0 += ways) {
          const int pair = p0 + sub;
          const bool have = pair < P.n_pairs;
          const int s_lo = have ? P.pair_aseg[pair] * NWG : 0, s_hi = have ? P.pair_aseg[pair + 1] * NWG : 0;
          const int r0 = have ? (int)((blockIdx.x + gridDim.x - (unsigned)(((long long)pair * P.rows) % gridDim.x)) % gridDim.x)
                              : P.rows;
          bool waited = false;
          for (int r = r0;; r += gridDim.x) {
            const bool active = have && r < P.rows;
            if (!__any_sync(0xffffffffu, active)) break;
            if (!waited) {
              const uint32_t want = (uint32_t)(s_hi - s_lo) * 4u * P.epoch;
              const long long t0 = clock64();
              for (;;) {
                const bool ready = !active || ld_acquire(&P.pair_cnt[pair]) >= want;
                if (__all_sync(0xffffffffu, ready)) break;
                publish();
                if (clock64() - t0 > P.spin_limit) { atomicCAS(P.status, 0, CAKE_ERR_TIMEOUT); ok = false; break; }
                __nanosleep(100);
              }
              if (!ok) break;
              waited = true;
            }
            float4 acc = make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);
            if (active) {
              for (int base = s_lo; base < s_hi; base += 8 * lpr) {
                float4 pv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const int sg = base + u * lpr + l8;
                  pv[u] = sg < s_hi ? __ldcg(&P.rowpart[(size_t)sg * 128 + r])
                                    : make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) acc = merge_rows(acc, pv[u]);
              }
            }
            for (int o = lpr >> 1; o > 0; o >>= 1) {           // inside the lanes of a row
              float4 other;
              other.x = __shfl_xor_sync(0xffffffffu, acc.x, o);
              other.y = __shfl_xor_sync(0xffffffffu, acc.y, o);
              other.z = __shfl_xor_sync(0xffffffffu, acc.z, o);
              other.w = __shfl_xor_sync(0xffffffffu, acc.w, o);
              acc = (lane & o) ? merge_rows(other, acc) : merge_rows(acc, other);
            }
            if (active && l8 == 0) {
              const float lz = log2f(acc.y);
              __stcg(&P.lse2[(size_t)pair * 128 + r], acc.x + lz);
              __stcg(&P.hrow[(size_t)pair * 128 + r], (acc.w - lz * (acc.y - acc.z)) / acc.y);
              __threadfence();
              atomicAdd(&P.pair_done[pair], 1u);
            }
          }
        }
      } else
      for (int pair = 0; pair < P.n_pairs && ok; ++pair) {
        const int s_lo = P.pair_aseg[pair] * NWG, s_hi = P.pair_aseg[pair + 1] * NWG;
        bool waited = false;
        // row r of pair p belongs to CTA (p * rows + r) % grid: with many short pairs every CTA
        // gets a few (pair, row) items instead of the first `rows` CTAs getting all of them
        const int r0 = (int)((blockIdx.x + gridDim.x - (unsigned)(((long long)pair * P.rows) % gridDim.x)) % gridDim.x);
        for (int r = r0; r < P.rows; r += gridDim.x) {
          if (!waited) {
            const uint32_t want = (uint32_t)(s_hi - s_lo) * 4u * P.epoch;   // one per warp
            const long long t0 = clock64();
            while (ld_acquire(&P.pair_cnt[pair]) < want) {
              publish();
              if (clock64() - t0 > P.spin_limit) { atomicCAS(P.status, 0, CAKE_ERR_TIMEOUT); ok = false; break; }
              __nanosleep(40);
            }
            if (!ok) break;
            waited = true;
          }
          float4 acc = make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);
          // 12 loads per lane in flight: the 384 partials of a row at 128 CTAs come in one round trip
          for (int base = s_lo; base < s_hi; base += 32 * 12) {
            float4 pv[12];
#pragma unroll
            for (int u = 0; u < 12; ++u) {
              const int sg = base + u * 32 + lane;
              pv[u] = sg < s_hi ? __ldcg(&P.rowpart[(size_t)sg * 128 + r])
                                : make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 12; ++u) acc = merge_rows(acc, pv[u]);
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            float4 other;
            other.x = __shfl_xor_sync(0xffffffffu, acc.x, o);
            other.y = __shfl_xor_sync(0xffffffffu, acc.y, o);
            other.z = __shfl_xor_sync(0xffffffffu, acc.z, o);
            other.w = __shfl_xor_sync(0xffffffffu, acc.w, o);
            // the lower lane's partial always goes first, so every lane gets the same result
            acc = (lane & o) ? merge_rows(other, acc) : merge_rows(acc, other);
          }
          if (lane == 0) {
            const float lz = log2f(acc.y);
            __stcg(&P.lse2[(size_t)pair * 128 + r], acc.x + lz);
            // sum_j p log2 p over the observed keys = (w - log2(z) * z_obs) / z
            __stcg(&P.hrow[(size_t)pair * 128 + r], (acc.w - lz * (acc.y - acc.z)) / acc.y);
            __threadfence();
            atomicAdd(&P.pair_done[pair], 1u);
          }
        }
      }
      // ops that finish after this warp's last merge
      const long long t0 = clock64();
      while (ok && !publish()) {
        if (clock64() - t0 > P.spin_limit) { atomicCAS(P.status, 0, CAKE_ERR_TIMEOUT); break; }
        __nanosleep(100);
      }
    }
  } else if (warp == WARP_LSE) {
    // ------------------------------------------------ denominator fetcher
    // For every pass-B op of this CTA, in program order: wait until all rows of the op's pair
    // are merged, copy the pair's 128 denominators into a two-slot shared-memory ring.
    uint32_t kb = 0;
    bool ok = true;
    for (int oi = op_lo; oi < op_hi && ok; ++oi) {
      const ScoreOp op = get_op(oi);
      if (op.nkeys <= 0 || !op.phase) continue;
      const int slot = kb & 1;
      const int pair = op.req * P.Hkv + op.g;
      if (lane == 0) {
        ok = mbar_wait(&S.lse_free[slot], ((kb >> 1) & 1) ^ 1, P.status, P.spin_limit);
        if (ok && P.pair_done) {
          const uint32_t want = (uint32_t)P.rows * P.epoch;
          const long long t0 = clock64();
          while (ld_acquire(&P.pair_done[pair]) < want) {
            if (clock64() - t0 > P.spin_limit) { atomicCAS(P.status, 0, CAKE_ERR_TIMEOUT); ok = false; break; }
            __nanosleep(32);
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      float4 v;
      if (P.lse_ext) {
        // the caller's natural-log values [req][H_q][S_w]: tile row r' = i*G + h, base 2
        float x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = 4 * lane + e, i = r / G, h = r - i * G;
          x[e] = r < P.rows ? __ldg(&P.lse_ext[((size_t)op.req * P.Hq + op.g * G + h) * P.Sw + i]) * kLog2e : 0.f;
        }
        v = make_float4(x[0], x[1], x[2], x[3]);
      } else {
        v = __ldcg(reinterpret_cast<const float4*>(P.lse2 + (size_t)pair * 128) + lane);
      }
      // -lse / scale as three bf16 terms (24 bits) in columns 0..2 of the rows' operand
      {
        const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = 4 * lane + e;
          const float t = -vv[e] * P.inv_scale2;
          const __nv_bfloat16 hi = __float2bfloat16_rn(t);
          const float r1 = t - __bfloat162float(hi);
          const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
          const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
          const uint32_t w0 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
          const uint32_t w1 = (uint32_t)__bfloat16_as_ushort(lo);
          *reinterpret_cast<uint2*>(S.ext_b + slot * kExtBytes + ext_row_offset(r)) =
              r < P.rows ? make_uint2(w0, w1) : make_uint2(0u, 0u);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&S.lse_full[slot]);
      ++kb;
    }
  } else {
    // ------------------------------------------------ statistics warps
    // Every warp works alone: it owns TMEM lanes 32*quad.. of the tiles its group takes, writes
    // its own partial results and never waits for another statistics warp.
    // Group wg takes the tiles t with t % NWG == wg; with as many buffers as groups that is
    // always buffer wg, whose "ready" barrier the group then meets in consecutive phases.
    const int wg = warp >> 2;
    const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
    const int lane_row = quad * 32 + lane;          // accumulator lane (row in pass A, key in pass B)
    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(wg * 128);
    uint64_t* const my_full = &S.acc_full[wg];
    uint64_t* const my_empty = &S.acc_empty[wg];
    const int b = wg;
    (void)b;
    uint32_t tmod = 0;                              // tiles of the ops so far, modulo NWG
    uint32_t fpar = 0;                              // phase parity of my_full
    uint32_t n_a_done = 0;                          // pass-A ops this warp has delivered
    bool ok = true;
    for (int oi = op_lo; oi < op_hi; ++oi) {
      const ScoreOp op = get_op(oi);
      if (op.nkeys <= 0) continue;
      const int ntiles = (op.nkeys + TILE - 1) / TILE;
      const int it0 = (int)((wg + NWG - tmod) % NWG);            // the group's first tile of the op
      tmod = (tmod + (uint32_t)ntiles) % NWG;
      if (op.phase) {
        // ---------------- pass B: thread = key, columns = rows r' = i*G + h
        float vacc[G], hs[G];
#pragma unroll
        for (int h = 0; h < G; ++h) { vacc[h] = 0.f; hs[h] = 0.f; }
        const float inv_sw = 1.f / (float)P.Sw, inv_g = 1.f / (float)G;
        for (int it = it0; it < ntiles; it += NWG) {
          if (ok) ok = mbar_wait(my_full, fpar, P.status, P.spin_limit);
          fpar ^= 1u;
          if (!ok) continue;
          tc_fence_after();
          float s1[G], s2[G], hk[G], a2 = 0.f;
#pragma unroll
          for (int h = 0; h < G; ++h) { s1[h] = 0.f; s2[h] = 0.f; hk[h] = 0.f; }
          f32x2 s1p[(G + 1) / 2], s2p[(G + 1) / 2], hkp[(G + 1) / 2];   // the same, two heads per register
#pragma unroll
          for (int hp = 0; hp < (G + 1) / 2; ++hp) { s1p[hp] = 0ull; s2p[hp] = 0ull; hkp[hp] = 0ull; }
          for (int c0 = 0; c0 < P.rows; c0 += 32) {
            uint32_t r[32];
            tmem_ld32_issue(taddr + c0, r);
            tmem_ld_wait(r);
            if (c0 + 32 >= P.rows) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(my_empty);
            }
            // 32 columns = 32/G window rows x G heads; the accumulator is q.k - lse/scale
            if constexpr (G % 2 == 0) {
              // two heads per instruction
              const f32x2 sc2 = pack2(P.scale2, P.scale2);
#pragma unroll
              for (int ii = 0; ii < 32 / G; ++ii) {
                f32x2 asum = 0ull;
#pragma unroll
                for (int hp = 0; hp < G / 2; ++hp) {
                  const int c = ii * G + 2 * hp;
                  const f32x2 tt2 = mul2(pack2(__uint_as_float(r[c]), __uint_as_float(r[c + 1])), sc2);
                  float t0, t1;
                  unpack2(tt2, t0, t1);
                  const f32x2 p2 = pack2(ex2(t0), ex2(t1));
                  s1p[hp] = add2(s1p[hp], p2);
                  s2p[hp] = fma2(p2, p2, s2p[hp]);
                  if (kEntropyB) hkp[hp] = fma2(p2, tt2, hkp[hp]);
                  asum = hp == 0 ? p2 : add2(asum, p2);
                }
                float a0, a1;
                unpack2(asum, a0, a1);
                const float a = a0 + a1;
                a2 = fmaf(a, a, a2);
              }
            } else {
#pragma unroll
              for (int ii = 0; ii < 32 / G; ++ii) {
                float a = 0.f;
#pragma unroll
                for (int h = 0; h < G; ++h) {
                  const float tt = __uint_as_float(r[ii * G + h]) * P.scale2;
                  const float p = ex2(tt);
                  s1[h] += p;
                  s2[h] = fmaf(p, p, s2[h]);
                  if (kEntropyB) hk[h] = fmaf(p, tt, hk[h]);
                  a += p;
                }
                a2 = fmaf(a, a, a2);
              }
            }
          }
          if constexpr (G % 2 == 0) {
#pragma unroll
            for (int hp = 0; hp < G / 2; ++hp) {
              unpack2(s1p[hp], s1[2 * hp], s1[2 * hp + 1]);
              unpack2(s2p[hp], s2[2 * hp], s2[2 * hp + 1]);
              if (kEntropyB) unpack2(hkp[hp], hk[2 * hp], hk[2 * hp + 1]);
            }
          }
          const int j = op.key0 + it * TILE + lane_row;          // key index inside the request
          if (j < op.n && it * TILE + lane_row < op.nkeys) {
            float a1 = 0.f;
#pragma unroll
            for (int h = 0; h < G; ++h) {
              a1 += s1[h];
              const float mh = s1[h] * inv_sw;
              vacc[h] += fmaxf(s2[h] * inv_sw - mh * mh, 0.f) * P.bessel;
              if (kEntropyB) hs[h] += hk[h];
            }
            const float mean = a1 * inv_g * inv_sw;
            const float var = fmaxf(a2 * inv_g * inv_g * inv_sw - mean * mean, 0.f) * P.bessel;
            P.raw[op.base + j] = combine_indicator(P.ind_mode, P.gamma, mean, var, (float)P.Sw);
          }
        }
        // fixed-order reduction over the warp's keys
#pragma unroll
        for (int h = 0; h < G; ++h) {
          float x = vacc[h], y = hs[h];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            x += __shfl_xor_sync(0xffffffffu, x, o);
            if (kEntropyB) y += __shfl_xor_sync(0xffffffffu, y, o);
          }
          if (lane == h) {
            float* dst = P.colpart + (((size_t)op.seg * NSTATW + warp) * G + h) * 2;
            dst[0] = y;
            dst[1] = x;
          }
        }
      } else {
        // ---------------- pass A: thread = window row r' = i*G + h, columns = keys
        const int i_row = lane_row / G;
        const int last = op.n + i_row;                 // last key this row may attend to
        float m = -CUDART_INF_F, z = 0.f, zwin = 0.f, w = 0.f;
        for (int it = it0; it < ntiles; it += NWG) {
          if (ok) ok = mbar_wait(my_full, fpar, P.status, P.spin_limit);
          fpar ^= 1u;
          if (!ok) continue;
          tc_fence_after();
          const int key0 = op.key0 + it * TILE;
          const bool interior = key0 + TILE <= op.n && it * TILE + TILE <= op.nkeys;
          if (quad * 32 >= P.rows) {                   // these TMEM lanes hold padding rows
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(my_empty);
            continue;
          }
#pragma unroll 1
          for (int c0 = 0; c0 < TILE; c0 += 32) {
            uint32_t r[32];
            tmem_ld32_issue(taddr + c0, r);
            tmem_ld_wait(r);
            if (c0 + 32 >= TILE) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(my_empty);
            }
            if (interior) {
              // Every key is visible and observed.  The exponentials are taken against the row's
              // running reference m without looking for the chunk's maximum first; a chunk whose
              // sum comes out beyond kChunkSumMax (or not finite: m still -inf) holds a logit far
              // above m and is done once more after m has moved to the chunk's maximum.  That is
              // rare after the first tiles, and any reference within reach of the fp32 exponent
              // range gives the same sums.
              const f32x2 sc2 = pack2(P.scale2, P.scale2);
              float zs, ws;
#pragma unroll 1
              for (int pass = 0;; ++pass) {
                // two keys per instruction: four partial sums in two packed accumulators
                const f32x2 nm2 = pack2(-m, -m);
                f32x2 zc[2] = {0ull, 0ull}, wc[2] = {0ull, 0ull};
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                  const f32x2 tt2 = fma2(pack2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), sc2, nm2);
                  float t0, t1;
                  unpack2(tt2, t0, t1);
                  const f32x2 ee2 = pack2(ex2(t0), ex2(t1));
                  zc[(e >> 1) & 1] = add2(zc[(e >> 1) & 1], ee2);
                  wc[(e >> 1) & 1] = fma2(ee2, tt2, wc[(e >> 1) & 1]);
                }
                float z0, z1, w0, w1;
                unpack2(add2(zc[0], zc[1]), z0, z1);
                unpack2(add2(wc[0], wc[1]), w0, w1);
                zs = z0 + z1;
                ws = w0 + w1;
                if (zs <= kChunkSumMax || pass > 0) break;
                float cm = __uint_as_float(r[0]);
#pragma unroll
                for (int e = 1; e < 32; ++e) cm = fmaxf(cm, __uint_as_float(r[e]));
                const float mn = cm * P.scale2;
                const float f = ex2(m - mn);                  // 0 while m = -inf
                const float dm = (m == -CUDART_INF_F) ? 0.f : (m - mn);
                w = f * fmaf(dm, z - zwin, w);
                z *= f; zwin *= f;
                m = mn;
              }
              z += zs;
              w += ws;
            } else {
              float cm = -CUDART_INF_F;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int j = key0 + c0 + e;
                const bool vis = (it * TILE + c0 + e < op.nkeys) && j <= last;
                cm = vis ? fmaxf(cm, __uint_as_float(r[e])) : cm;
              }
              if (cm != -CUDART_INF_F) {
                cm *= P.scale2;
                if (cm > m) {
                  const float mn = cm;
                  const float f = ex2(m - mn);
                  const float dm = (m == -CUDART_INF_F) ? 0.f : (m - mn);
                  w = f * fmaf(dm, z - zwin, w);
                  z *= f; zwin *= f;
                  m = mn;
                }
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  const int j = key0 + c0 + e;
                  const bool vis = (it * TILE + c0 + e < op.nkeys) && j <= last;
                  const bool obs = j < op.n;
                  const float tt = fmaf(__uint_as_float(r[e]), P.scale2, -m);
                  const float ee = vis ? ex2(tt) : 0.f;
                  z += ee;
                  zwin += obs ? 0.f : ee;
                  w = (vis && obs) ? fmaf(ee, tt, w) : w;
                }
              }
            }
          }
        }
        // Deliver this warp's 32 partial rows of the segment.  Making them visible to the other
        // CTAs takes a fence of a few thousand cycles; the merger warp pays it once per op for all
        // twelve warps, which only tell it, inside the CTA, that their rows are written.
        __stcg(&P.rowpart[((size_t)op.seg * NWG + wg) * 128 + lane_row], make_float4(m, z, zwin, w));
        __syncwarp();
        ++n_a_done;
        if (lane == 0) smem_store_release(&S.a_done[warp], n_a_done);
      }
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512)
                 : "memory");
  }
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


template <int G>
cudaError_t launch_g(int device, bool entropy_b, int n_cta, cudaStream_t st, const CUtensorMap& qmap,
                     const CUtensorMap& kmap, const TcParams& P) {
  static PerDeviceOnce attr;
  if (attr.need(device)) {
    cudaError_t e = cudaFuncSetAttribute(score_fused_kernel<G, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(score_fused_kernel<G, true>,
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    attr.mark(device);
  }
  if (entropy_b) score_fused_kernel<G, true><<<n_cta, TC_THREADS, kSmemBytes, st>>>(qmap, kmap, P);
  else           score_fused_kernel<G, false><<<n_cta, TC_THREADS, kSmemBytes, st>>>(qmap, kmap, P);
  return cudaGetLastError();
}

// Cuts the `tiles` tiles of one (request, head) pair, which start at flat tile index `flat`
// of a wave of `W` tiles shared by `n_cta` CTAs (slot c owns flat tiles
// [c*W/n_cta, (c+1)*W/n_cta)), into per-slot segments; slot c belongs to CTA (c+rot)%n_cta.
// With `split`, a slot's segment of two or more tiles becomes two ops (pad = 1: first half,
// pad = 2: second half) that the program builder may place apart.
void cut_pair(std::vector<std::vector<ScoreOp>>& per_cta, int rot, int n_cta, int64_t W, int64_t flat,
              int tiles, int keys, int req, int g, int phase, int32_t& seg_counter, int64_t base,
              int n_obs, bool split = false) {
  int t0 = 0;
  while (t0 < tiles) {
    const int64_t f = flat + t0;
    int c = (int)(f * n_cta / W);
    while (c + 1 < n_cta && (int64_t)(c + 1) * W / n_cta <= f) ++c;
    while (c > 0 && (int64_t)c * W / n_cta > f) --c;
    const int64_t share_end = (int64_t)(c + 1) * W / n_cta;
    const int t1 = (int)((share_end - flat) < tiles ? (share_end - flat) : tiles);
    const int parts = (split && t1 - t0 >= 2) ? 2 : 1;
    const int tm = t0 + (t1 - t0 + 1) / 2;
    for (int part = 0; part < parts; ++part) {
      const int a = part == 0 ? t0 : tm, b = (parts == 2 && part == 0) ? tm : t1;
      ScoreOp op;
      op.base = base; op.n = n_obs;
      op.pad = parts == 2 ? part + 1 : 0;
      op.req = req; op.g = g; op.key0 = a * TILE;
      const int kend = b * TILE < keys ? b * TILE : keys;
      op.nkeys = kend - a * TILE;
      op.phase = phase;
      op.seg = seg_counter++;
      per_cta[(c + rot) % n_cta].push_back(op);
    }
    t0 = t1;
  }
}

// Waves of consecutive (request, KV head) pairs: K of the wave in pass B and of the wave in pass A
// must fit L2 together, so a wave is closed before the pair that would take it past kWaveBytes.
// (One wave for a whole layer of up to 64 MB was tried: no faster at 34 MB, slower at 64 MB.)
std::vector<int> tc_waves(const ReqInfo* reqs, int n_req, int Hkv, int head_dim) {
  const int n_pairs = n_req * Hkv;
  std::vector<int> wave_begin{0};
  int64_t bytes = 0;
  for (int p = 0; p < n_pairs; ++p) {
    const int64_t pb = (int64_t)reqs[p / Hkv].N * head_dim * 2;
    if (bytes > 0 && bytes + pb > kWaveBytes) {
      wave_begin.push_back(p);
      bytes = 0;
    }
    bytes += pb;
  }
  wave_begin.push_back(n_pairs);
  return wave_begin;
}

}  // namespace

bool tc_path_supported(const cake_config& c) {
  const int G = c.n_q_heads / c.n_kv_heads;
  const int rows = G * c.window;
  return c.dtype == CAKE_DTYPE_BF16 && (c.head_dim == 64 || c.head_dim == 128) && rows % 32 == 0 &&
         rows <= 128 && (G == 1 || G == 2 || G == 4 || G == 8) && c.window <= 256;
}

// Upper bound on the segments of one pass: every pair gives one segment plus one per CTA
// boundary inside its wave; two consecutive waves hold more than kWaveBytes of K, and there
// are no more waves than pairs.
int64_t tc_max_segments(const cake_config& c, int n_sm) {
  const int64_t pairs = (int64_t)c.max_requests * c.n_kv_heads;
  const int64_t bytes = (int64_t)c.n_kv_heads * c.max_total_tokens * c.head_dim * 2;
  int64_t waves = 2 * (bytes / kWaveBytes) + 2;
  if (waves > pairs) waves = pairs;
  return pairs + (waves + 2) * n_sm;          // + the two waves whose ops are halved
}

// Builds the per-CTA programs of the batch in ctx->h_req[0..n_req): `full` = both passes
// interleaved by wave, `bonly` = pass B alone (denominators supplied by the caller).
int32_t tc_build_plan(cake_ctx* ctx, int32_t n_req) {
  const cake_config& c = ctx->cfg;
  const int Hkv = c.n_kv_heads;
  const int n_pairs = n_req * Hkv;
  const int64_t T = n_req > 0 ? ctx->h_req[n_req - 1].cu + ctx->h_req[n_req - 1].N : 0;
  int64_t tilesA_total = 0;
  for (int r = 0; r < n_req; ++r) tilesA_total += (int64_t)Hkv * ((ctx->h_req[r].N + TILE - 1) / TILE);
  int n_cta = (int)(tilesA_total < ctx->n_sm_score ? tilesA_total : ctx->n_sm_score);
  ctx->n_tc_ctas = n_cta;
  ctx->n_tc_ops_full = ctx->n_tc_ops_b = 0;
  ctx->n_tc_asegs = ctx->n_tc_bsegs = 0;
  ctx->n_tc_waves = 0;
  if (n_cta == 0) return CAKE_OK;

  const std::vector<int> wave_begin = tc_waves(ctx->h_req, n_req, Hkv, c.head_dim);
  const int n_waves = (int)wave_begin.size() - 1;
  ctx->n_tc_waves = n_waves;
  // Every wave ends when its slowest CTA does, i.e. after ceil(tiles / CTAs) tiles, and both
  // passes walk it.  Among the CTA counts down to three quarters of the SMs on offer, take the
  // smallest one that reaches the minimum of the summed quotients: the SMs left over shorten
  // nothing here and go to the cascade kernels that run beside this one.
  {
    std::vector<int64_t> w(n_waves, 0);
    for (int wv = 0; wv < n_waves; ++wv)
      for (int p = wave_begin[wv]; p < wave_begin[wv + 1]; ++p) w[wv] += (ctx->h_req[p / Hkv].N + TILE - 1) / TILE;
    int64_t best = -1;
    int best_n = n_cta;
    for (int n = n_cta; n >= 1 && n >= n_cta - n_cta / 4; --n) {
      int64_t steps = 0;
      for (int wv = 0; wv < n_waves; ++wv) steps += (w[wv] + n - 1) / n;
      if (best < 0 || steps <= best) { best = steps; best_n = n; }
      else break;
    }
    n_cta = best_n;
    ctx->n_tc_ctas = n_cta;
  }
  // Program of a CTA, by waves:  A0 A1 B0 A2 B1 ... A(n-1) B(n-2) B(n-1).  Pass B of a wave waits
  // for the wave's merged denominators, which trail the slowest CTA's pass A by some 7 us; in
  // the steady state the pass A in between covers that.  At the two ends it does not, so there
  // (when the waves are single pairs, and there are at least four) one op is halved and its halves
  // placed apart: A2's first half goes before B0, and B(n-3)'s second half goes after A(n-1).
  std::vector<std::vector<std::vector<ScoreOp>>> was(n_waves), wbs(n_waves);   // [wave][CTA]
  std::vector<std::vector<ScoreOp>> full(n_cta), bonly(n_cta);
  int32_t aseg = 0, bseg = 0;
  int32_t* pair_aseg = ctx->h_tc_index;                    // [pairs+1]
  int32_t* pair_bseg = ctx->h_tc_index + (n_pairs + 1);    // [pairs+1]
  const bool ends = kWaveDepth == 1 && n_waves >= 4;
  auto single = [&](int wv) { return wave_begin[wv + 1] - wave_begin[wv] == 1; };
  const int split_a = ends && single(2) ? 2 : -1;
  const int split_b = ends && single(n_waves - 3) ? n_waves - 3 : -1;
  int rot = 0;
  for (int wv = 0; wv < n_waves; ++wv) {
    int64_t WA = 0;
    for (int p = wave_begin[wv]; p < wave_begin[wv + 1]; ++p)
      WA += (ctx->h_req[p / Hkv].N + TILE - 1) / TILE;
    was[wv].assign(n_cta, {});
    wbs[wv].assign(n_cta, {});
    int64_t fa = 0;
    for (int p = wave_begin[wv]; p < wave_begin[wv + 1]; ++p) {
      const int r = p / Hkv, g = p % Hkv;
      const ReqInfo& rq = ctx->h_req[r];
      const int ta = (rq.N + TILE - 1) / TILE, tb = (rq.n + TILE - 1) / TILE;
      pair_aseg[p] = aseg;
      pair_bseg[p] = bseg;
      const int64_t base = (int64_t)g * T + rq.cu;
      cut_pair(was[wv], rot, n_cta, WA, fa, ta, rq.N, r, g, 0, aseg, base, rq.n, wv == split_a);
      // pass B walks the same flat tile positions, so a CTA re-reads the tiles it brought in
      if (tb > 0) cut_pair(wbs[wv], rot, n_cta, WA, fa, tb, rq.n, r, g, 1, bseg, base, rq.n, wv == split_b);
      fa += ta;
    }
    // a wave's remainder tiles land on different CTAs each time (golden-ratio stride)
    rot = (rot + (int)(n_cta * 0.381966) + 1) % n_cta;
  }
  // which = 0: every op, 1: first halves and unsplit ops, 2: second halves
  auto put = [&](std::vector<ScoreOp>& dst, const std::vector<ScoreOp>& src, int which) {
    for (const ScoreOp& op : src)
      if (which == 0 || (which == 1 && op.pad != 2) || (which == 2 && op.pad == 2)) dst.push_back(op);
  };
  for (int cta = 0; cta < n_cta; ++cta) {
    for (int wv = 0; wv < n_waves; ++wv) {
      // pass A of this wave
      if (wv == split_a) {
        put(full[cta], was[wv][cta], 1);                       // A2 first half
        put(full[cta], wbs[wv - 2][cta], 0);                   // B0 (held back one slot)
        put(full[cta], was[wv][cta], 2);                       // A2 second half
      } else {
        put(full[cta], was[wv][cta], 0);
      }
      // pass B of the wave kWaveDepth behind
      if (split_b >= 0 && wv == split_b + 2) put(full[cta], wbs[split_b][cta], 2);   // B(n-3) second half, after A(n-1)
      const int bw = wv - kWaveDepth;
      if (bw >= 0 && !(split_a >= 0 && bw == split_a - 2 && wv == split_a - 1)) {
        if (bw == split_b) put(full[cta], wbs[bw][cta], 1);    // B(n-3) first half in its usual place
        else put(full[cta], wbs[bw][cta], 0);
      }
      put(bonly[cta], wbs[wv][cta], 0);
    }
    for (int wv = n_waves > kWaveDepth ? n_waves - kWaveDepth : 0; wv < n_waves; ++wv)
      put(full[cta], wbs[wv][cta], 0);
  }
  pair_aseg[n_pairs] = aseg;
  pair_bseg[n_pairs] = bseg;
  if (aseg > ctx->max_tc_segs || bseg > ctx->max_tc_segs) return CAKE_ERR_CAPACITY;

  int32_t* cta_full = ctx->h_tc_index + 2 * (n_pairs + 1);   // [n_sm+1]
  int32_t* cta_b = cta_full + (ctx->n_sm + 1);               // [n_sm+1]
  int64_t total = 0;
  for (int cta = 0; cta < n_cta; ++cta) total += (int64_t)(full[cta].size() + bonly[cta].size());
  if (total > ctx->max_tc_ops) return CAKE_ERR_CAPACITY;
  int32_t o = 0;
  for (int cta = 0; cta < n_cta; ++cta) {
    cta_full[cta] = o;
    for (const ScoreOp& op : full[cta]) ctx->h_tc_ops[o++] = op;
  }
  cta_full[n_cta] = o;
  ctx->n_tc_ops_full = o;
  for (int cta = 0; cta < n_cta; ++cta) {
    cta_b[cta] = o;
    for (const ScoreOp& op : bonly[cta]) ctx->h_tc_ops[o++] = op;
  }
  cta_b[n_cta] = o;
  ctx->n_tc_ops_b = o - ctx->n_tc_ops_full;
  ctx->n_tc_asegs = aseg;
  ctx->n_tc_bsegs = bseg;
  // several rows at a time when there are pairs to take them from and a row has few partials
  {
    int max_segs = 0;
    for (int p = 0; p < n_pairs; ++p) max_segs = std::max(max_segs, pair_aseg[p + 1] - pair_aseg[p]);
    const int partials = max_segs * NWG;
    // at most 16 partials per lane (two batches of loads): 32 lanes / ways per row
    int ways = 1;
    while (ways < 32 && 2 * ways <= n_pairs && partials * 2 * ways <= 512) ways *= 2;
    if (n_pairs < 4) ways = 1;
    // The merger handles `ways` consecutive pairs at once and waits for the pass A of all of them.
    // A CTA's program only guarantees A(w+1) before B(w): a group that reached from wave w into
    // wave w+2 would make B(w) wait for an A(w+2) that comes after it.  So every group must lie
    // in at most two adjacent waves.
    std::vector<int> wave_of(n_pairs, 0);
    for (int wv = 0; wv < n_waves; ++wv)
      for (int p = wave_begin[wv]; p < wave_begin[wv + 1]; ++p) wave_of[p] = wv;
    auto span_ok = [&](int wy) {
      for (int p0 = 0; p0 < n_pairs; p0 += wy) {
        const int p1 = std::min(n_pairs, p0 + wy) - 1;
        if (wave_of[p1] - wave_of[p0] > kWaveDepth) return false;
      }
      return true;
    };
    while (ways > 1 && !span_ok(ways)) ways >>= 1;
    ctx->tc_merge_ways = ways;
  }
  return CAKE_OK;
}

// Builds the plan of a batch on the host alone (no device, no context) and checks the properties
// the kernel relies on.  Returns CAKE_OK, an error of the plan builder, or CAKE_ERR_STATE with
// info8[7] = the number of the violated property:
//   1  every key tile of every pair is covered exactly once by the pass-A ops, and every non-window
//      tile exactly once by the pass-B ops
//   2  inside every CTA's program the pass-B ops come in non-decreasing wave order and every
//      pass-A op of a wave w' <= w precedes the first pass-B op of wave w (so a wave's pass B can
//      only ever wait for pass-A ops that wait for nothing themselves)
//   3  the pairs the merger warps handle side by side lie in at most two adjacent waves
//   4  op counts and segment numbers stay inside the tables the context would allocate
int32_t tc_plan_check(const cake_config& c, int n_sm, int reserved, int32_t n_req, const int64_t* cu,
                      int32_t* info8) {
  if (!tc_path_supported(c)) return CAKE_ERR_ARG;
  cake_ctx x;
  memset(&x, 0, sizeof(x));
  x.cfg = c;
  x.n_sm = n_sm;
  x.n_sm_score = n_sm - reserved > 0 ? n_sm - reserved : 1;
  const int Hkv = c.n_kv_heads, n_pairs = n_req * Hkv;
  std::vector<ReqInfo> reqs(n_req > 0 ? n_req : 1);
  for (int r = 0; r < n_req; ++r) {
    memset(&reqs[r], 0, sizeof(ReqInfo));
    reqs[r].cu = cu[r];
    reqs[r].N = (int32_t)(cu[r + 1] - cu[r]);
    reqs[r].n = reqs[r].N - c.window;
  }
  x.h_req = reqs.data();
  x.max_tc_segs = (int32_t)tc_max_segments(c, n_sm);
  x.max_tc_ops = 3 * x.max_tc_segs + 8;
  std::vector<ScoreOp> ops((size_t)x.max_tc_ops);
  std::vector<int32_t> index(2 * (size_t)(n_pairs + 1) + 2 * (size_t)(n_sm + 1));
  x.h_tc_ops = ops.data();
  x.h_tc_index = index.data();
  const int32_t rc = tc_build_plan(&x, n_req);
  info8[0] = x.n_tc_ctas; info8[1] = x.n_tc_waves; info8[2] = x.tc_merge_ways; info8[3] = x.n_tc_asegs;
  info8[4] = x.n_tc_bsegs; info8[5] = x.n_tc_ops_full; info8[6] = x.n_tc_ops_b; info8[7] = 0;
  if (rc != CAKE_OK || x.n_tc_ctas == 0) return rc;
  auto fail = [&](int what) { info8[7] = what; return (int32_t)CAKE_ERR_STATE; };
  if (x.n_tc_ops_full + x.n_tc_ops_b > x.max_tc_ops || x.n_tc_asegs > x.max_tc_segs ||
      x.n_tc_bsegs > x.max_tc_segs) return fail(4);
  // waves as the builder forms them
  std::vector<int> wave_of(n_pairs, 0);
  {
    const std::vector<int> wb = tc_waves(reqs.data(), n_req, Hkv, c.head_dim);
    for (int wv = 0; wv + 1 < (int)wb.size(); ++wv)
      for (int p = wb[wv]; p < wb[wv + 1]; ++p) wave_of[p] = wv;
  }
  const int32_t* cta_full = index.data() + 2 * (n_pairs + 1);
  // 1: coverage, per pair and pass, in tiles
  std::vector<std::vector<int>> cover[2];
  for (int ph = 0; ph < 2; ++ph) {
    cover[ph].resize(n_pairs);
    for (int p = 0; p < n_pairs; ++p) {
      const ReqInfo& rq = reqs[p / Hkv];
      cover[ph][p].assign(((ph ? rq.n : rq.N) + TILE - 1) / TILE, 0);
    }
  }
  for (int cta = 0; cta < x.n_tc_ctas; ++cta) {
    int last_b_wave = -1;
    std::vector<int> first_b_pos(x.n_tc_waves + 1, -1);
    std::vector<int> last_a_pos(x.n_tc_waves + 1, -1);
    for (int o = cta_full[cta]; o < cta_full[cta + 1]; ++o) {
      const ScoreOp& op = ops[o];
      const int p = op.req * Hkv + op.g;
      if (p < 0 || p >= n_pairs || op.key0 % TILE != 0 || op.nkeys <= 0) return fail(1);
      if (op.seg < 0 || op.seg >= (op.phase ? x.n_tc_bsegs : x.n_tc_asegs)) return fail(4);
      const int t0 = op.key0 / TILE, t1 = (op.key0 + op.nkeys + TILE - 1) / TILE;
      if (t1 > (int)cover[op.phase][p].size()) return fail(1);
      for (int t = t0; t < t1; ++t) cover[op.phase][p][t] += 1;
      const int wv = wave_of[p], pos = o - cta_full[cta];
      if (op.phase) {
        if (wv < last_b_wave) return fail(2);
        last_b_wave = wv;
        if (first_b_pos[wv] < 0) first_b_pos[wv] = pos;
      } else {
        last_a_pos[wv] = pos;
      }
    }
    for (int w = 0; w < x.n_tc_waves; ++w)
      if (first_b_pos[w] >= 0)
        for (int w2 = 0; w2 <= w; ++w2)
          if (last_a_pos[w2] > first_b_pos[w]) return fail(2);
  }
  for (int ph = 0; ph < 2; ++ph)
    for (int p = 0; p < n_pairs; ++p)
      for (int v : cover[ph][p])
        if (v != 1) return fail(1);
  // 3: merge groups
  const int ways = x.tc_merge_ways;
  for (int p0 = 0; p0 < n_pairs; p0 += ways) {
    const int p1 = std::min(n_pairs, p0 + ways) - 1;
    if (wave_of[p1] - wave_of[p0] > kWaveDepth) return fail(3);
  }
  return CAKE_OK;
}

int32_t launch_score_tc(cake_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                        const float* lse, cudaStream_t st) {
  const cake_config& c = ctx->cfg;
  if (ctx->n_tc_ctas == 0) return CAKE_OK;
  if ((int64_t)c.n_kv_heads * ctx->total_tokens >= ((int64_t)1 << 31)) return CAKE_ERR_ARG;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return CAKE_ERR_CUDA;
  const int G = c.n_q_heads / c.n_kv_heads;
  CUtensorMap qmap, kmap;
  {
    // K [rows][d] seen as (64 elements, rows, d/64 slabs): one box of 128 rows brings both
    // 64-element halves of the rows, each as its own 128-byte-swizzled slab
    const cuuint64_t dims[3] = {64, (cuuint64_t)c.n_kv_heads * ctx->total_tokens, (cuuint64_t)(c.head_dim / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)c.head_dim * 2, 128};
    const cuuint32_t box[3] = {64, TILE, (cuuint32_t)(c.head_dim / 64)};
    const cuuint32_t es[3] = {1, 1, 1};
    if (enc(&kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(k), dims, strides, box, es,
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
  const int n_pairs = ctx->n_req * c.n_kv_heads;
  TcParams P;
  P.ops = ctx->d_tc_ops;
  P.reqs = ctx->d_req;
  P.pair_aseg = ctx->d_tc_index;
  P.pair_cnt = ctx->d_tc_sync;
  P.lse2 = ctx->d_lse2_tc;
  P.lse_ext = lse;
  P.rowpart = ctx->d_tc_rowpart;
  P.raw = ctx->d_raw[layer & 1];
  P.colpart = ctx->d_colpart[layer & 1];
  P.hrow = ctx->d_hrow[layer & 1];
  P.n_pairs = n_pairs;
  P.status = ctx->d_status;
  P.T = ctx->total_tokens;
  P.Hkv = c.n_kv_heads; P.Hq = c.n_q_heads; P.Sw = c.window; P.rows = ctx->rows; P.d = c.head_dim;
  P.scale2 = kLog2e / sqrtf((float)c.head_dim);
  P.inv_scale2 = 1.f / P.scale2;
  P.gamma = c.gamma;
  P.ind_mode = c.indicator_mode;
  P.merge_ways = ctx->tc_merge_ways;
  P.spin_limit = ctx->wait_limit_cycles > 0 ? ctx->wait_limit_cycles : kSpinLimit;
  P.bessel = c.var_ddof ? (float)c.window / (float)(c.window - 1) : 1.f;

  const int sp = prof_begin(ctx, CAKE_PROF_SCORE, st);
  const int32_t* cta_full = ctx->d_tc_index + 2 * (n_pairs + 1);
  if (lse) {
    // denominators supplied: pass B alone, entropy from its columns
    ctx->hhead_from_rows = false;
    P.cta_op = cta_full + (ctx->n_sm + 1);
    P.pair_done = nullptr;
    P.epoch = 0;
  } else {
    ctx->hhead_from_rows = true;
    P.cta_op = cta_full;
    P.pair_done = ctx->d_tc_sync + ctx->max_pairs;
    P.epoch = ++ctx->tc_epoch + (uint32_t)ctx->debug_epoch_skew;
  }
  cudaError_t e;
  const bool eb = lse != nullptr;
  switch (G) {
    case 1: e = launch_g<1>(ctx->device, eb, ctx->n_tc_ctas, st, qmap, kmap, P); break;
    case 2: e = launch_g<2>(ctx->device, eb, ctx->n_tc_ctas, st, qmap, kmap, P); break;
    case 4: e = launch_g<4>(ctx->device, eb, ctx->n_tc_ctas, st, qmap, kmap, P); break;
    default: e = launch_g<8>(ctx->device, eb, ctx->n_tc_ctas, st, qmap, kmap, P); break;
  }
  count_launch();
  prof_end(ctx, sp, st);
  return cuda_status(e);
}

}  // namespace cake
