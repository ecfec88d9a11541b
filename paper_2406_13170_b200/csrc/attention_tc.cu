// Tree attention for bf16 caches on the 5th-generation tensor cores (Section 2 "Tree Attention", Appendix A.1):
// split-KV flash-decoding in which the tree is a per-row 128-bit ancestor mask.
//
// Grid (head, KV split, block of 64 query rows).  One CTA walks its key range in chunks of 128 keys:
//   warp 0      TMA producer: Q tile once, then K and V chunks into a shared-memory ring (cp.async.bulk.tensor through
//               tensor maps over this GPU's own cache, no multicast).  Chunks that lie wholly inside the committed
//               context do not depend on the kernel before this one and are requested BEFORE the dependency wait.
//   warp 1      MMA issuer: S = Q K^T (tcgen05.mma, M = 64 rows, N = 128 keys, accumulator in tensor memory), then
//               O_c = P V (A = the probabilities written back to shared memory as a K-major operand, B = the V rows
//               as they sit in the cache, i.e. an MN-major operand).
//   warps 2-5   softmax: scores from tensor memory (tcgen05.ld), mask, running max / sum in fp32, probabilities to
//               shared memory in bf16, running output in registers (the chunk outputs are added with the usual
//               rescaling, so tensor memory never has to be rescaled).
// The KV splits of one head form a thread-block cluster and merge their partial outputs through distributed shared
// memory; with more than 8 splits the partials go to global scratch for attn_combine_kernel.
// Every barrier wait is bounded; a wait that gives up raises the error flag and the CTA leaves in order.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <map>
#include <tuple>

#include "amph.h"
#include "amph_internal.cuh"

namespace amph {

typedef __nv_bfloat16 bf16;

namespace {

constexpr int kRows = 64;            // query rows per CTA (UMMA M)
constexpr int kChunk = 128;          // keys per pipeline stage (UMMA N of the score MMA)
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;       // S in columns [0, 128), O in [128, 128 + DH): room is left for the projection CTAs that
                                     // become resident beside this kernel and allocate their accumulators
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

constexpr int kMaxGroups = AMPH_MAX_BATCH;   // row groups (sequences, or chunks of one prompt) one launch may carry

// NG = 1 for the usual launch (kernel parameters stay small: they are copied with every launch), kMaxGroups for the grouped one
template <int NG>
struct AttnMaps {
  CUtensorMap q;                      // all groups' query rows: group g starts at row g * rows_per_group
  CUtensorMap k[NG], v[NG];           // the cache each group reads
};

template <int NG>
struct AttnParams {
  const RowMeta* meta[NG];
  int nrb, rpg;              // 64-row blocks per group (grid.z = groups * nrb), rows per group
  int same_cache;            // the groups are consecutive chunks of one sequence: slots from meta[0]->base on are written by this pass
  float* po;                 // partial outputs / (max, sum) for the separate merge (one group only)
  float* pml;
  bf16* out;                 // merged output rows (cluster merge), or NULL
  int rows_cap, n_heads, max_ctx, stages;
  int* err_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false (and the CTA-wide abort flag raised) if the phase never completes or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = now_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool elect_one() {
  uint32_t e;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
  return e != 0;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle, 8-row (or, for an MN-major operand, 8-column) groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// The same for the MN-major operand V ([key][64 head dims] rows of 128 bytes): an MMA of N = 64 spans exactly one swizzle
// atom along MN, so the only stride in play is the one between groups of 8 keys (1024 bytes); both offset fields carry it.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(1024 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// D = f32, A = B = bf16, A K-major, B K-major (b_mn = 0) or MN-major (b_mn = 1), M = 64.
__device__ __forceinline__ uint32_t umma_idesc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16 TMEM lanes x 64 columns, spread over the whole warp (checked on the device): thread t, register 4 * rep + 2 * hi + e
// holds lane (t / 4 + 8 * hi), column 8 * rep + 2 * (t % 4) + e: the layout of an mma accumulator fragment.
__device__ __forceinline__ void tmem_ld_frag64(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
               : "r"(taddr)
               : "memory");
}
// 2^x on the special-function unit: ex2(-inf) = +0, so masked scores need no test of their own
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t peer_smem(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_peer4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_peer2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}

// Bits [0, 128) of (ones below `nctx`, then the 128-bit mask m shifted up by nctx), shifted down by `sh` (< 8).
// nctx = base - key0 may be negative (the chunk starts inside the tree slots) or beyond 128 (all context).
__device__ __forceinline__ void chunk_visibility(u64 m0, u64 m1, bool live, int nctx, int sh, u64& v0, u64& v1) {
  u64 a0, a1;
  if (!live) { a0 = a1 = 0ull; }
  else if (nctx >= 128) { a0 = a1 = ~0ull; }
  else if (nctx >= 64) { const int k = nctx - 64; a0 = ~0ull; a1 = (k ? ((1ull << k) - 1ull) : 0ull) | (m0 << k); }
  else if (nctx > 0) { a0 = ((1ull << nctx) - 1ull) | (m0 << nctx); a1 = (m0 >> (64 - nctx)) | (m1 << nctx); }
  else if (nctx == 0) { a0 = m0; a1 = m1; }
  else if (nctx > -64) { const int k = -nctx; a0 = (m0 >> k) | (m1 << (64 - k)); a1 = m1 >> k; }
  else if (nctx > -128) { a0 = m1 >> (-nctx - 64); a1 = 0ull; }
  else { a0 = a1 = 0ull; }
  v0 = sh ? ((a0 >> sh) | (a1 << (64 - sh))) : a0;
  v1 = a1 >> sh;
}

template <int DH, bool MERGE, int NG>
__global__ void __launch_bounds__(kThreads, 2)
tree_attn_tc_kernel(const __grid_constant__ AttnMaps<NG> maps, const AttnParams<NG> prm) {
  constexpr int NB = DH / 64;                        // 64-wide blocks of the head dimension (one 128-byte swizzle row each)
  constexpr uint32_t kQBlock = kRows * 128;          // bytes of one Q / P block: 64 rows x 128 bytes
  constexpr uint32_t kKvBlock = kChunk * 128;        // bytes of one K / V block: 128 keys x 128 bytes
  constexpr uint32_t kStage = 2 * NB * kKvBlock;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t q_full, p_ready, o_full;
  __shared__ __align__(8) uint64_t k_full[4], v_full[4], k_empty[4], v_empty[4], s_full;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x, split = blockIdx.y;
  const int grp = NG == 1 ? 0 : (int)blockIdx.z / prm.nrb, rb = NG == 1 ? (int)blockIdx.z : (int)blockIdx.z - grp * prm.nrb;
  const RowMeta* const meta = prm.meta[grp];
  const int row_base = grp * prm.rpg;                // first row of this group in the query / output buffers
  const int stages = prm.stages;
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* Qs = smem;
  uint8_t* Ps = Qs + NB * kQBlock;
  uint8_t* St = Ps + 2 * kQBlock;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&q_full, 1);
    mbar_init(&p_ready, 128);
    mbar_init(&o_full, 1);
    for (int s = 0; s < 4; ++s) { mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_empty[s], 1); }
    mbar_init(&s_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_base_slot;

  // The row table was written several kernels ago (every kernel between it and this one waits for its own
  // predecessor before it lets its successor start), so it may be read before the dependency wait.
  const int base = meta->base, n_rows = meta->n_rows;
  const int total = base + n_rows;
  int len = (total + (int)gridDim.y - 1) / (int)gridDim.y;
  len = (len + kChunk - 1) / kChunk * kChunk;          // whole chunks: a chunk never straddles two splits
  const int s_lo = split * len;
  int s_hi = s_lo + len;
  if (s_hi > total) s_hi = total;
  if (s_hi > prm.max_ctx) s_hi = prm.max_ctx;
  const int n_chunks = s_hi > s_lo ? (s_hi - s_lo + kChunk - 1) / kChunk : 0;

  // softmax warps: running output of rows row_a and row_a + 8 as accumulator fragments
  // (acc[4 * rep + 2 * hi + e] = row row_a + 8 * hi, head dim 8 * rep + 2 * qd + e), running max (base 2) and sum
  float acc[DH / 2];
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
#pragma unroll
  for (int i = 0; i < DH / 2; ++i) acc[i] = 0.f;
  const int quarter = warp & 3;
  const int row_a = quarter * 16 + (lane >> 2), qd = lane & 3;

  if (warp == 0) {
    // ---------------- TMA producer
    const bool leader = elect_one();
    if (leader) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.q) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.k[grp]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.v[grp]) : "memory");
    }
    int issued = 0;
    bool k_only = false;                               // gave up between the key and the value copies of chunk `issued`
    // committed context: nothing the previous kernel writes
    if (leader) {
      // slots the kernel before this one may still be writing must wait: everything from this group's base on, and, when
      // the groups are chunks of one prompt, everything from the first group's base on (earlier chunks of the same pass)
      const int settled = (NG > 1 && prm.same_cache) ? prm.meta[0]->base : base;
      while (issued < n_chunks && issued < stages && s_lo + (issued + 1) * kChunk <= settled) {
        uint8_t* kdst = St + (size_t)issued * kStage;
        mbar_expect_tx(&k_full[issued], NB * kKvBlock);
        mbar_expect_tx(&v_full[issued], NB * kKvBlock);
        for (int j = 0; j < NB; ++j) tma_load_3d(kdst + j * kKvBlock, &maps.k[grp], 64 * j, s_lo + issued * kChunk, h, &k_full[issued]);
        for (int j = 0; j < NB; ++j) tma_load_3d(kdst + (NB + j) * kKvBlock, &maps.v[grp], 64 * j, s_lo + issued * kChunk, h, &v_full[issued]);
        ++issued;
      }
    }
    issued = __shfl_sync(0xffffffffu, issued, __ffs(__ballot_sync(0xffffffffu, leader)) - 1);
    pdl_wait();
    pdl_launch_dependents();
    if (leader && n_chunks > 0) {
      mbar_expect_tx(&q_full, NB * kQBlock);
      for (int j = 0; j < NB; ++j) tma_load_2d(Qs + j * kQBlock, &maps.q, h * DH + 64 * j, row_base + rb * kRows, &q_full);
    }
    for (int c = issued; c < n_chunks; ++c) {
      const int st = c % stages, round = c / stages;
      // the key half of a stage is free once the scores that read it are complete, the value half once P V is: the next
      // keys arrive while this chunk's softmax and P V run, the next values while the next scores and softmax run
      uint8_t* kdst = St + (size_t)st * kStage;
      if (round > 0 && !__all_sync(0xffffffffu, mbar_wait(&k_empty[st], (round & 1) ^ 1, &abort_flag))) break;
      if (leader) {
        mbar_expect_tx(&k_full[st], NB * kKvBlock);
        for (int j = 0; j < NB; ++j) tma_load_3d(kdst + j * kKvBlock, &maps.k[grp], 64 * j, s_lo + c * kChunk, h, &k_full[st]);
      }
      __syncwarp();
      if (round > 0 && !__all_sync(0xffffffffu, mbar_wait(&v_empty[st], (round & 1) ^ 1, &abort_flag))) { k_only = true; break; }
      if (leader) {
        mbar_expect_tx(&v_full[st], NB * kKvBlock);
        for (int j = 0; j < NB; ++j) tma_load_3d(kdst + (NB + j) * kKvBlock, &maps.v[grp], 64 * j, s_lo + c * kChunk, h, &v_full[st]);
      }
      __syncwarp();
      issued = c + 1;
    }
    if (abort_flag && lane == 0) {                     // drain: let every copy that was issued land
      const unsigned long long t0 = now_ns();
      const int first = issued > stages ? issued - stages : 0;
      for (int c = first; c < issued; ++c) {
        const int st = c % stages, round = c / stages;
        while (!(mbar_try(&k_full[st], round & 1) && mbar_try(&v_full[st], round & 1)) && now_ns() - t0 < kWaitLimitNs) {}
      }
      if (k_only && issued < n_chunks)
        while (!mbar_try(&k_full[issued % stages], (issued / stages) & 1) && now_ns() - t0 < kWaitLimitNs) {}
      if (n_chunks > 0) while (!mbar_try(&q_full, 0) && now_ns() - t0 < kWaitLimitNs) {}
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    pdl_wait();
    const bool leader = elect_one();
    const uint32_t idesc_s = umma_idesc(kChunk, 0), idesc_o = umma_idesc(64, 1);
    const uint32_t q_addr = smem_u32(Qs), p_addr = smem_u32(Ps);
    auto issue_scores = [&](int c) {                   // S[c & 1] = Q K_c^T
      const uint32_t k_addr = smem_u32(St + (size_t)(c % stages) * kStage);
      const uint32_t d = tmem;
#pragma unroll
      for (int j = 0; j < NB; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_f16(d, umma_desc(q_addr + j * kQBlock) + (uint64_t)(2 * k), umma_desc(k_addr + j * kKvBlock) + (uint64_t)(2 * k),
                   idesc_s, (j | k) ? 1u : 0u);
      umma_commit(&s_full);
      umma_commit(&k_empty[c % stages]);
    };
    bool ok = n_chunks > 0;
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&q_full, 0, &abort_flag));
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&k_full[0], 0, &abort_flag));
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (leader) issue_scores(0);
      __syncwarp();
    }
    for (int c = 0; ok && c < n_chunks; ++c) {
      const int st = c % stages, round = c / stages;
      ok = __all_sync(0xffffffffu, mbar_wait(&p_ready, c & 1, &abort_flag));      // P_c written, S and O read
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&v_full[st], round & 1, &abort_flag));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (leader) {
        // O_c = P_c V_c: 8 steps of 16 keys; V is the MN-major operand (128-byte rows of 64 head dims, one row per key:
        // the next 8 keys are 1024 bytes on, a step of 16 keys 2048 bytes), one N = 64 MMA per 64-wide block of the head dim
        const uint32_t v_addr = smem_u32(St + (size_t)st * kStage) + NB * kKvBlock;
#pragma unroll
        for (int k = 0; k < kChunk / 16; ++k) {
          const uint64_t adesc = umma_desc(p_addr + (uint32_t)(k >> 2) * kQBlock) + (uint64_t)(2 * (k & 3));
#pragma unroll
          for (int j = 0; j < NB; ++j)
            umma_f16(tmem + kChunk + 64 * j, adesc, umma_desc_mn(v_addr + j * kKvBlock + (uint32_t)k * 2048), idesc_o, k ? 1u : 0u);
        }
        umma_commit(&o_full);
        umma_commit(&v_empty[st]);
      }
      __syncwarp();
      if (c + 1 < n_chunks) {                          // scores of the next chunk (the softmax has read this chunk's)
        const int st1 = (c + 1) % stages, round1 = (c + 1) / stages;
        ok = __all_sync(0xffffffffu, mbar_wait(&k_full[st1], round1 & 1, &abort_flag));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (leader) issue_scores(c + 1);
        __syncwarp();
      }
    }
  } else {
    // ---------------- softmax.  Warp w may touch TMEM lanes 32 (w % 4) .. + 31; an M = 64 accumulator keeps row r in lane
    // 32 (r / 16) + r % 16, so a warp owns 16 rows.  They are read as accumulator fragments (all 32 lanes busy): this
    // thread holds rows row_a and row_a + 8, two adjacent columns of every group of 8.
    pdl_wait();                                        // these warps write the output rows
    const int ga = rb * kRows + row_a, gb = ga + 8;
    const bool live_a = ga < n_rows, live_b = gb < n_rows;
    u64 ma0 = 0, ma1 = 0, mb0 = 0, mb1 = 0;
    if (live_a) { ma0 = meta->mask[ga][0]; ma1 = meta->mask[ga][1]; }
    if (live_b) { mb0 = meta->mask[gb][0]; mb1 = meta->mask[gb][1]; }
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    auto add_output = [&]() {                          // acc += O of the chunk whose P V has completed
#pragma unroll
      for (int hb = 0; hb < DH / 64; ++hb) {
        uint32_t r[32];
        tmem_ld_frag64(lane_addr + kChunk + 64 * hb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[hb * 32 + i] += __uint_as_float(r[i]);
      }
    };
    bool ok = true;
    for (int c = 0; c < n_chunks; ++c) {
      ok = __all_sync(0xffffffffu, mbar_wait(&s_full, c & 1, &abort_flag));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (c > 0) {             // the previous chunk's output (its P V was issued before these scores, so it is complete):
                               // added while the running output is still at the previous chunk's scale
        ok = __all_sync(0xffffffffu, mbar_wait(&o_full, (c - 1) & 1, &abort_flag));
        if (!ok) break;
        add_output();
      }
      uint32_t sr[kChunk / 2];
      tmem_ld_frag64(lane_addr, sr);
      tmem_ld_frag64(lane_addr + 64, sr + 32);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      float s[kChunk / 2];
      const int key0 = s_lo + c * kChunk;
      float tmax_a = -INFINITY, tmax_b = -INFINITY;
      // visibility of the chunk's 128 keys for the two rows, as bit vectors already shifted to this thread's first column
      // (key0 + 2 qd): committed slots are visible to every live row, slot base + m iff bit m of the row's ancestor mask
      u64 va0, va1, vb0, vb1;
      chunk_visibility(ma0, ma1, live_a, base - key0, 2 * qd, va0, va1);
      chunk_visibility(mb0, mb1, live_b, base - key0, 2 * qd, vb0, vb1);
      if (base - key0 >= kChunk && live_a && live_b) {                       // committed context: nothing is masked
#pragma unroll
        for (int i = 0; i < kChunk / 2; ++i) s[i] = __uint_as_float(sr[i]);
      } else {
#pragma unroll
        for (int i = 0; i < kChunk / 2; ++i) {
          const int bit = 8 * (i >> 2) + (i & 1);                            // column of this register minus 2 qd
          const u64 w = ((i >> 1) & 1) ? (bit < 64 ? vb0 : vb1) : (bit < 64 ? va0 : va1);
          s[i] = ((w >> (bit & 63)) & 1ull) ? __uint_as_float(sr[i]) : -INFINITY;       // raw scores; the scale joins the exponent below
        }
      }
#pragma unroll
      for (int i = 0; i < kChunk / 2; ++i) {
        if ((i >> 1) & 1) tmax_b = fmaxf(tmax_b, s[i]);
        else tmax_a = fmaxf(tmax_a, s[i]);
      }
      tmax_a = fmaxf(tmax_a, __shfl_xor_sync(0xffffffffu, tmax_a, 1));
      tmax_a = fmaxf(tmax_a, __shfl_xor_sync(0xffffffffu, tmax_a, 2));
      tmax_b = fmaxf(tmax_b, __shfl_xor_sync(0xffffffffu, tmax_b, 1));
      tmax_b = fmaxf(tmax_b, __shfl_xor_sync(0xffffffffu, tmax_b, 2));
      const float mn_a = fmaxf(m_a, tmax_a * scale_log2), mn_b = fmaxf(m_b, tmax_b * scale_log2);     // base-2 logits
      // a row that has seen no visible key yet (m = -inf) holds zeros: any finite factor will do
      const float ca = m_a == -INFINITY ? 1.f : ex2_approx(m_a - mn_a);
      const float cb = m_b == -INFINITY ? 1.f : ex2_approx(m_b - mn_b);
      if (ca != 1.f || cb != 1.f) {                    // the running maximum moved: bring the running output to the new scale
#pragma unroll
        for (int i = 0; i < DH / 2; ++i) acc[i] *= ((i >> 1) & 1) ? cb : ca;
      }
      const float sub_a = mn_a == -INFINITY ? 0.f : mn_a, sub_b = mn_b == -INFINITY ? 0.f : mn_b;
      float ps_a = 0.f, ps_b = 0.f;
#pragma unroll
      for (int rep = 0; rep < kChunk / 8; ++rep) {
        float p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          p[e] = ex2_approx(fmaf(s[rep * 4 + e], scale_log2, -(e < 2 ? sub_a : sub_b)));
        }
        ps_a += p[0] + p[1];
        ps_b += p[2] + p[3];
        // P block rep / 8 (64 keys each): row r, 16-byte chunk (rep % 8) of its 128-byte row sits at chunk ^ (r % 8)
        uint8_t* blk = Ps + (rep >> 3) * kQBlock + ((((rep & 7) ^ (row_a & 7)) << 4) + qd * 4);
        *reinterpret_cast<uint32_t*>(blk + row_a * 128) = pack_bf16(p[0], p[1]);
        *reinterpret_cast<uint32_t*>(blk + (row_a + 8) * 128) = pack_bf16(p[2], p[3]);
      }
      l_a = l_a * ca + ps_a;                           // this thread's share of the row sums (added up at the end)
      l_b = l_b * cb + ps_b;
      m_a = mn_a;
      m_b = mn_b;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // P is read by the tensor core's async proxy
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(&p_ready);
    }
    if (ok && n_chunks > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(&o_full, (n_chunks - 1) & 1, &abort_flag));
      if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        add_output();
      }
    }
    l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
    l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
    if (!ok) {                                         // a wait gave up: contribute nothing
#pragma unroll
      for (int i = 0; i < DH / 2; ++i) acc[i] = 0.f;
      m_a = m_b = -INFINITY;
      l_a = l_b = 0.f;
    }
  }

  // ---------------- all tensor-core work of this CTA is complete (or abandoned): free tensor memory, then merge
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && prm.err_flag) *prm.err_flag = AMPH_ERR_TIMEOUT;
  constexpr float kLn2 = 0.6931471805599453f;          // the running maximum is kept in base-2 units
  if constexpr (MERGE) {
    // park the partial output and (max, sum); the K / V ring is free now
    float* Os = reinterpret_cast<float*>(St);                       // [64][DH]
    float* MLs = Os + kRows * DH;                                   // [64][2]
    if (warp >= 2) {
#pragma unroll
      for (int rep = 0; rep < DH / 8; ++rep) {
        *reinterpret_cast<float2*>(Os + row_a * DH + 8 * rep + 2 * qd) = make_float2(acc[4 * rep], acc[4 * rep + 1]);
        *reinterpret_cast<float2*>(Os + (row_a + 8) * DH + 8 * rep + 2 * qd) = make_float2(acc[4 * rep + 2], acc[4 * rep + 3]);
      }
      if (qd == 0) {
        *reinterpret_cast<float2*>(MLs + row_a * 2) = make_float2(m_a * kLn2, l_a);
        *reinterpret_cast<float2*>(MLs + (row_a + 8) * 2) = make_float2(m_b * kLn2, l_b);
      }
    }
    cluster_sync_all();
    // CTA `split` of the S in the cluster merges rows split, split + S, ...; one warp per row, a lane per 4 columns
    const int S = gridDim.y;
    const uint32_t os0 = smem_u32(Os), ml0 = smem_u32(MLs);
    for (int r = split + S * warp; r < kRows; r += S * (kThreads / 32)) {
      const int gr = rb * kRows + r;
      if (gr >= prm.rows_cap) continue;
      // every remote load of the row is issued before the first use: one round trip through the cluster
      float2 ml = make_float2(-INFINITY, 0.f);
      if (lane < S) ml = ld_peer2(peer_smem(ml0 + (uint32_t)r * 8, (uint32_t)lane));
      float4 v[8];
#pragma unroll
      for (int s = 0; s < 8; ++s)
        v[s] = (s < S && lane * 4 < DH) ? ld_peer4(peer_smem(os0 + (uint32_t)(r * DH + lane * 4) * 4, (uint32_t)s))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
      float M = ml.x;
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      const float wgt = ml.x == -INFINITY ? 0.f : expf(ml.x - M);
      float den = ml.y * wgt;
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const float ws = __shfl_sync(0xffffffffu, wgt, s);
        if (s < S && ws != 0.f) { a.x += v[s].x * ws; a.y += v[s].y * ws; a.z += v[s].z * ws; a.w += v[s].w * ws; }
      }
      if (lane * 4 < DH) {
        const float inv = den > 0.f ? 1.0f / den : 0.f;
        uint2 u;
        u.x = pack_bf16(a.x * inv, a.y * inv);
        u.y = pack_bf16(a.z * inv, a.w * inv);
        *reinterpret_cast<uint2*>(prm.out + (size_t)(row_base + gr) * prm.n_heads * DH + h * DH + lane * 4) = u;
      }
    }
    cluster_sync_all();                                // nobody leaves while a peer may still read its shared memory
  } else {
    if (warp >= 2) {
      const int ga = rb * kRows + row_a;
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const int gr = ga + 8 * hi;
        if (gr >= prm.rows_cap) continue;
        const size_t o = ((size_t)split * prm.n_heads + h) * prm.rows_cap + gr;
#pragma unroll
        for (int rep = 0; rep < DH / 8; ++rep)
          *reinterpret_cast<float2*>(prm.po + o * DH + 8 * rep + 2 * qd) = make_float2(acc[4 * rep + 2 * hi], acc[4 * rep + 2 * hi + 1]);
        if (qd == 0) { prm.pml[o * 2] = (hi ? m_b : m_a) * kLn2; prm.pml[o * 2 + 1] = hi ? l_b : l_a; }
      }
    }
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct AttnTc {
  EncodeFn encode = nullptr;
  int sm_count = 148;
  std::map<std::tuple<const void*, int, int>, CUtensorMap> q_maps;          // (q buffer, rows, d)
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> kv_maps;    // (cache, heads, max_ctx, head_dim)

  const CUtensorMap* q_map(const void* q, int rows, int d) {
    auto key = std::make_tuple(q, rows, d);
    auto it = q_maps.find(key);
    if (it != q_maps.end()) return &it->second;
    CUtensorMap m;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kRows};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return nullptr;
    return &(q_maps[key] = m);
  }
  // one layer's K (or V) cache [head][slot][head_dim] as (head dim, slot, head); a box is 64 dims x 128 slots of one head
  const CUtensorMap* kv_map(const void* c, int heads, int max_ctx, int dh) {
    auto key = std::make_tuple(c, heads, max_ctx, dh);
    auto it = kv_maps.find(key);
    if (it != kv_maps.end()) return &it->second;
    CUtensorMap m;
    const cuuint64_t dims[3] = {(cuuint64_t)dh, (cuuint64_t)max_ctx, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)dh * 2, (cuuint64_t)max_ctx * dh * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kChunk, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(c), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return nullptr;
    return &(kv_maps[key] = m);
  }
};

AttnTc* attn_tc_create() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  int dev = 0, major = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (major != 10) return nullptr;
  AttnTc* a = new AttnTc();
  a->encode = (EncodeFn)fn;
  cudaDeviceGetAttribute(&a->sm_count, cudaDevAttrMultiProcessorCount, dev);
  return a;
}

void attn_tc_destroy(AttnTc* a) { delete a; }

// KV splits per head: a split owns at least one chunk of 128 keys; the splits of a head form one cluster.
int attn_tc_splits(const AttnTc* a, int keys_bound, int n_heads, int rows, int max_splits) {
  (void)a; (void)n_heads; (void)rows;
  int s = (keys_bound + kChunk - 1) / kChunk;
  if (s > max_splits) s = max_splits;
  // clusters of 8 measured 3-6 us per launch slower than clusters of 7 at every context from 1k to 8k tokens (they are
  // harder to place beside the resident projection CTAs), so a head is cut into at most 7 splits
  if (s > 7) s = 7;
  return s < 1 ? 1 : s;
}

// Ring depth.  At head_dim 128 a stage is 64 KB: one stage keeps the CTA at 97 KB, so that two CTAs (or one and a
// projection CTA of the next kernel) share an SM, and the loads of one CTA overlap the arithmetic of the other.
int attn_tc_stages(int keys_bound, int splits, int head_dim) {
  int len = (keys_bound + splits - 1) / splits;
  const int chunks = (len + kChunk - 1) / kChunk;
  int stages = head_dim == 64 && chunks > 1 ? 2 : 1;
  return stages;
}

namespace {

template <int DH, int NG>
bool launch_t(AttnTc* a, const void* q, int q_rows_cap, int G, const KvView* kv, const RowMeta* const* meta, AttnScratch sc, int rows,
              int n_heads, int max_ctx, int splits, int keys_bound, cudaStream_t st, void* merged_out, int* err_flag) {
  const CUtensorMap* mq = a->q_map(q, q_rows_cap, n_heads * DH);
  if (!mq) return false;
  AttnMaps<NG> maps;
  AttnParams<NG> prm;
  if (G > NG) return false;
  memset(&maps, 0, sizeof maps);
  memset(&prm, 0, sizeof prm);
  maps.q = *mq;
  for (int g = 0; g < G; ++g) {
    const CUtensorMap* mk = a->kv_map(kv[g].k, n_heads, max_ctx, DH);
    const CUtensorMap* mv = a->kv_map(kv[g].v, n_heads, max_ctx, DH);
    if (!mk || !mv) return false;
    maps.k[g] = *mk;
    maps.v[g] = *mv;
    prm.meta[g] = meta[g];
    if (g > 0 && kv[g].k == kv[0].k) prm.same_cache = 1;
  }
  constexpr int NB = DH / 64;
  constexpr size_t stage = 2 * NB * (size_t)kChunk * 128;
  const int stages = attn_tc_stages(keys_bound, splits, DH);
  prm.nrb = (rows + kRows - 1) / kRows;
  prm.rpg = rows;
  prm.po = sc.o;
  prm.pml = sc.ml;
  prm.out = (bf16*)merged_out;
  prm.rows_cap = rows;
  prm.n_heads = n_heads;
  prm.max_ctx = max_ctx;
  prm.stages = stages;
  prm.err_flag = err_flag;
  const size_t smem = 1024 + NB * (size_t)kRows * 128 + 2 * (size_t)kRows * 128 + stages * stage;
  dim3 grid(n_heads, splits, G * prm.nrb);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  if (merged_out != nullptr) {
    cudaFuncSetAttribute(tree_attn_tc_kernel<DH, true, NG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 1;
    at[1].val.clusterDim.y = splits;
    at[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<DH, true, NG>, maps, prm) == cudaSuccess;
  }
  cudaFuncSetAttribute(tree_attn_tc_kernel<DH, false, NG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<DH, false, NG>, maps, prm) == cudaSuccess;
}

}  // namespace

// q: bf16 [q_rows_cap][n_heads * head_dim].  keys_bound: host-side upper bound of committed slots + rows of this call.
// merged_out != NULL: the splits (<= 8) run as one cluster and write the final bf16 rows; otherwise partial results go to
// sc for attn_combine_kernel.  Returns false (nothing launched) if the form is not available.
bool launch_tree_attention_tc(AttnTc* a, const void* q, int q_rows_cap, KvView kv, const RowMeta* meta, AttnScratch sc, int rows,
                              int n_heads, int head_dim, int max_ctx, int splits, int keys_bound, cudaStream_t st,
                              void* merged_out, int* err_flag) {
  if (!a || splits < 1 || (merged_out && splits > 8)) return false;
  if (q_rows_cap < 1) return false;                   // rows of a Q box past the end of the buffer read as zeros
  if (head_dim == 64)
    return launch_t<64, 1>(a, q, q_rows_cap, 1, &kv, &meta, sc, rows, n_heads, max_ctx, splits, keys_bound, st, merged_out, err_flag);
  if (head_dim == 128)
    return launch_t<128, 1>(a, q, q_rows_cap, 1, &kv, &meta, sc, rows, n_heads, max_ctx, splits, keys_bound, st, merged_out, err_flag);
  return false;
}

// The same for G row groups in ONE launch (grid.z = groups x row blocks): group g's `rows` query rows start at row g * rows of
// q and of merged_out, read the cache kv[g] and the row table meta[g].  Merged form only (splits <= 8).
bool launch_tree_attention_tc_groups(AttnTc* a, const void* q, int q_rows_cap, int G, const KvView* kv, const RowMeta* const* meta,
                                     int rows, int n_heads, int head_dim, int max_ctx, int splits, int keys_bound, cudaStream_t st,
                                     void* merged_out, int* err_flag) {
  if (!a || G < 1 || G > kMaxGroups || splits < 1 || splits > 8 || !merged_out || q_rows_cap < G * rows) return false;
  AttnScratch none = {nullptr, nullptr};
  if (head_dim == 64)
    return launch_t<64, kMaxGroups>(a, q, q_rows_cap, G, kv, meta, none, rows, n_heads, max_ctx, splits, keys_bound, st, merged_out, err_flag);
  if (head_dim == 128)
    return launch_t<128, kMaxGroups>(a, q, q_rows_cap, G, kv, meta, none, rows, n_heads, max_ctx, splits, keys_bound, st, merged_out, err_flag);
  return false;
}

}  // namespace amph
