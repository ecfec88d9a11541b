// Skinny bf16 projection on the 5th-generation tensor cores:  Y^T[out][rows] = W[out][in] . X^T.
//
// The weight matrix is the 128-row MMA operand A (K-major, streamed once from HBM by TMA), the few
// activation rows are operand B (N = 16..128 rows, K-major, re-read from L2), the fp32 accumulator
// lives in tensor memory.  One CTA owns one 128-row weight tile and one K-range (split-K); partial
// sums go to global memory as P[split][row][feature] and are reduced, in a fixed order, by the
// kernel that consumes them.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns the TMEM
// allocation), warps 2-5 = epilogue (TMEM -> registers -> global).  Every barrier wait is bounded:
// if one gives up the CTA sets *err_flag, drains its own copies and exits cleanly.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>

#include <map>
#include <tuple>

#include "amph.h"
#include "amph_internal.cuh"
#include "gemm_tc.cuh"

namespace amph {

namespace {

constexpr int kTileM = 128;           // weight rows per CTA (UMMA M)
constexpr int kTileK = 64;            // bf16 elements per 128-byte swizzle row
constexpr int kUmmaK = 16;            // K per tcgen05.mma for 16-bit inputs
constexpr int kStageKb = 2;           // 64-wide K blocks fetched by one TMA copy (one pipeline stage) when both operands' stage fits twice per CTA
constexpr int kMaxSeg = 8;
constexpr int kThreads = 192;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // a barrier wait gives up after one second

struct TmapPack {
  CUtensorMap w[kMaxSeg];
  CUtensorMap x;
};

struct TcParams {
  float* P;
  size_t split_stride;      // floats between splits
  int ld;                   // floats per row of P
  int tiles_per_seg;        // out / 128
  int kblocks;              // in / 64
  int splits;
  int nt;                   // activation rows of one MMA (multiple of 16, at most 128)
  int nblk;                 // row blocks of nt rows that share each weight tile (1..4; more than 1 only with nt = 128)
  int rows;                 // live rows (only these are stored)
  int stages;
  int l2_prefetch;          // weight tiles (beyond the ring) each CTA pulls into L2 before it waits
  int ks;                   // K blocks per stage (depth of the tensor maps' boxes): kStageKb, or 1 for many activation rows
  // SWIGLU launches: a tile is 64 gate rows + the 64 up rows of the same features; the epilogue writes
  //   act[row][feature] = silu(gate * inv_rms(row)) * (up * inv_rms(row))   (bf16, row pitch f)
  __nv_bfloat16* act;
  int f;
  int up_first;             // the tensor map's outer index 0 is the up matrix (it has the lower address)
  RowScale rs;
  // ROPE launches (q / k / v projection): a tile is 32 rotation pairs of one head, rows [32 j, 32 j + 32) and
  // [dh/2 + 32 j, dh/2 + 32 j + 32); the epilogue rotates, scales and writes the query rows and the cache rows
  __nv_bfloat16* q;         // [rows][n_heads * dh]
  __nv_bfloat16* kc;        // [n_heads][max_ctx][dh]
  __nv_bfloat16* vc;
  const RowMeta* meta;      // slot of every row, number of live rows
  const float2* rope;       // [rows][dh / 2] (cos, sin)
  int n_heads, dh, max_ctx;
  int* err_flag;
  unsigned long long wait_limit_ns;   // a barrier wait gives up after this long
  uint32_t extra_tx;                   // self-test only: bytes the first stage's barrier expects beyond what is copied
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// Bounded wait; returns false (and raises the shared abort flag) if the phase never completes or
// another role already gave up.
__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = now_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > limit_ns) break;
    }
  }
  *abort_flag = 1;
  return false;
}

// One lane of a converged warp.  TMA and MMA instructions are issued by the elected lane while the other
// lanes stay with it: issued by a lone thread of a diverged warp, a tcgen05.mma costs about 210 clocks
// instead of the 48 that a 128 x 64 x 16 MMA occupies the tensor pipe (both measured), which would cap
// a CTA at about 37 GB/s of weights.
__device__ __forceinline__ bool elect_one() {
  uint32_t e;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
  return e != 0;
}

// The operands are described to the TMA unit as 3-D tensors (64 columns, rows, K block): one copy brings
// kStageKb consecutive K blocks of a row range, each landing as its own 128-byte-swizzled K-major tile.
// An SM retires roughly one tiled copy per 400 clocks whatever its size (measured with copies of 8 to
// 32 KB), so larger copies are what lets L2-resident weights arrive faster than HBM delivers them.
// The first coordinate is always 0 (16-byte rule); K blocks past the end of the tensor read as zeros.
// Asks the TMA unit to bring the weight tiles of one stage into L2 (no shared-memory destination, no barrier).
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* map, int row, int kb) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(0), "r"(row), "r"(kb) : "memory");
}

// 4-D form for the fused gate / up launch: (column, row, K block, matrix) with the distance between the two weight
// matrices as the outermost stride, so ONE copy brings the gate and the up rows of a tile.
// Weight tiles are read exactly once per pass: they are loaded with an evict-first L2 policy so that the stream of
// weights (100-180 MB per launch, about the size of L2) does not push out the activations, partial sums and KV rows
// that the neighbouring kernels re-read from L2 (measured: -3.8 % on the 7B step).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int row, int kb, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(0), "r"(row), "r"(kb), "r"(0), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
// (column, row, half, K block): the two 32-row halves of a rotation tile land as 64 consecutive rows per K block
__device__ __forceinline__ void tma_load_4d_kb_outer(void* dst, const CUtensorMap* map, int row, int kb, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(0), "r"(row), "r"(0), "r"(kb), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_l2_4d_kb_outer(const CUtensorMap* map, int row, int kb) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(map), "r"(0), "r"(row), "r"(0), "r"(kb) : "memory");
}
__device__ __forceinline__ void tma_prefetch_l2_4d(const CUtensorMap* map, int row, int kb) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(map), "r"(0), "r"(row), "r"(kb), "r"(0) : "memory");
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int row, int kb, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(0), "r"(row), "r"(kb), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int row, int kb, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(0), "r"(row), "r"(kb), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                                // leading-dimension offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                      // stride between 8-row groups
  d |= (uint64_t)1 << 46;                                // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                                // 128-byte swizzle
  return d;
}

// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = m (128 or 64), N = nt.
__device__ __forceinline__ uint32_t umma_idesc(int nt, int m = kTileM) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nt >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
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

// SWIGLU: the gate / up projection with SwiGLU in the epilogue.  A CTA owns 64 features and the whole K range; per K
// step it issues two M = 64 MMAs, gate rows into accumulator columns [0, nt) and up rows into [ntc, ntc + nt).  Row r
// of an M = 64 accumulator lives in TMEM lane 32 (r / 16) + r % 16 (checked on the device), so lane l < 16 of the
// epilogue warp of quarter q holds gate and up of feature 16 q + l for all rows: no exchange between warps.
//
// ROPE: the q / k / v projection with the rotary embedding and the cache write in the epilogue.  A CTA owns 64 weight
// rows that hold 32 complete rotation pairs of one head (both halves fetched by one 4-D copy) and the whole K range,
// one M = 64 MMA per K step.  The partners of a pair sit in different epilogue warps; the accumulator tile goes through
// shared memory (the ring is free by then), then every thread rotates 16 pairs of one row and writes 32-byte pieces.
enum { EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_ROPE = 2 };
constexpr int kRopePitch = 68;        // floats per activation row of the exchanged tile (64 + 4: conflict-free float4 reads)

template <int EPI>
__global__ void __launch_bounds__(kThreads)
tc_gemm_kernel(const __grid_constant__ TmapPack maps, const TcParams prm) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU, ROPE = EPI == EPI_ROPE;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ float inv_s[EPI != EPI_PARTIAL ? kTileM : 1];         // 1 / rms of the activation rows (SWIGLU, ROPE)
  __shared__ __align__(8) uint64_t full_bar[8];
  __shared__ __align__(8) uint64_t empty_bar[8];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  pdl_launch_dependents();                          // the consumer kernel may get resident and wait
  const unsigned long long limit_ns = prm.wait_limit_ns;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int seg = tile / prm.tiles_per_seg;
  int row0 = SWIGLU ? tile * (kTileM / 2) : (tile - seg * prm.tiles_per_seg) * kTileM;   // first weight row of this tile
  if constexpr (ROPE) {
    const int tph = prm.dh >> 6, tt = tile - seg * prm.tiles_per_seg;       // tiles per head = (dh / 2) / 32
    row0 = (tt / tph) * prm.dh + (tt % tph) * 32;
  }
  // K range of this split in whole stages (ks blocks), so that every copy starts on a stage boundary
  const int ks = prm.ks;
  const int units = (prm.kblocks + ks - 1) / ks;
  const int kb_lo = (int)((long long)split * units / prm.splits) * ks;
  int kb_hi = (int)((long long)(split + 1) * units / prm.splits) * ks;
  if (kb_hi > prm.kblocks) kb_hi = prm.kblocks;
  const int nkb = kb_hi - kb_lo;
  const int nit = (nkb + ks - 1) / ks;                  // pipeline iterations
  const int nt = prm.nt, stages = prm.stages;
  const uint32_t a_tile = (ROPE ? kTileM / 2 : kTileM) * kTileK * 2, b_tile = (uint32_t)nt * kTileK * 2;     // one K block of each operand
  const uint32_t a_bytes = ks * a_tile, b_bytes = ks * b_tile;
  const int nblk = EPI != EPI_PARTIAL ? 1 : prm.nblk;              // row blocks: each gets its own activation tile and accumulator
  const uint32_t b_slot = (b_bytes + 1023u) & ~1023u;
  const uint32_t stage_bytes = a_bytes + (uint32_t)nblk * b_slot;
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint32_t ntc = 32;
  while ((int)ntc < nt) ntc <<= 1;
  uint32_t tmem_cols = SWIGLU ? 2 * ntc : ntc * (uint32_t)nblk;
  if (tmem_cols == 384) tmem_cols = 512;             // allocations are powers of two

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&accum_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                                   // TMEM allocation belongs to the MMA warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;

  if (warp == 0) {
    // ---------------- TMA producer (the warp stays converged, its elected lane issues)
    const bool leader = elect_one();
    const uint64_t wpol = l2_evict_first_policy();
    const CUtensorMap* wmap = &maps.w[seg];
    if (leader) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(wmap) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.x) : "memory");
    }
    // Weights do not depend on the previous kernel: fill the ring with weight tiles first, then wait for
    // the producer of the activations, then fetch the activation tiles of those stages.
    const int npre = nit < stages ? nit : stages;
    const int npf = nit < npre + prm.l2_prefetch ? nit : npre + prm.l2_prefetch;
    if (leader) {
      for (int i = 0; i < npre; ++i) {
        // extra_tx is 0 except in the failure-path self-test, where the first barrier expects bytes that never come
        mbar_expect_tx(&full_bar[i], a_bytes + (uint32_t)nblk * b_bytes + (i == 0 ? prm.extra_tx : 0u));
        if (SWIGLU) tma_load_4d(smem + (size_t)i * stage_bytes, wmap, row0, kb_lo + i * ks, &full_bar[i], wpol);
        else if (ROPE) tma_load_4d_kb_outer(smem + (size_t)i * stage_bytes, wmap, row0, kb_lo + i * ks, &full_bar[i], wpol);
        else tma_load_3d(smem + (size_t)i * stage_bytes, wmap, row0, kb_lo + i * ks, &full_bar[i], wpol);
      }
      // While the previous kernel still runs, HBM would idle: pull the next weight tiles into L2 as well.
      for (int i = npre; i < npf; ++i) {
        if (SWIGLU) tma_prefetch_l2_4d(wmap, row0, kb_lo + i * ks);
        else if (ROPE) tma_prefetch_l2_4d_kb_outer(wmap, row0, kb_lo + i * ks);
        else tma_prefetch_l2_3d(wmap, row0, kb_lo + i * ks);
      }
    }
    __syncwarp();
    pdl_wait();
    if (leader)
      for (int i = 0; i < npre; ++i)
        for (int z = 0; z < nblk; ++z)
          tma_load_3d(smem + (size_t)i * stage_bytes + a_bytes + (size_t)z * b_slot, &maps.x, z * nt, kb_lo + i * ks, &full_bar[i]);
    __syncwarp();
    int issued = npre;
    for (int i = npre; i < nit; ++i) {
      const int s = i % stages, round = i / stages;
      if (!__all_sync(0xffffffffu, mbar_wait(&empty_bar[s], (round & 1) ^ 1, &abort_flag, limit_ns))) break;
      if (leader) {
        uint8_t* a = smem + (size_t)s * stage_bytes;
        mbar_expect_tx(&full_bar[s], a_bytes + (uint32_t)nblk * b_bytes);
        if (SWIGLU) tma_load_4d(a, wmap, row0, kb_lo + i * ks, &full_bar[s], wpol);
        else if (ROPE) tma_load_4d_kb_outer(a, wmap, row0, kb_lo + i * ks, &full_bar[s], wpol);
        else tma_load_3d(a, wmap, row0, kb_lo + i * ks, &full_bar[s], wpol);
        for (int z = 0; z < nblk; ++z) tma_load_3d(a + a_bytes + (size_t)z * b_slot, &maps.x, z * nt, kb_lo + i * ks, &full_bar[s]);
      }
      __syncwarp();
      issued = i + 1;
    }
    if (abort_flag && lane == 0) {                     // drain: let every copy that was issued land
      const int first = issued > stages ? issued - stages : 0;
      for (int i = first; i < issued; ++i) {
        const int s = i % stages, round = i / stages;
        const unsigned long long t0 = now_ns();
        while (!mbar_try(&full_bar[s], round & 1) && now_ns() - t0 < limit_ns) {}
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (the warp stays converged, its elected lane issues)
    const bool leader = elect_one();
    const uint32_t idesc = umma_idesc(nt, EPI != EPI_PARTIAL ? kTileM / 2 : kTileM);
    bool ok = true;
    for (int i = 0; i < nit; ++i) {
      const int s = i % stages, round = i / stages;
      ok = __all_sync(0xffffffffu, mbar_wait(&full_bar[s], round & 1, &abort_flag, limit_ns));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (leader) {
        const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
        const int nk = nkb - i * ks < ks ? nkb - i * ks : ks;   // blocks of the stage inside the K range
        for (int kk = 0; kk < nk; ++kk) {
          const uint64_t bdesc = umma_desc(a_addr + a_bytes + (uint32_t)kk * b_tile);
          if constexpr (SWIGLU) {
            // the copy landed as [matrix][K block][64 rows]: two half tiles per K block, one MMA each
            const uint32_t half = a_tile / 2;
            const int gi = prm.up_first ? 1 : 0;
            const uint64_t gdesc = umma_desc(a_addr + (uint32_t)(gi * ks + kk) * half);
            const uint64_t udesc = umma_desc(a_addr + (uint32_t)((1 - gi) * ks + kk) * half);
#pragma unroll
            for (int k = 0; k < kTileK / kUmmaK; ++k) {
              umma_f16(tmem_d, gdesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (i | kk | k) ? 1u : 0u);
              umma_f16(tmem_d + ntc, udesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (i | kk | k) ? 1u : 0u);
            }
          } else {
            const uint64_t adesc = umma_desc(a_addr + (uint32_t)kk * a_tile);
            for (int z = 0; z < nblk; ++z) {             // the weight tile is read from shared memory once per row block
              const uint64_t bz = umma_desc(a_addr + a_bytes + (uint32_t)z * b_slot + (uint32_t)kk * b_tile);
#pragma unroll
              for (int k = 0; k < kTileK / kUmmaK; ++k)    // +32 bytes (2 x 16 B) per K step inside the swizzle row
                umma_f16(tmem_d + (uint32_t)z * ntc, adesc + (uint64_t)(2 * k), bz + (uint64_t)(2 * k), idesc, (i | kk | k) ? 1u : 0u);
            }
          }
        }
        umma_commit(&empty_bar[s]);                    // frees the stage once these MMAs have read it
      }
      __syncwarp();
    }
    if (ok && leader) umma_commit(&accum_bar);
    __syncwarp();
  } else {
    // ---------------- epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
    const int quarter = warp & 3;
    pdl_wait();                                      // P may still be read by the kernel before this one
    if constexpr (EPI != EPI_PARTIAL) {              // 1 / rms of the rows, while the main loop runs
      const int et = threadIdx.x - 64;
      if (et < prm.rows) inv_s[et] = row_scale(prm.rs, et);
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    const bool ok = __all_sync(0xffffffffu, nkb > 0 ? mbar_wait(&accum_bar, 0, &abort_flag, limit_ns) : false);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if constexpr (SWIGLU) {
      // lanes 0..15 of the warp of quarter q hold features 16 q .. 16 q + 15 of the tile (gate and up alike); the
      // upper half of the warp takes over the second half of each block of 16 rows
      const int feat = row0 + quarter * 16 + (lane & 15);
      const int jb = (lane >> 4) * 8;
      for (int c0 = 0; c0 < nt && c0 < prm.rows; c0 += 16) {
        uint32_t g[16], u[16];
        const uint32_t taddr = tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
        if (ok) {
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
              : "=r"(g[0]), "=r"(g[1]), "=r"(g[2]), "=r"(g[3]), "=r"(g[4]), "=r"(g[5]), "=r"(g[6]), "=r"(g[7]),
                "=r"(g[8]), "=r"(g[9]), "=r"(g[10]), "=r"(g[11]), "=r"(g[12]), "=r"(g[13]), "=r"(g[14]), "=r"(g[15])
              : "r"(taddr)
              : "memory");
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
              : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
                "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
              : "r"(taddr + ntc)
              : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) g[j] = u[j] = 0u;
        }
        float gv[8], uv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {                  // rows c0 + 8 .. c0 + 15 move to lanes 16 .. 31
          const uint32_t gh = __shfl_sync(0xffffffffu, g[8 + j], lane & 15), uh = __shfl_sync(0xffffffffu, u[8 + j], lane & 15);
          gv[j] = __uint_as_float(lane < 16 ? g[j] : gh);
          uv[j] = __uint_as_float(lane < 16 ? u[j] : uh);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = c0 + jb + j;
          if (r < prm.rows) {
            const float sc = inv_s[r];
            const float t = gv[j] * sc;
            prm.act[(size_t)r * prm.f + feat] = __float2bfloat16(__fdividef(t, 1.0f + __expf(-t)) * (uv[j] * sc));
          }
        }
      }
    } else if constexpr (ROPE) {
      // lane l < 16 of the warp of quarter q holds tile row 16 q + l (pair member lo for q < 2, hi for q >= 2) for all
      // activation rows: park the tile as ex[activation row][tile row] in the ring, which no copy or MMA touches any more
      float* ex = reinterpret_cast<float*>(smem);
      for (int c0 = 0; c0 < nt; c0 += 16) {
        uint32_t v[16];
        if (ok) {
          const uint32_t taddr = tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
              : "r"(taddr)
              : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
        if (lane < 16) {
#pragma unroll
          for (int j = 0; j < 16; ++j) ex[(c0 + j) * kRopePitch + quarter * 16 + lane] = __uint_as_float(v[j]);
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      // thread e: activation row e / 2, pairs 16 (e % 2) .. + 15 of the tile
      const int et = threadIdx.x - 64;
      const int r = et >> 1, t0 = (et & 1) * 16;
      if (r < prm.rows) {
        const int half = prm.dh >> 1;
        const int tt = tile - seg * prm.tiles_per_seg, tph = prm.dh >> 6;
        const int h = tt / tph, i0 = (tt % tph) * 32 + t0;               // head, first pair index of this thread
        const float sc = inv_s[r];
        float a[16], b[16];
#pragma unroll
        for (int j = 0; j < 16; j += 4) {
          const float4 va = *reinterpret_cast<const float4*>(ex + r * kRopePitch + t0 + j);
          const float4 vb = *reinterpret_cast<const float4*>(ex + r * kRopePitch + 32 + t0 + j);
          a[j] = va.x * sc; a[j + 1] = va.y * sc; a[j + 2] = va.z * sc; a[j + 3] = va.w * sc;
          b[j] = vb.x * sc; b[j + 1] = vb.y * sc; b[j + 2] = vb.z * sc; b[j + 3] = vb.w * sc;
        }
        uint32_t lo[8], hi[8];
        if (seg < 2) {                                 // queries and keys: rotate pair (i, i + dh / 2) by the row's angle
          const float2* cs = prm.rope + (size_t)r * half + i0;
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const float4 c2 = *reinterpret_cast<const float4*>(cs + j);        // (cos, sin) of pairs j, j + 1
            const __nv_bfloat162 l2 = __floats2bfloat162_rn(a[j] * c2.x - b[j] * c2.y, a[j + 1] * c2.z - b[j + 1] * c2.w);
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(b[j] * c2.x + a[j] * c2.y, b[j + 1] * c2.z + a[j + 1] * c2.w);
            lo[j >> 1] = *reinterpret_cast<const uint32_t*>(&l2);
            hi[j >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const __nv_bfloat162 l2 = __floats2bfloat162_rn(a[j], a[j + 1]), h2 = __floats2bfloat162_rn(b[j], b[j + 1]);
            lo[j >> 1] = *reinterpret_cast<const uint32_t*>(&l2);
            hi[j >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        }
        __nv_bfloat16* dst = nullptr;
        if (seg == 0) {
          dst = prm.q + (size_t)r * prm.n_heads * prm.dh + h * prm.dh + i0;
        } else {
          const int slot = prm.meta->slot[r];
          if (r < prm.meta->n_rows && slot >= 0 && slot < prm.max_ctx)
            dst = (seg == 1 ? prm.kc : prm.vc) + ((size_t)h * prm.max_ctx + slot) * prm.dh + i0;
        }
        if (dst != nullptr) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(dst + 8) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
          *reinterpret_cast<uint4*>(dst + half) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(dst + half + 8) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        }
      }
    } else {
    const int feat = seg * prm.tiles_per_seg * kTileM + row0 + quarter * 32 + lane;
    float* out = prm.P + (size_t)split * prm.split_stride + feat;
    for (int z = 0; z < nblk; ++z) {
      const int rbase = z * nt;
      for (int c0 = 0; c0 < nt; c0 += 16) {
        if (rbase + c0 >= prm.rows) break;
        uint32_t v[16];
        if (ok) {
          const uint32_t taddr = tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)z * ntc + (uint32_t)c0;
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
              : "r"(taddr)
              : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;          // empty K-range or aborted: contribute zeros
        }
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (rbase + c0 + j < prm.rows) out[(size_t)(rbase + c0 + j) * prm.ld] = __uint_as_float(v[j]);
      }
    }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(tmem_cols) : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && prm.err_flag) *prm.err_flag = AMPH_ERR_TIMEOUT;
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct TcGemm {
  EncodeFn encode = nullptr;
  int* err_flag = nullptr;
  int n_x = 0;
  void* xptr[16];
  int xrows[16], xcols[16];
  std::map<std::tuple<const void*, int, int, int, int>, CUtensorMap> cache;   // (ptr, rows, cols, box rows, box K blocks)
  int sm_count = 148;
  int max_smem = 0;
  unsigned long long wait_limit_ns = kWaitLimitNs;
  uint32_t extra_tx = 0;
  std::map<std::tuple<const void*, const void*, int, int, int>, CUtensorMap> pair_cache;   // (lower, upper matrix, rows, cols, K blocks)

  // Two [rows, cols] matrices as one 4-D tensor (column, row, K block, matrix): a box of 64 rows of both.
  const CUtensorMap* get_pair(const void* lo, const void* hi, int rows, int cols, int box_kb) {
    auto key = std::make_tuple(lo, hi, rows, cols, box_kb);
    auto it = pair_cache.find(key);
    if (it != pair_cache.end()) return &it->second;
    const uint64_t gap = (uint64_t)((const char*)hi - (const char*)lo);
    if (gap == 0 || (gap & 15) || gap >= (1ull << 40)) return nullptr;
    CUtensorMap m;
    const cuuint64_t dims[4] = {(cuuint64_t)kTileK, (cuuint64_t)rows, (cuuint64_t)cols / kTileK, 2};
    const cuuint64_t strides[3] = {(cuuint64_t)cols * 2, (cuuint64_t)kTileK * 2, (cuuint64_t)gap};
    const cuuint32_t box[4] = {(cuuint32_t)kTileK, (cuuint32_t)(kTileM / 2), (cuuint32_t)box_kb, 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(lo), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return nullptr;
    return &(pair_cache[key] = m);
  }

  // A [rows, cols] matrix as (column, row, half, K block) with the half `half_rows` rows apart: a box is 32 rows of
  // both halves, i.e. 32 rotation pairs of one head, over box_kb K blocks.
  std::map<std::tuple<const void*, int, int, int, int>, CUtensorMap> rope_cache;
  const CUtensorMap* get_rope(const void* ptr, int rows, int cols, int half_rows, int box_kb) {
    auto key = std::make_tuple(ptr, rows, cols, half_rows, box_kb);
    auto it = rope_cache.find(key);
    if (it != rope_cache.end()) return &it->second;
    CUtensorMap m;
    const cuuint64_t dims[4] = {(cuuint64_t)kTileK, (cuuint64_t)rows, 2, (cuuint64_t)cols / kTileK};
    const cuuint64_t strides[3] = {(cuuint64_t)cols * 2, (cuuint64_t)half_rows * cols * 2, (cuuint64_t)kTileK * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kTileK, 32, 2, (cuuint32_t)box_kb};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return nullptr;
    return &(rope_cache[key] = m);
  }

  const CUtensorMap* get(const void* ptr, int rows, int cols, int box_rows, int box_kb = kStageKb) {
    auto key = std::make_tuple(ptr, rows, cols, box_rows, box_kb);
    auto it = cache.find(key);
    if (it != cache.end()) return &it->second;
    CUtensorMap m;
    // (column within a K block, row, K block): stride of a row = its pitch, of a K block = 128 bytes
    const cuuint64_t dims[3] = {(cuuint64_t)kTileK, (cuuint64_t)rows, (cuuint64_t)cols / kTileK};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)kTileK * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows, (cuuint32_t)box_kb};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return nullptr;
    return &(cache[key] = m);
  }
};

TcGemm* tc_gemm_create(void* const* xbufs, const int* xrows, const int* xcols, int n, int* err_flag) {
  if (n > 16) return nullptr;
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
  TcGemm* g = new TcGemm();
  g->encode = (EncodeFn)fn;
  g->err_flag = err_flag;
  g->n_x = n;
  for (int i = 0; i < n; ++i) { g->xptr[i] = xbufs[i]; g->xrows[i] = xrows[i]; g->xcols[i] = xcols[i]; }
  cudaDeviceGetAttribute(&g->sm_count, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&g->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaFuncSetAttribute(tc_gemm_kernel<EPI_PARTIAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, g->max_smem - 2048);
  cudaFuncSetAttribute(tc_gemm_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, g->max_smem - 2048);
  cudaFuncSetAttribute(tc_gemm_kernel<EPI_ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, g->max_smem - 2048);
  return g;
}

bool tc_gemm_launch(TcGemm* g, int xb, const void* const* w, int n_seg, int out, int in, int rows, float* P,
                    size_t p_floats, int* splits_out, size_t* split_stride, cudaStream_t st) {
  if (!g || xb < 0 || xb >= g->n_x) return false;
  if (out % kTileM || in % kTileK || n_seg < 1 || n_seg > kMaxSeg || rows < 1) return false;
  if (g->xcols[xb] != in) return false;
  // up to 128 rows: one MMA of N = rows rounded up to 16; more: 2..4 row blocks of 128 rows that share every weight tile
  // (the tile is streamed from HBM once and multiplied with each block: batched verification, dense prefill)
  const int nt_all = rows <= 16 ? 16 : (rows <= 128 ? (rows + 15) / 16 * 16 : (rows + 127) / 128 * 128);
  const int nblk = nt_all <= 128 ? 1 : nt_all / 128;
  const int nt = nblk == 1 ? nt_all : 128;
  if (nblk > 4 || nt_all > g->xrows[xb]) return false;
  const int tiles = n_seg * (out / kTileM), kblocks = in / kTileK;
  const size_t ld = (size_t)n_seg * out;
  // K-splits: nearly two CTAs per SM (7/8 of the slots measured best: one split fewer costs no bandwidth and
  // saves partial sums), keep at least four 64-wide K blocks per CTA.  With several row blocks a CTA needs most of an
  // SM's shared and tensor memory: one CTA per SM.
  int splits = ((nblk == 1 ? 2 : 1) * g->sm_count * 7 / 8) / tiles;
  if (splits > kblocks / 4) splits = kblocks / 4;
  // many activation rows: a two-block stage would leave room for one CTA per SM only, so stage single blocks
  const int ks = nt <= 64 ? kStageKb : 1;
  if (splits > (kblocks + ks - 1) / ks) splits = (kblocks + ks - 1) / ks;
  if (splits > 16) splits = 16;
  while (splits > 1 && (size_t)splits * nt_all * ld > p_floats) --splits;
  if (splits < 1) splits = 1;
  if ((size_t)nt_all * ld > p_floats) return false;
  TmapPack pack;
  memset(&pack, 0, sizeof pack);
  for (int s = 0; s < n_seg; ++s) {
    if ((uintptr_t)w[s] & 15) return false;
    const CUtensorMap* m = g->get(w[s], out, in, kTileM, ks);
    if (!m) return false;
    pack.w[s] = *m;
  }
  const CUtensorMap* mx = g->get(g->xptr[xb], g->xrows[xb], in, nt, ks);
  if (!mx) return false;
  pack.x = *mx;
  const uint32_t stage_bytes = ks * kTileM * kTileK * 2 + (uint32_t)nblk * ((ks * (uint32_t)nt * kTileK * 2 + 1023u) & ~1023u);
  int stages = (int)(((nblk == 1 ? 110 : 200) * 1024) / stage_bytes);   // <= ~110 KB per CTA: two CTAs per SM (one with row blocks)
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  TcParams prm;
  prm.P = P;
  prm.nblk = nblk;
  prm.split_stride = (size_t)nt_all * ld;
  prm.ld = (int)ld;
  prm.tiles_per_seg = out / kTileM;
  prm.kblocks = kblocks;
  prm.splits = splits;
  prm.nt = nt;
  prm.rows = rows;
  prm.stages = stages;
  prm.ks = ks;
  // One more stage per CTA is asked into L2 before the dependency wait.  The TMA unit of an SM serves its copies
  // and prefetches in order, so a deeper prefetch sits in front of the activation tiles issued after the wait:
  // 1 stage measured best (0: +0.7 %, 2: +1.2 %, the former 40 MB budget: +3 % on the step).
  prm.l2_prefetch = 1;
  prm.err_flag = g->err_flag;
  prm.wait_limit_ns = g->wait_limit_ns;
  prm.extra_tx = g->extra_tx;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  launch_pdl(tc_gemm_kernel<EPI_PARTIAL>, dim3(tiles, splits), dim3(kThreads), smem, st, pack, prm);
  *splits_out = splits;
  *split_stride = prm.split_stride;
  return true;
}

bool tc_gemm_launch_swiglu(TcGemm* g, int xb, const void* w_gate, const void* w_up, int f, int in, int rows, void* act,
                           const RowScale& rs, cudaStream_t st) {
  if (!g || xb < 0 || xb >= g->n_x || !w_gate || !w_up || !act) return false;
  if (f % (kTileM / 2) || in % kTileK || rows < 1 || g->xcols[xb] != in) return false;
  if (((uintptr_t)w_gate | (uintptr_t)w_up) & 15) return false;
  const int nt = rows <= 16 ? 16 : (rows + 15) / 16 * 16;
  if (nt > 64 || nt > g->xrows[xb]) return false;          // two accumulators of nt columns; stages of two K blocks
  const int ks = kStageKb, kblocks = in / kTileK, tiles = f / (kTileM / 2);
  const bool up_first = (const char*)w_up < (const char*)w_gate;
  const CUtensorMap* mw = g->get_pair(up_first ? w_up : w_gate, up_first ? w_gate : w_up, f, in, ks);
  const CUtensorMap* mx = g->get(g->xptr[xb], g->xrows[xb], in, nt, ks);
  if (!mw || !mx) return false;
  TmapPack pack;
  memset(&pack, 0, sizeof pack);
  pack.w[0] = *mw;
  pack.x = *mx;
  const uint32_t stage_bytes = ks * kTileM * kTileK * 2 + ((ks * (uint32_t)nt * kTileK * 2 + 1023u) & ~1023u);
  int stages = (int)((110 * 1024) / stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  TcParams prm;
  memset(&prm, 0, sizeof prm);
  prm.tiles_per_seg = tiles;
  prm.kblocks = kblocks;
  prm.splits = 1;
  prm.nt = nt;
  prm.rows = rows;
  prm.stages = stages;
  prm.ks = ks;
  prm.l2_prefetch = 1;
  prm.act = (__nv_bfloat16*)act;
  prm.f = f;
  prm.up_first = up_first ? 1 : 0;
  prm.rs = rs;
  prm.err_flag = g->err_flag;
  prm.wait_limit_ns = g->wait_limit_ns;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  return launch_pdl(tc_gemm_kernel<EPI_SWIGLU>, dim3(tiles, 1), dim3(kThreads), smem, st, pack, prm) == cudaSuccess;
}

bool tc_gemm_launch_qkv_rope(TcGemm* g, int xb, const void* wq, const void* wk, const void* wv, int n_heads, int dh, int in,
                             int rows, void* q, KvView kv, const RowMeta* meta, const float2* rope, int max_ctx,
                             const RowScale& rs, cudaStream_t st) {
  if (!g || xb < 0 || xb >= g->n_x || !wq || !wk || !wv || !q || !kv.k || !kv.v || !meta || !rope) return false;
  if ((dh != 64 && dh != 128) || in % kTileK || rows < 1 || g->xcols[xb] != in) return false;
  if (((uintptr_t)wq | (uintptr_t)wk | (uintptr_t)wv) & 15) return false;
  const int d = n_heads * dh;
  const int nt = rows <= 16 ? 16 : (rows + 15) / 16 * 16;
  if (nt > 64 || nt > g->xrows[xb]) return false;          // the exchanged tile is 64 activation rows at most
  const int ks = kStageKb, kblocks = in / kTileK, tiles_per_seg = d / 64;
  TmapPack pack;
  memset(&pack, 0, sizeof pack);
  const void* w[3] = {wq, wk, wv};
  for (int s = 0; s < 3; ++s) {
    const CUtensorMap* m = g->get_rope(w[s], d, in, dh / 2, ks);
    if (!m) return false;
    pack.w[s] = *m;
  }
  const CUtensorMap* mx = g->get(g->xptr[xb], g->xrows[xb], in, nt, ks);
  if (!mx) return false;
  pack.x = *mx;
  const uint32_t stage_bytes = ks * (kTileM / 2) * kTileK * 2 + ((ks * (uint32_t)nt * kTileK * 2 + 1023u) & ~1023u);
  int stages = (int)((110 * 1024) / stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  if ((size_t)stages * stage_bytes < (size_t)nt * kRopePitch * 4) return false;   // the ring doubles as the exchange buffer
  TcParams prm;
  memset(&prm, 0, sizeof prm);
  prm.tiles_per_seg = tiles_per_seg;
  prm.kblocks = kblocks;
  prm.splits = 1;
  prm.nt = nt;
  prm.nblk = 1;
  prm.rows = rows;
  prm.stages = stages;
  prm.ks = ks;
  prm.l2_prefetch = 1;
  prm.rs = rs;
  prm.q = (__nv_bfloat16*)q;
  prm.kc = (__nv_bfloat16*)kv.k;
  prm.vc = (__nv_bfloat16*)kv.v;
  prm.meta = meta;
  prm.rope = rope;
  prm.n_heads = n_heads;
  prm.dh = dh;
  prm.max_ctx = max_ctx;
  prm.err_flag = g->err_flag;
  prm.wait_limit_ns = g->wait_limit_ns;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  return launch_pdl(tc_gemm_kernel<EPI_ROPE>, dim3(3 * tiles_per_seg, 1), dim3(kThreads), smem, st, pack, prm) == cudaSuccess;
}

namespace {
// One thread per CTA asks the TMA unit to bring the first `stages` pipeline stages of every gate / up tile into L2 (stage by
// stage over all tiles, the order in which the projection's CTAs will ask for them), with the same evict-first policy as the
// copies themselves: prefetched at normal priority, the weights push the step's L2-resident working set out.
__global__ void tc_prefetch_pair_kernel(const __grid_constant__ CUtensorMap map, int tiles, int stages, int ks) {
  if (threadIdx.x != 0) return;
  const uint64_t pol = l2_evict_first_policy();
  for (int i = 0; i < stages; ++i)
    for (int t = blockIdx.x; t < tiles; t += gridDim.x)
      asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile.L2::cache_hint [%0, {%1, %2, %3, %4}], %5;"
                   ::"l"(&map), "r"(0), "r"(t * (kTileM / 2)), "r"(i * ks), "r"(0), "l"(pol) : "memory");
}
}  // namespace

bool tc_gemm_prefetch_swiglu(TcGemm* g, const void* w_gate, const void* w_up, int f, int in, size_t budget_bytes, cudaStream_t st) {
  if (!g || f % (kTileM / 2) || in % (kTileK * kStageKb)) return false;
  const int stages = (int)(budget_bytes / ((size_t)(f / (kTileM / 2)) * kStageKb * kTileM * kTileK * 2));
  if (stages <= 0) return false;
  const bool up_first = (const char*)w_up < (const char*)w_gate;
  const CUtensorMap* mw = g->get_pair(up_first ? w_up : w_gate, up_first ? w_gate : w_up, f, in, kStageKb);
  if (!mw) return false;
  const int max_stages = in / kTileK / kStageKb;
  tc_prefetch_pair_kernel<<<g->sm_count, 32, 0, st>>>(*mw, f / (kTileM / 2), stages < max_stages ? stages : max_stages, kStageKb);
  return true;
}

void tc_gemm_destroy(TcGemm* g) { delete g; }

void tc_gemm_rebind(TcGemm* g, int xb, void* ptr, int rows, int cols, int* err_flag) {
  if (!g || xb < 0 || xb >= g->n_x) return;
  g->xptr[xb] = ptr;
  g->xrows[xb] = rows;
  g->xcols[xb] = cols;
  g->err_flag = err_flag;
  if (g->cache.size() > 512) g->cache.clear();          // a long-lived plan set must not grow without bound
}

void tc_gemm_set_selftest(TcGemm* g, unsigned long long wait_limit_ns, unsigned extra_tx) {
  g->wait_limit_ns = wait_limit_ns;
  g->extra_tx = extra_tx;
}

}  // namespace amph
