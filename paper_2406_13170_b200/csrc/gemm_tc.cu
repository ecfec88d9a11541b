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
  int nt;                   // activation rows in the MMA (multiple of 16)
  int rows;                 // live rows (only these are stored)
  int stages;
  int l2_prefetch;          // weight tiles (beyond the ring) each CTA pulls into L2 before it waits
  int* err_flag;
  TcEpilogue epi;
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

// Asks the TMA unit to bring one weight tile into L2 (no shared-memory destination, no barrier).
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
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

// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = nt.
__device__ __forceinline__ uint32_t umma_idesc(int nt) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nt >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
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

__device__ __forceinline__ float4 sum_tile4(const TcParams& prm, int r, int col) {
  const float* p = prm.P + (size_t)r * prm.ld + col;
  float4 acc = __ldcg(reinterpret_cast<const float4*>(p));
  for (int s = 1; s < prm.splits; ++s) {                         // split order: deterministic
    const float4 v = __ldcg(reinterpret_cast<const float4*>(p + (size_t)s * prm.split_stride));
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  return acc;
}
__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 u;
  u.x = *reinterpret_cast<const unsigned*>(&lo);
  u.y = *reinterpret_cast<const unsigned*>(&hi);
  return u;
}
__device__ __forceinline__ float4 unpack4_bf16(const __nv_bfloat16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}

// Runs in the CTA that completed a tile: et = 0..127 indexes the four epilogue warps' threads,
// inv_s[r] is the deferred RMS division of row r (1 when none).
__device__ void fused_epilogue(const TcParams& prm, int tile, int et, const float* inv_s) {
  const TcEpilogue& e = prm.epi;
  typedef __nv_bfloat16 bf16;
  const int rows = prm.rows, tps = prm.tiles_per_seg;
  const int lane = et & 31, ew = et >> 5;
  if (e.mode == TC_EPI_RESIDUAL) {
    const int d = prm.ld, c = tile * kTileM + 4 * lane;
    for (int r = ew; r < rows; r += 4) {
      float4 v = sum_tile4(prm, r, c);
      float* xr = e.x + (size_t)r * d + c;
      const float4 o = *reinterpret_cast<const float4*>(xr);
      v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
      *reinterpret_cast<float4*>(xr) = v;
      if (e.gain != nullptr) {
        const float4 g = unpack4_bf16(reinterpret_cast<const bf16*>(e.gain) + c);
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.xn) + (size_t)r * d + c) =
            pack4_bf16(g.x * v.x, g.y * v.y, g.z * v.z, g.w * v.w);
        float ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        for (int o2 = 16; o2 > 0; o2 >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o2);
        if (lane == 0) e.ss_part[(size_t)r * tps + tile] = ss;
      }
    }
  } else if (e.mode == TC_EPI_SWIGLU) {
    const int f = prm.ld / 2, c = (tile % tps) * kTileM + 4 * lane;
    for (int r = ew; r < rows; r += 4) {
      const float sc = inv_s[r];
      const float4 g = sum_tile4(prm, r, c), u = sum_tile4(prm, r, f + c);
      float t0 = g.x * sc, t1 = g.y * sc, t2 = g.z * sc, t3 = g.w * sc;
      t0 = t0 / (1.0f + expf(-t0)) * (u.x * sc);
      t1 = t1 / (1.0f + expf(-t1)) * (u.y * sc);
      t2 = t2 / (1.0f + expf(-t2)) * (u.z * sc);
      t3 = t3 / (1.0f + expf(-t3)) * (u.w * sc);
      *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.act) + (size_t)r * f + c) = pack4_bf16(t0, t1, t2, t3);
    }
  } else if (e.mode == TC_EPI_QKV_ROPE) {
    const int dh = e.head_dim, half = dh >> 1, quads = half >> 2, d = e.n_heads * dh;
    const int seg = tile / tps, feat0 = (tile - seg * tps) * kTileM;
    const int item = et & 15, rsub = et >> 4;                  // 16 items (4 rotation pairs each) per row
    const int hh = item / quads, i = (item - hh * quads) * 4;
    const int c0 = feat0 + hh * dh + i, c1 = c0 + half;
    const int h = c0 / dh;
    const int n_rows = e.meta->n_rows;
    for (int r = rsub; r < rows; r += 8) {
      const float sc = inv_s[r];
      float4 a = sum_tile4(prm, r, seg * d + c0), b = sum_tile4(prm, r, seg * d + c1);
      a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; b.x *= sc; b.y *= sc; b.z *= sc; b.w *= sc;
      const int slot = e.meta->slot[r];
      const bool store = r < n_rows && slot >= 0 && slot < e.max_ctx;
      const size_t co = ((size_t)h * e.max_ctx + (store ? slot : 0)) * dh + i;
      if (seg == 2) {
        if (store) {
          *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.vc) + co) = pack4_bf16(a.x, a.y, a.z, a.w);
          *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.vc) + co + half) = pack4_bf16(b.x, b.y, b.z, b.w);
        }
        continue;
      }
      const float4 cs0 = *reinterpret_cast<const float4*>(e.rope + r * half + i);
      const float4 cs1 = *reinterpret_cast<const float4*>(e.rope + r * half + i + 2);
      const uint2 lo = pack4_bf16(a.x * cs0.x - b.x * cs0.y, a.y * cs0.z - b.y * cs0.w,
                                  a.z * cs1.x - b.z * cs1.y, a.w * cs1.z - b.w * cs1.w);
      const uint2 hi = pack4_bf16(b.x * cs0.x + a.x * cs0.y, b.y * cs0.z + a.y * cs0.w,
                                  b.z * cs1.x + a.z * cs1.y, b.w * cs1.z + a.w * cs1.w);
      if (seg == 0) {
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.q) + (size_t)r * d + c0) = lo;
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.q) + (size_t)r * d + c1) = hi;
      } else if (store) {
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.kc) + co) = lo;
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(e.kc) + co + half) = hi;
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads)
tc_gemm_kernel(const __grid_constant__ TmapPack maps, const TcParams prm) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[8];
  __shared__ __align__(8) uint64_t empty_bar[8];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ int last_flag;
  __shared__ float inv_s[AMPH_MAX_NODES];

  pdl_launch_dependents();                          // the consumer kernel may get resident and wait
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int seg = tile / prm.tiles_per_seg;
  const int row0 = (tile - seg * prm.tiles_per_seg) * kTileM;       // first weight row of this tile
  const int kb_lo = (int)((long long)split * prm.kblocks / prm.splits);
  const int kb_hi = (int)((long long)(split + 1) * prm.kblocks / prm.splits);
  const int nkb = kb_hi - kb_lo;
  const int nt = prm.nt, stages = prm.stages;
  const uint32_t a_bytes = kTileM * kTileK * 2, b_bytes = (uint32_t)nt * kTileK * 2;
  const uint32_t stage_bytes = a_bytes + ((b_bytes + 1023u) & ~1023u);
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < nt) tmem_cols <<= 1;

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
    // ---------------- TMA producer
    if (lane == 0) {
      const CUtensorMap* wmap = &maps.w[seg];
      asm volatile("prefetch.tensormap [%0];" ::"l"(wmap) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.x) : "memory");
      // Weights do not depend on the previous kernel: fill the ring with weight tiles first, then wait for
      // the producer of the activations, then fetch the activation tiles of those stages.
      const int npre = nkb < stages ? nkb : stages;
      for (int i = 0; i < npre; ++i) {
        mbar_expect_tx(&full_bar[i], a_bytes + b_bytes);
        tma_load_2d(smem + (size_t)i * stage_bytes, wmap, (kb_lo + i) * kTileK, row0, &full_bar[i]);
      }
      // While the previous kernel still runs, HBM would idle: pull the next weight tiles into L2 as well.
      const int npf = nkb < npre + prm.l2_prefetch ? nkb : npre + prm.l2_prefetch;
      for (int i = npre; i < npf; ++i) tma_prefetch_l2_2d(wmap, (kb_lo + i) * kTileK, row0);
      pdl_wait();
      for (int i = 0; i < npre; ++i)
        tma_load_2d(smem + (size_t)i * stage_bytes + a_bytes, &maps.x, (kb_lo + i) * kTileK, 0, &full_bar[i]);
      int issued = npre;
      for (int i = npre; i < nkb; ++i) {
        const int s = i % stages, round = i / stages;
        if (!mbar_wait(&empty_bar[s], (round & 1) ^ 1, &abort_flag)) break;
        uint8_t* a = smem + (size_t)s * stage_bytes;
        mbar_expect_tx(&full_bar[s], a_bytes + b_bytes);
        tma_load_2d(a, wmap, (kb_lo + i) * kTileK, row0, &full_bar[s]);
        tma_load_2d(a + a_bytes, &maps.x, (kb_lo + i) * kTileK, 0, &full_bar[s]);
        issued = i + 1;
      }
      if (abort_flag) {                              // drain: let every copy this thread issued land
        const int first = issued > stages ? issued - stages : 0;
        for (int i = first; i < issued; ++i) {
          const int s = i % stages, round = i / stages;
          const unsigned long long t0 = now_ns();
          while (!mbar_try(&full_bar[s], round & 1) && now_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(nt);
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const int s = i % stages, round = i / stages;
        ok = mbar_wait(&full_bar[s], round & 1, &abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
        const uint64_t adesc = umma_desc(a_addr), bdesc = umma_desc(a_addr + a_bytes);
#pragma unroll
        for (int k = 0; k < kTileK / kUmmaK; ++k)      // +32 bytes (2 x 16 B) per K step inside the swizzle row
          umma_f16(tmem_d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (i | k) ? 1u : 0u);
        umma_commit(&empty_bar[s]);                    // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(&accum_bar);
    }
  } else {
    // ---------------- epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
    const int quarter = warp & 3;
    pdl_wait();                                      // P may still be read by the kernel before this one
    const bool ok = __all_sync(0xffffffffu, nkb > 0 ? mbar_wait(&accum_bar, 0, &abort_flag) : false);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int feat = seg * prm.tiles_per_seg * kTileM + row0 + quarter * 32 + lane;
    float* out = prm.P + (size_t)split * prm.split_stride + feat;
    for (int c0 = 0; c0 < nt; c0 += 16) {
      if (c0 >= prm.rows) break;
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
        for (int j = 0; j < 16; ++j) v[j] = 0u;          // empty K-range or aborted: contribute zeros
      }
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (c0 + j < prm.rows) out[(size_t)(c0 + j) * prm.ld] = __uint_as_float(v[j]);
    }
    if (prm.epi.mode != TC_EPI_NONE) {
      // Last arriver at this tile (both tiles of a gate / up pair for SWIGLU) reduces and finishes it.
      const int et = threadIdx.x - 64;
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        const bool pair = prm.epi.mode == TC_EPI_SWIGLU;
        const int idx = pair ? tile % prm.tiles_per_seg : tile;
        const int target = (pair ? 2 : 1) * prm.splits;
        const int old = atomicAdd(&prm.epi.counters[idx], 1);
        const int last = (old == target - 1) && !abort_flag;
        if (old == target - 1) prm.epi.counters[idx] = 0;        // ready for the next launch
        last_flag = last;
      }
      for (int r = et; r < prm.rows; r += 128) {
        float sc = 1.0f;
        if (prm.epi.rs.ss != nullptr) {
          float tot = 0.f;
          for (int c = 0; c < prm.epi.rs.chunks; ++c) tot += prm.epi.rs.ss[r * prm.epi.rs.chunks + c];
          sc = 1.0f / sqrtf(tot / (float)prm.epi.rs.d + prm.epi.rs.eps);
        }
        inv_s[r] = sc;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (last_flag) {
        __threadfence();
        fused_epilogue(prm, tile, et, inv_s);
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
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> cache;   // (ptr, rows, cols, box rows)
  int sm_count = 148;
  int max_smem = 0;

  const CUtensorMap* get(const void* ptr, int rows, int cols, int box_rows) {
    auto key = std::make_tuple(ptr, rows, cols, box_rows);
    auto it = cache.find(key);
    if (it != cache.end()) return &it->second;
    CUtensorMap m;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
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
  cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, g->max_smem - 2048);
  return g;
}

bool tc_gemm_launch(TcGemm* g, int xb, const void* const* w, int n_seg, int out, int in, int rows, float* P,
                    size_t p_floats, int* splits_out, size_t* split_stride, cudaStream_t st, const TcEpilogue* epi) {
  if (!g || xb < 0 || xb >= g->n_x) return false;
  if (epi && epi->mode != TC_EPI_NONE) {
    if (!epi->counters || n_seg * (out / kTileM) > kTcCounterInts) return false;
    if (epi->mode == TC_EPI_RESIDUAL && n_seg != 1) return false;
    if (epi->mode == TC_EPI_SWIGLU && n_seg != 2) return false;
    if (epi->mode == TC_EPI_QKV_ROPE &&
        (n_seg != 3 || epi->head_dim < 8 || kTileM % epi->head_dim || out != epi->n_heads * epi->head_dim)) return false;
  }
  if (out % kTileM || in % kTileK || n_seg < 1 || n_seg > kMaxSeg || rows < 1) return false;
  if (g->xcols[xb] != in) return false;
  const int nt = rows <= 16 ? 16 : (rows + 15) / 16 * 16;
  if (nt > 128 || nt > g->xrows[xb]) return false;
  const int tiles = n_seg * (out / kTileM), kblocks = in / kTileK;
  const size_t ld = (size_t)n_seg * out;
  // K-splits: fill about two CTAs per SM, keep at least four 64-wide K blocks per CTA
  int splits = (2 * g->sm_count) / tiles;
  if (splits > kblocks / 4) splits = kblocks / 4;
  if (splits > 16) splits = 16;
  while (splits > 1 && (size_t)splits * nt * ld > p_floats) --splits;
  if (splits < 1) splits = 1;
  if ((size_t)nt * ld > p_floats) return false;
  TmapPack pack;
  memset(&pack, 0, sizeof pack);
  for (int s = 0; s < n_seg; ++s) {
    if ((uintptr_t)w[s] & 15) return false;
    const CUtensorMap* m = g->get(w[s], out, in, kTileM);
    if (!m) return false;
    pack.w[s] = *m;
  }
  const CUtensorMap* mx = g->get(g->xptr[xb], g->xrows[xb], in, nt);
  if (!mx) return false;
  pack.x = *mx;
  const uint32_t stage_bytes = kTileM * kTileK * 2 + (((uint32_t)nt * kTileK * 2 + 1023u) & ~1023u);
  int stages = (int)((100 * 1024) / stage_bytes);          // <= ~100 KB per CTA: two CTAs per SM
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  TcParams prm;
  prm.P = P;
  prm.split_stride = (size_t)nt * ld;
  prm.ld = (int)ld;
  prm.tiles_per_seg = out / kTileM;
  prm.kblocks = kblocks;
  prm.splits = splits;
  prm.nt = nt;
  prm.rows = rows;
  prm.stages = stages;
  // about 40 MB of L2 for prefetched weight tiles, shared by the CTAs that can be resident at once
  {
    const long long resident = (long long)tiles * splits < 2LL * g->sm_count ? (long long)tiles * splits : 2LL * g->sm_count;
    long long pf = (40LL << 20) / (resident * (kTileM * kTileK * 2));
    prm.l2_prefetch = (int)(pf > 32 ? 32 : pf);
  }
  prm.err_flag = g->err_flag;
  prm.epi = epi ? *epi : TcEpilogue();
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  launch_pdl(tc_gemm_kernel, dim3(tiles, splits), dim3(kThreads), smem, st, pack, prm);
  *splits_out = splits;
  *split_stride = prm.split_stride;
  return true;
}

void tc_gemm_destroy(TcGemm* g) { delete g; }

}  // namespace amph
