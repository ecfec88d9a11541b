// Tree attention for bf16 caches on the warp-level tensor-core path (mma.sync m16n8k16, fp32
// accumulate): split-KV flash-decoding where the tree is a per-row 128-bit ancestor mask.
//
// Grid (head, split, block of 64 query rows); 4 warps, each owns 16 query rows and the whole head
// dimension.  Keys / values stream through a double-buffered shared-memory ring filled by cp.async
// (16-byte chunks, XOR-swizzled so that ldmatrix is bank-conflict free).  Scores, the online softmax and
// the output accumulator stay in registers; each CTA leaves an unnormalised partial output plus the
// running (max, sum) per row, merged by attn_combine_kernel.
//
// Merge in the same launch (MERGE = true): the KV splits of one head form a thread-block cluster (up to 8).
// Each CTA parks its partial output in its own shared memory; after a cluster barrier CTA j merges rows
// j, j + S, ... of all S partials through distributed shared memory and writes the final bf16 rows, so the
// partials never travel through L2 and the merge kernel with its launch boundary disappears.
#include <math.h>

#include "amph_internal.cuh"

namespace amph {

typedef __nv_bfloat16 bf16;

namespace {

constexpr int kRows = 64;          // query rows per CTA
constexpr int kKeys = 64;          // keys per tile
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;                      // 0 source bytes => the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Row-major [rows][DH] bf16 tile in shared memory; 16-byte chunk c of row r lives at chunk c ^ (r & 7).
template <int DH>
__device__ __forceinline__ uint32_t tile_addr(uint32_t base, int row, int chunk) {
  return base + (uint32_t)(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int DH>
__device__ __forceinline__ void load_tile(bf16* dst, const bf16* src, int s0, int s_hi, int tid) {
  constexpr int CH = DH / 8;                         // 16-byte chunks per row
  for (int i = tid; i < kKeys * CH; i += kThreads) {
    const int r = i / CH, c = i - r * CH;
    const int s = s0 + r;
    const bool valid = s < s_hi;
    const bf16* g = src + (size_t)(valid ? s : 0) * DH + c * 8;
    cp_async16(reinterpret_cast<char*>(dst) + r * (DH * 2) + ((c ^ (r & 7)) << 4), g, valid);
  }
}

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in the CTA of rank `rank` of this cluster
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

template <int DH, bool MERGE>
__global__ void __launch_bounds__(kThreads)
tree_attn_mma_kernel(const bf16* __restrict__ q, const bf16* __restrict__ kc, const bf16* __restrict__ vc,
                     const RowMeta* __restrict__ meta, float* __restrict__ po, float* __restrict__ pml,
                     int rows_cap, int n_heads, int max_ctx, bf16* __restrict__ out) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int KS = DH / 16;                        // k-steps over the head dimension
  constexpr int NT = DH / 8;                         // 8-wide output tiles
  extern __shared__ __align__(128) unsigned char sm_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(sm_raw);                       // [64][DH]
  bf16* Ks = Qs + kRows * DH;                                        // [2][64][DH]
  bf16* Vs = Ks + 2 * kKeys * DH;                                    // [2][64][DH]
  const int h = blockIdx.x, split = blockIdx.y, rb = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int base = meta->base, n_rows = meta->n_rows;
  const int d = n_heads * DH;
  const int total = base + n_rows;
  int chunk = (total + gridDim.y - 1) / gridDim.y;
  chunk = (chunk + kKeys - 1) / kKeys * kKeys;
  const int s_lo = split * chunk;
  int s_hi = s_lo + chunk;
  if (s_hi > total) s_hi = total;
  if (s_hi > max_ctx) s_hi = max_ctx;
  const int n_tiles = s_hi > s_lo ? (s_hi - s_lo + kKeys - 1) / kKeys : 0;
  const bf16* kh = kc + (size_t)h * max_ctx * DH;
  const bf16* vh = vc + (size_t)h * max_ctx * DH;

  // the two rows this thread holds scores for, and their masks
  const int row_a = rb * kRows + warp * 16 + g, row_b = row_a + 8;
  const bool live_a = row_a < n_rows, live_b = row_b < n_rows;
  u64 ma0 = 0, ma1 = 0, mb0 = 0, mb1 = 0;
  if (live_a) { ma0 = meta->mask[row_a][0]; ma1 = meta->mask[row_a][1]; }
  if (live_b) { mb0 = meta->mask[row_b][0]; mb1 = meta->mask[row_b][1]; }

  // stage Q (rows beyond the buffer are zero) and the first K / V tile
  {
    constexpr int CH = DH / 8;
    for (int i = tid; i < kRows * CH; i += kThreads) {
      const int r = i / CH, c = i - r * CH;
      const int gr = rb * kRows + r;
      const bool valid = gr < rows_cap;
      cp_async16(reinterpret_cast<char*>(Qs) + r * (DH * 2) + ((c ^ (r & 7)) << 4),
                 q + (size_t)(valid ? gr : 0) * d + h * DH + c * 8, valid);
    }
    if (n_tiles > 0) { load_tile<DH>(Ks, kh, s_lo, s_hi, tid); load_tile<DH>(Vs, vh, s_lo, s_hi, tid); }
    cp_async_commit();
  }

  float oacc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  const float scale = 1.0f / sqrtf((float)DH);
  uint32_t qf[KS][4];

  for (int it = 0; it < n_tiles; ++it) {
    const int buf = it & 1;
    if (it + 1 < n_tiles) {                          // prefetch the next tile into the other buffer
      load_tile<DH>(Ks + (buf ^ 1) * kKeys * DH, kh, s_lo + (it + 1) * kKeys, s_hi, tid);
      load_tile<DH>(Vs + (buf ^ 1) * kKeys * DH, vh, s_lo + (it + 1) * kKeys, s_hi, tid);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (it == 0) {
      const uint32_t qb = smem_u32(Qs);
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
        ldsm_x4(tile_addr<DH>(qb, warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, ks * 2 + (lane >> 4)),
                qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    const uint32_t kb = smem_u32(Ks + buf * kKeys * DH), vb = smem_u32(Vs + buf * kKeys * DH);
    const int t0 = s_lo + it * kKeys;

    // ---- S = Q K^T for 64 keys
    float sacc[kKeys / 8][4];
#pragma unroll
    for (int j = 0; j < kKeys / 8; ++j) {
      sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f;
#pragma unroll
      for (int b = 0; b < DH / 32; ++b) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4(tile_addr<DH>(kb, j * 8 + (lane & 7), b * 4 + (lane >> 3)), r0, r1, r2, r3);
        mma_bf16(sacc[j], qf[2 * b], r0, r1);
        mma_bf16(sacc[j], qf[2 * b + 1], r2, r3);
      }
    }
    // ---- mask, online softmax (rows g and g+8 of this warp's 16)
    float tmax_a = -INFINITY, tmax_b = -INFINITY;
#pragma unroll
    for (int j = 0; j < kKeys / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int s = t0 + j * 8 + 2 * t + e;
        bool va = live_a && s < s_hi, vb2 = live_b && s < s_hi;
        if (s >= base) {
          const int m = s - base;
          const u64 bit = 1ull << (m & 63);
          va = va && ((m < 64 ? ma0 : ma1) & bit);
          vb2 = vb2 && ((m < 64 ? mb0 : mb1) & bit);
        }
        sacc[j][e] = va ? sacc[j][e] * scale : -INFINITY;
        sacc[j][2 + e] = vb2 ? sacc[j][2 + e] * scale : -INFINITY;
        tmax_a = fmaxf(tmax_a, sacc[j][e]);
        tmax_b = fmaxf(tmax_b, sacc[j][2 + e]);
      }
    }
    tmax_a = fmaxf(tmax_a, __shfl_xor_sync(0xffffffffu, tmax_a, 1));
    tmax_a = fmaxf(tmax_a, __shfl_xor_sync(0xffffffffu, tmax_a, 2));
    tmax_b = fmaxf(tmax_b, __shfl_xor_sync(0xffffffffu, tmax_b, 1));
    tmax_b = fmaxf(tmax_b, __shfl_xor_sync(0xffffffffu, tmax_b, 2));
    const float mn_a = fmaxf(m_a, tmax_a), mn_b = fmaxf(m_b, tmax_b);
    const float ca = mn_a == -INFINITY ? 1.f : expf(m_a - mn_a);       // exp(-inf) = 0 on the first visible tile
    const float cb = mn_b == -INFINITY ? 1.f : expf(m_b - mn_b);
    float ps_a = 0.f, ps_b = 0.f;
#pragma unroll
    for (int j = 0; j < kKeys / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float pa = sacc[j][e] == -INFINITY ? 0.f : expf(sacc[j][e] - mn_a);
        const float pb = sacc[j][2 + e] == -INFINITY ? 0.f : expf(sacc[j][2 + e] - mn_b);
        sacc[j][e] = pa;
        sacc[j][2 + e] = pb;
        ps_a += pa;
        ps_b += pb;
      }
    }
    ps_a += __shfl_xor_sync(0xffffffffu, ps_a, 1);
    ps_a += __shfl_xor_sync(0xffffffffu, ps_a, 2);
    ps_b += __shfl_xor_sync(0xffffffffu, ps_b, 1);
    ps_b += __shfl_xor_sync(0xffffffffu, ps_b, 2);
    l_a = l_a * ca + ps_a;
    l_b = l_b * cb + ps_b;
    m_a = mn_a;
    m_b = mn_b;
#pragma unroll
    for (int i = 0; i < NT; ++i) { oacc[i][0] *= ca; oacc[i][1] *= ca; oacc[i][2] *= cb; oacc[i][3] *= cb; }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < kKeys / 16; ++kk) {
      uint32_t pf[4];
      pf[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
      pf[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
      pf[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
      pf[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
      for (int c = 0; c < NT; c += 2) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4_t(tile_addr<DH>(vb, kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c + (lane >> 4)), r0, r1, r2, r3);
        mma_bf16(oacc[c], pf, r0, r1);
        mma_bf16(oacc[c + 1], pf, r2, r3);
      }
    }
    __syncthreads();                                 // everyone is done with this buffer before it is refilled
  }
  if (n_tiles == 0) cp_async_wait<0>();

  if constexpr (MERGE) {
    // ---- park the partial output and (max, sum) in shared memory (the K / V ring is free now)
    float* Os = reinterpret_cast<float*>(Ks);                        // [64][DH]
    float* MLs = Os + kRows * DH;                                    // [64][2]
    const int la = warp * 16 + g, lb = la + 8;
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      *reinterpret_cast<float2*>(Os + la * DH + i * 8 + 2 * t) = make_float2(oacc[i][0], oacc[i][1]);
      *reinterpret_cast<float2*>(Os + lb * DH + i * 8 + 2 * t) = make_float2(oacc[i][2], oacc[i][3]);
    }
    if (t == 0) {
      *reinterpret_cast<float2*>(MLs + la * 2) = make_float2(m_a, l_a);
      *reinterpret_cast<float2*>(MLs + lb * 2) = make_float2(m_b, l_b);
    }
    cluster_sync_all();
    // ---- CTA `split` of the S in the cluster merges rows split, split + S, ...; one warp per row, a lane per 4 columns
    const int S = gridDim.y;
    const uint32_t os0 = smem_u32(Os), ml0 = smem_u32(MLs);
    for (int r = split + S * warp; r < kRows; r += S * (kThreads / 32)) {
      const int gr = rb * kRows + r;
      if (gr >= rows_cap) continue;
      float2 ml = make_float2(-INFINITY, 0.f);
      if (lane < S) ml = ld_peer2(peer_smem(ml0 + (uint32_t)r * 8, (uint32_t)lane));
      float M = ml.x;
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      const float wgt = ml.x == -INFINITY ? 0.f : expf(ml.x - M);     // lane s holds the weight of split s
      float den = ml.y * wgt;
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < S; ++s) {
        const float ws = __shfl_sync(0xffffffffu, wgt, s);
        if (lane * 4 < DH && ws != 0.f) {
          const float4 v = ld_peer4(peer_smem(os0 + (uint32_t)(r * DH + lane * 4) * 4, (uint32_t)s));
          acc.x += v.x * ws; acc.y += v.y * ws; acc.z += v.z * ws; acc.w += v.w * ws;
        }
      }
      if (lane * 4 < DH) {
        const float inv = den > 0.f ? 1.0f / den : 0.f;
        uint2 u;
        u.x = pack_bf16(acc.x * inv, acc.y * inv);
        u.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(out + (size_t)gr * n_heads * DH + h * DH + lane * 4) = u;
      }
    }
    cluster_sync_all();                              // nobody leaves while a peer may still read its shared memory
    return;
  }
  // ---- partial results
  const size_t oa = ((size_t)split * n_heads + h) * rows_cap + row_a;
  const size_t ob = oa + 8;
  if (row_a < rows_cap) {
#pragma unroll
    for (int i = 0; i < NT; ++i)
      *reinterpret_cast<float2*>(po + oa * DH + i * 8 + 2 * t) = make_float2(oacc[i][0], oacc[i][1]);
    if (t == 0) { pml[oa * 2] = m_a; pml[oa * 2 + 1] = l_a; }
  }
  if (row_b < rows_cap) {
#pragma unroll
    for (int i = 0; i < NT; ++i)
      *reinterpret_cast<float2*>(po + ob * DH + i * 8 + 2 * t) = make_float2(oacc[i][2], oacc[i][3]);
    if (t == 0) { pml[ob * 2] = m_b; pml[ob * 2 + 1] = l_b; }
  }
}

template <int DH>
bool launch_t(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, int rows, int n_heads, int max_ctx,
              int splits, cudaStream_t st, void* merged_out) {
  const size_t smem = sizeof(bf16) * (kRows * DH + 4 * kKeys * DH);
  dim3 grid(n_heads, splits, (rows + kRows - 1) / kRows);
  if (merged_out != nullptr && splits <= 8) {
    // the KV splits of a head as one cluster; merge through distributed shared memory
    static_assert(sizeof(float) * (kRows * DH + kRows * 2) <= sizeof(bf16) * 4 * kKeys * DH, "partial output must fit the K / V ring");
    cudaFuncSetAttribute(tree_attn_mma_kernel<DH, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 1;
    at[1].val.clusterDim.y = splits;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, tree_attn_mma_kernel<DH, true>, (const bf16*)q, (const bf16*)kv.k, (const bf16*)kv.v,
                                             meta, sc.o, sc.ml, rows, n_heads, max_ctx, (bf16*)merged_out);
    if (e == cudaSuccess) return true;
    cudaGetLastError();                              // cluster launch refused: fall back to two launches
  }
  cudaFuncSetAttribute(tree_attn_mma_kernel<DH, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  launch_pdl(tree_attn_mma_kernel<DH, false>, dim3(grid), dim3(kThreads), smem, st, (const bf16*)q, (const bf16*)kv.k, (const bf16*)kv.v, meta, sc.o,
                                                        sc.ml, rows, n_heads, max_ctx, (bf16*)nullptr);
  return false;
}

}  // namespace

bool launch_tree_attention_mma(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, int rows, int n_heads,
                               int head_dim, int max_ctx, int splits, cudaStream_t st, void* merged_out) {
  if (head_dim == 64) return launch_t<64>(q, kv, meta, sc, rows, n_heads, max_ctx, splits, st, merged_out);
  return launch_t<128>(q, kv, meta, sc, rows, n_heads, max_ctx, splits, st, merged_out);
}

}  // namespace amph
