// Memory-bound and control kernels of the Amphista step: embedding, fused residual + RMSNorm,
// rotary embedding + KV write, split-KV tree attention with a bitmask, SwiGLU, the draft
// module's head kernels (Eq. 2-6), tree construction, greedy acceptance and KV compaction.
#include <math.h>

#include "amph_internal.cuh"

namespace amph {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

#define AMPH_DISPATCH(dtype, ...)                                    \
  do {                                                               \
    if ((dtype) == AMPH_DTYPE_F32) { typedef float T; __VA_ARGS__; } \
    else { typedef bf16 T; __VA_ARGS__; }                            \
  } while (0)

__device__ __forceinline__ float sum_partials(const PartialView& P, int row, int col) {
  const float* p = P.p + (size_t)row * P.ld + col;
  float acc = p[0];
  for (int s = 1; s < P.splits; ++s) acc += p[(size_t)s * P.split_stride];   // fixed order: deterministic
  return acc;
}

// The partial sums sit in L2, one round trip each: the loads of a batch of N splits are issued together,
// then added in split order.
template <int N>
__device__ __forceinline__ void add_splits(const float* p, size_t stride, int s0, int splits, float4& acc) {
  float4 v[N];
#pragma unroll
  for (int s = 0; s < N; ++s)
    if (s0 + s < splits) v[s] = *reinterpret_cast<const float4*>(p + (size_t)(s0 + s) * stride);
#pragma unroll
  for (int s = 0; s < N; ++s)
    if (s0 + s < splits) { acc.x += v[s].x; acc.y += v[s].y; acc.z += v[s].z; acc.w += v[s].w; }
}

// Same sum for kernels with registers to spare and many splits to read (the residual kernels).
__device__ __forceinline__ float4 sum_partials4_wide(const PartialView& P, int row, int col) {
  const float* p = P.p + (size_t)row * P.ld + col;
  float4 acc = *reinterpret_cast<const float4*>(p);
  const int n = P.splits;
  if (n == 1) return acc;
  for (int s0 = 1; s0 < n; s0 += 8) add_splits<8>(p, P.split_stride, s0, n, acc);
  return acc;
}

__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<unsigned*>(&a);
  u.y = *reinterpret_cast<unsigned*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const bf16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[w] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += red[i];
  return t;
}

// --------------------------------------------------------------------------------------------
// embedding rows
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const T* __restrict__ emb, const int* __restrict__ toks, int vocab, int d,
                             float* __restrict__ x) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = blockIdx.x;
  int t = toks[r];
  t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
  const T* e = emb + (size_t)t * d;
  for (int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4; c < d; c += gridDim.y * blockDim.x * 4)
    store4(x + (size_t)r * d + c, load4(e + c));
}

void launch_embed(const void* tok_emb, int dtype, const int* toks, int vocab, int rows, int d, float* x,
                  cudaStream_t st) {
  const int gy = (d / 4 + 255) / 256;
  AMPH_DISPATCH(dtype, launch_pdl(embed_kernel<T>, dim3(rows, gy), dim3(256), 0, st, (const T*)tok_emb, toks, vocab, d, x));
}

// --------------------------------------------------------------------------------------------
// residual update + RMSNorm (one block per row)
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(1024)
resid_norm_kernel(float* __restrict__ x, PartialView P, int col_off, int mode, const T* __restrict__ gain,
                  T* __restrict__ xn, float* __restrict__ hid, float eps, int d) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) float rowbuf[];
  __shared__ float red[32];
  const int r = blockIdx.x;
  float* xr = x + (size_t)r * d;
  float ss = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    float4 v;
    if (mode == 0) {
      v = load4(xr + c);
    } else {
      v = sum_partials4(P, r, col_off + c);
      if (mode == 1) { const float4 o = load4(xr + c); v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
      store4(xr + c, v);
    }
    store4(rowbuf + c, v);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  if (xn == nullptr && hid == nullptr) return;
  if (gain == nullptr) {                       // plain cast of the updated row (each thread re-reads its own chunk)
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
      const float4 v = load4(rowbuf + c);
      if (xn) store4(xn + (size_t)r * d + c, v);
      if (hid) store4(hid + (size_t)r * d + c, v);
    }
    return;
  }
  const float tot = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(tot / (float)d + eps);
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    const float4 v = load4(rowbuf + c), g = load4(gain + c);
    const float4 n = make_float4(g.x * (v.x * inv), g.y * (v.y * inv), g.z * (v.z * inv), g.w * (v.w * inv));
    if (xn) store4(xn + (size_t)r * d + c, n);
    if (hid) store4(hid + (size_t)r * d + c, n);
  }
}

void launch_resid_norm(float* x, PartialView P, int col_off, int mode, const void* gain, int dtype,
                       void* xn, float* hid, float eps, int rows, int d, cudaStream_t st) {
  int threads = (d / 4 + 31) / 32 * 32;
  if (threads > 1024) threads = 1024;
  AMPH_DISPATCH(dtype, launch_pdl(resid_norm_kernel<T>, dim3(rows), dim3(threads), d * sizeof(float), st, 
                           x, P, col_off, mode, (const T*)gain, (T*)xn, hid, eps, d));
}

// Residual update without the row-wide reduction: grid (row, 512-column chunk).  The division by the row's
// RMS is left to the kernel that consumes the next projection (RowScale), so every block is independent.
template <typename T>
__global__ void __launch_bounds__(128)
resid_scale_kernel(float* __restrict__ x, PartialView P, int col_off, int mode, const T* __restrict__ gain,
                   T* __restrict__ xn, float* __restrict__ ss_part, int d, int early) {
  if (early) pdl_launch_dependents();
  pdl_wait();
  if (!early) pdl_launch_dependents();
  __shared__ float red[32];
  const int r = blockIdx.x;
  const int c = blockIdx.y * kScaleChunkCols + threadIdx.x * 4;
  float ss = 0.f;
  if (c < d) {
    float* xr = x + (size_t)r * d + c;
    float4 v = sum_partials4_wide(P, r, col_off + c);
    if (mode == 1) { const float4 o = load4(xr); v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
    store4(xr, v);
    if (gain != nullptr) {
      const float4 g = load4(gain + c);
      store4(xn + (size_t)r * d + c, make_float4(g.x * v.x, g.y * v.y, g.z * v.z, g.w * v.w));
      ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  }
  if (gain == nullptr) return;
  const float tot = block_sum(ss, red);
  if (threadIdx.x == 0) ss_part[r * gridDim.y + blockIdx.y] = tot;
}

void launch_resid_scale(float* x, PartialView P, int col_off, int mode, const void* gain, int dtype, void* xn,
                        float* ss_part, int rows, int d, cudaStream_t st, int early) {
  const int chunks = (d + kScaleChunkCols - 1) / kScaleChunkCols;
  AMPH_DISPATCH(dtype, launch_pdl(resid_scale_kernel<T>, dim3(rows, chunks), dim3(128), 0, st, x, P, col_off, mode,
                                  (const T*)gain, (T*)xn, ss_part, d, early));
}

// --------------------------------------------------------------------------------------------
// rotary table for the rows of one call: table[r][i] = (cos, sin)(pos[r] * theta^(-2i/dh))
// --------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(const RowMeta* __restrict__ meta, const double* __restrict__ inv_freq,
                                  float2* __restrict__ table, int half) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = blockIdx.x;
  const double p = (double)meta->pos[r];
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    double s, c;
    sincos(p * inv_freq[i], &s, &c);
    table[r * half + i] = make_float2((float)c, (float)s);
  }
}

void launch_rope_table(const RowMeta* meta, const double* inv_freq, float2* table, int rows, int half,
                       cudaStream_t st) {
  launch_pdl(rope_table_kernel, dim3(rows), dim3(64), 0, st, meta, inv_freq, table, half);
}

// --------------------------------------------------------------------------------------------
// q / k rotation, KV-cache write (one block per row)
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
qkv_rope_kernel(PartialView P, const RowMeta* __restrict__ meta, const float2* __restrict__ rope, T* __restrict__ q,
                T* __restrict__ kc, T* __restrict__ vc, int n_heads, int dh, int max_ctx, RowScale rs) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = blockIdx.x;
  const int half = dh >> 1, d = n_heads * dh, quads = half >> 2;
  const bool live = r < meta->n_rows;
  const int slot = meta->slot[r];
  const bool store = live && slot >= 0 && slot < max_ctx;
  const float sc = row_scale(rs, r);
  // one item = four rotation pairs (i..i+3, i+half..) of one head; grid.y strides over the items of the row
  for (int idx = blockIdx.y * blockDim.x + threadIdx.x; idx < n_heads * quads; idx += gridDim.y * blockDim.x) {
    const int h = idx / quads, i = (idx - h * quads) * 4;
    const float4 cs0 = *reinterpret_cast<const float4*>(rope + r * half + i);       // (c0,s0,c1,s1)
    const float4 cs1 = *reinterpret_cast<const float4*>(rope + r * half + i + 2);   // (c2,s2,c3,s3)
    const int c0 = h * dh + i, c1 = c0 + half;
    {
      float4 a = sum_partials4(P, r, c0), b = sum_partials4(P, r, c1);
      a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; b.x *= sc; b.y *= sc; b.z *= sc; b.w *= sc;
      store4(q + (size_t)r * d + c0, make_float4(a.x * cs0.x - b.x * cs0.y, a.y * cs0.z - b.y * cs0.w,
                                                 a.z * cs1.x - b.z * cs1.y, a.w * cs1.z - b.w * cs1.w));
      store4(q + (size_t)r * d + c1, make_float4(b.x * cs0.x + a.x * cs0.y, b.y * cs0.z + a.y * cs0.w,
                                                 b.z * cs1.x + a.z * cs1.y, b.w * cs1.z + a.w * cs1.w));
    }
    if (store) {
      float4 a = sum_partials4(P, r, d + c0), b = sum_partials4(P, r, d + c1);
      a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; b.x *= sc; b.y *= sc; b.z *= sc; b.w *= sc;
      const size_t o = ((size_t)h * max_ctx + slot) * dh + i;
      store4(kc + o, make_float4(a.x * cs0.x - b.x * cs0.y, a.y * cs0.z - b.y * cs0.w,
                                 a.z * cs1.x - b.z * cs1.y, a.w * cs1.z - b.w * cs1.w));
      store4(kc + o + half, make_float4(b.x * cs0.x + a.x * cs0.y, b.y * cs0.z + a.y * cs0.w,
                                        b.z * cs1.x + a.z * cs1.y, b.w * cs1.z + a.w * cs1.w));
      float4 v0 = sum_partials4(P, r, 2 * d + c0), v1 = sum_partials4(P, r, 2 * d + c1);
      store4(vc + o, make_float4(v0.x * sc, v0.y * sc, v0.z * sc, v0.w * sc));
      store4(vc + o + half, make_float4(v1.x * sc, v1.y * sc, v1.z * sc, v1.w * sc));
    }
  }
}

// The same for G row groups in one launch (blockIdx.z = group): group g's rows start at row g * rpg of P, q and rs and
// use their own row table, rotary table and cache.
template <typename T>
__global__ void __launch_bounds__(256)
qkv_rope_groups_kernel(PartialView P, RopeGroups gr, T* __restrict__ q, int n_heads, int dh, int max_ctx, RowScale rs) {
  pdl_wait();
  pdl_launch_dependents();
  const int g = blockIdx.z, rl = blockIdx.x, r = g * gr.rpg + rl;
  const RowMeta* meta = gr.meta[g];
  const float2* rope = gr.rope[g];
  T* kc = (T*)gr.kc[g];
  T* vc = (T*)gr.vc[g];
  const int half = dh >> 1, d = n_heads * dh, quads = half >> 2;
  const bool live = rl < meta->n_rows;
  const int slot = meta->slot[rl];
  const bool store = live && slot >= 0 && slot < max_ctx;
  const float sc = row_scale(rs, r);
  for (int idx = blockIdx.y * blockDim.x + threadIdx.x; idx < n_heads * quads; idx += gridDim.y * blockDim.x) {
    const int h = idx / quads, i = (idx - h * quads) * 4;
    const float4 cs0 = *reinterpret_cast<const float4*>(rope + rl * half + i);
    const float4 cs1 = *reinterpret_cast<const float4*>(rope + rl * half + i + 2);
    const int c0 = h * dh + i, c1 = c0 + half;
    {
      float4 a = sum_partials4(P, r, c0), b = sum_partials4(P, r, c1);
      a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; b.x *= sc; b.y *= sc; b.z *= sc; b.w *= sc;
      store4(q + (size_t)r * d + c0, make_float4(a.x * cs0.x - b.x * cs0.y, a.y * cs0.z - b.y * cs0.w,
                                                 a.z * cs1.x - b.z * cs1.y, a.w * cs1.z - b.w * cs1.w));
      store4(q + (size_t)r * d + c1, make_float4(b.x * cs0.x + a.x * cs0.y, b.y * cs0.z + a.y * cs0.w,
                                                 b.z * cs1.x + a.z * cs1.y, b.w * cs1.z + a.w * cs1.w));
    }
    if (store) {
      float4 a = sum_partials4(P, r, d + c0), b = sum_partials4(P, r, d + c1);
      a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; b.x *= sc; b.y *= sc; b.z *= sc; b.w *= sc;
      const size_t o = ((size_t)h * max_ctx + slot) * dh + i;
      store4(kc + o, make_float4(a.x * cs0.x - b.x * cs0.y, a.y * cs0.z - b.y * cs0.w,
                                 a.z * cs1.x - b.z * cs1.y, a.w * cs1.z - b.w * cs1.w));
      store4(kc + o + half, make_float4(b.x * cs0.x + a.x * cs0.y, b.y * cs0.z + a.y * cs0.w,
                                        b.z * cs1.x + a.z * cs1.y, b.w * cs1.z + a.w * cs1.w));
      float4 v0 = sum_partials4(P, r, 2 * d + c0), v1 = sum_partials4(P, r, 2 * d + c1);
      store4(vc + o, make_float4(v0.x * sc, v0.y * sc, v0.z * sc, v0.w * sc));
      store4(vc + o + half, make_float4(v1.x * sc, v1.y * sc, v1.z * sc, v1.w * sc));
    }
  }
}

void launch_qkv_rope_groups(PartialView P, const RopeGroups& gr, void* q, int dtype, int n_heads, int head_dim, int max_ctx,
                            cudaStream_t st, RowScale rs) {
  const int items = n_heads * head_dim / 8;
  const int threads = items >= 128 ? 128 : (items + 31) / 32 * 32;
  const int gy = (items + threads - 1) / threads;
  AMPH_DISPATCH(dtype, launch_pdl(qkv_rope_groups_kernel<T>, dim3(gr.rpg, gy, gr.G), dim3(threads), 0, st, P, gr, (T*)q, n_heads,
                                  head_dim, max_ctx, rs));
}

void launch_qkv_rope(PartialView P, const RowMeta* meta, const float2* rope, void* q, KvView kv, int dtype,
                     int rows, int n_heads, int head_dim, int max_ctx, cudaStream_t st, RowScale rs) {
  const int items = n_heads * head_dim / 8;
  const int threads = items >= 128 ? 128 : (items + 31) / 32 * 32;
  const int gy = (items + threads - 1) / threads;
  AMPH_DISPATCH(dtype, launch_pdl(qkv_rope_kernel<T>, dim3(rows, gy), dim3(threads), 0, st, P, meta, rope, (T*)q,
                                  (T*)kv.k, (T*)kv.v, n_heads, head_dim, max_ctx, rs));
}

// --------------------------------------------------------------------------------------------
// Tree attention, split over the KV axis (flash-decoding form), with the tree as a bitmask.
// Grid (head, split, row block of 64).  Slots below meta->base are visible to every row;
// slot base + m is visible to row r iff bit m of mask[r] is set.
// --------------------------------------------------------------------------------------------
constexpr int kAttRows = 64;     // query rows per block
constexpr int kAttTile = 32;     // keys per inner tile
constexpr int kAttThreads = 256;

template <typename T, int DH>
__global__ void __launch_bounds__(kAttThreads)
tree_attn_kernel(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                 const RowMeta* __restrict__ meta, float* __restrict__ po, float* __restrict__ pml,
                 int rows_cap, int n_heads, int max_ctx) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int QS = DH + 4;                       // padded row strides (bank-conflict free float4 reads)
  constexpr int SEG = DH / 4;                      // output dims owned by one thread
  extern __shared__ __align__(16) float sm[];
  float* Qs = sm;                                  // [64][QS]
  float* Ks = Qs + kAttRows * QS;                  // [32][QS]
  float* Vs = Ks + kAttTile * QS;                  // [32][DH]
  float* Ss = Vs + kAttTile * DH;                  // [64][33]
  const int h = blockIdx.x, split = blockIdx.y, rb = blockIdx.z;
  const int tid = threadIdx.x;
  const int r = tid >> 2, qd = tid & 3;
  const int rg = rb * kAttRows + r;                // global row
  const int base = meta->base, n_rows = meta->n_rows;
  const int d = n_heads * DH;
  const int total = base + n_rows;                 // slots that can be visible
  int chunk = (total + gridDim.y - 1) / gridDim.y;
  chunk = (chunk + kAttTile - 1) / kAttTile * kAttTile;
  const int s_lo = split * chunk;
  int s_hi = s_lo + chunk;
  if (s_hi > total) s_hi = total;
  if (s_hi > max_ctx) s_hi = max_ctx;
  const bool live = rg < n_rows;
  u64 m0 = 0, m1 = 0;
  if (live) { m0 = meta->mask[rg][0]; m1 = meta->mask[rg][1]; }
  for (int i = tid; i < kAttRows * DH; i += kAttThreads) {
    const int rr = i / DH, c = i - rr * DH;
    const int g = rb * kAttRows + rr;
    Qs[rr * QS + c] = g < rows_cap ? to_f(q[(size_t)g * d + h * DH + c]) : 0.f;
  }
  float acc[SEG];
#pragma unroll
  for (int i = 0; i < SEG; ++i) acc[i] = 0.f;
  float mrun = -INFINITY, lrun = 0.f;
  const float scale = 1.0f / sqrtf((float)DH);
  const T* kh = kc + (size_t)h * max_ctx * DH;
  const T* vh = vc + (size_t)h * max_ctx * DH;
  for (int t0 = s_lo; t0 < s_hi; t0 += kAttTile) {
    __syncthreads();
    for (int i = tid; i < kAttTile * DH; i += kAttThreads) {
      const int j = i / DH, c = i - j * DH;
      const int s = t0 + j;
      float kvv = 0.f, vvv = 0.f;
      if (s < s_hi) { kvv = to_f(kh[(size_t)s * DH + c]); vvv = to_f(vh[(size_t)s * DH + c]); }
      Ks[j * QS + c] = kvv;
      Vs[j * DH + c] = vvv;
    }
    __syncthreads();
    float sc[kAttTile / 4];
    float tmax = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < kAttTile / 4; ++jj) {
      const int j = jj * 4 + qd;
      const int s = t0 + j;
      bool vis = live && s < s_hi;
      if (vis && s >= base) {
        const int m = s - base;
        vis = m < 64 ? ((m0 >> m) & 1ull) : ((m1 >> (m - 64)) & 1ull);
      }
      float dot = -INFINITY;
      if (vis) {
        const float4* qa = reinterpret_cast<const float4*>(Qs + r * QS);
        const float4* ka = reinterpret_cast<const float4*>(Ks + j * QS);
        dot = 0.f;
#pragma unroll 8
        for (int c = 0; c < DH / 4; ++c) {
          const float4 a = qa[c], b = ka[c];
          dot += a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
        }
        dot *= scale;
        tmax = fmaxf(tmax, dot);
      }
      sc[jj] = dot;
    }
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
    const float mnew = fmaxf(mrun, tmax);
    float corr = 1.f, psum = 0.f;
    if (mnew == -INFINITY) {                       // nothing visible yet for this row
#pragma unroll
      for (int jj = 0; jj < kAttTile / 4; ++jj) Ss[r * (kAttTile + 1) + jj * 4 + qd] = 0.f;
    } else {
      corr = expf(mrun - mnew);                    // exp(-inf) = 0 on the first visible tile
#pragma unroll
      for (int jj = 0; jj < kAttTile / 4; ++jj) {
        const float p = sc[jj] == -INFINITY ? 0.f : expf(sc[jj] - mnew);
        Ss[r * (kAttTile + 1) + jj * 4 + qd] = p;
        psum += p;
      }
    }
    psum += __shfl_xor_sync(0xffffffffu, psum, 1);
    psum += __shfl_xor_sync(0xffffffffu, psum, 2);
    lrun = lrun * corr + psum;
    mrun = mnew;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < SEG; ++i) acc[i] *= corr;
    for (int j = 0; j < kAttTile; ++j) {
      const float p = Ss[r * (kAttTile + 1) + j];
      if (p != 0.f) {
        const float4* va = reinterpret_cast<const float4*>(Vs + j * DH + qd * SEG);
#pragma unroll
        for (int c = 0; c < SEG / 4; ++c) {
          const float4 v = va[c];
          acc[c * 4 + 0] += p * v.x; acc[c * 4 + 1] += p * v.y;
          acc[c * 4 + 2] += p * v.z; acc[c * 4 + 3] += p * v.w;
        }
      }
    }
    __syncwarp();
  }
  if (rg < rows_cap) {
    const size_t o = (((size_t)split * n_heads + h) * rows_cap + rg);
    float4* dst = reinterpret_cast<float4*>(po + o * DH + qd * SEG);
#pragma unroll
    for (int c = 0; c < SEG / 4; ++c)
      dst[c] = make_float4(acc[c * 4], acc[c * 4 + 1], acc[c * 4 + 2], acc[c * 4 + 3]);
    if (qd == 0) { pml[o * 2] = mrun; pml[o * 2 + 1] = lrun; }
  }
}

template <typename T>
__global__ void attn_combine_kernel(const float* __restrict__ po, const float* __restrict__ pml,
                                    T* __restrict__ out, int splits, int rows_cap, int n_heads, int dh, int early) {
  if (early) pdl_launch_dependents();
  pdl_wait();
  if (!early) pdl_launch_dependents();
  const int r = blockIdx.x, h = blockIdx.y;
  const size_t stride = (size_t)n_heads * rows_cap, o0 = (size_t)h * rows_cap + r;
  if (splits <= 16) {
    // every load of the launch is issued before the first use: (max, sum) of all splits, then the partial
    // outputs of all splits for this thread's column
    float2 ml[16];
#pragma unroll
    for (int s = 0; s < 16; ++s)
      ml[s] = s < splits ? *reinterpret_cast<const float2*>(pml + (o0 + s * stride) * 2) : make_float2(-INFINITY, 0.f);
    for (int c = threadIdx.x; c < dh; c += blockDim.x) {
      float v[16];
#pragma unroll
      for (int s = 0; s < 16; ++s) v[s] = s < splits ? po[(o0 + s * stride) * dh + c] : 0.f;
      float M = -INFINITY;
#pragma unroll
      for (int s = 0; s < 16; ++s) M = fmaxf(M, ml[s].x);
      float den = 0.f, num = 0.f;
#pragma unroll
      for (int s = 0; s < 16; ++s)
        if (ml[s].x != -INFINITY) {
          const float w = expf(ml[s].x - M);
          den += ml[s].y * w;
          num += v[s] * w;
        }
      out[(size_t)r * n_heads * dh + h * dh + c] = from_f<T>(den > 0.f ? num / den : 0.f);
    }
    return;
  }
  float M = -INFINITY;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, pml[(o0 + s * stride) * 2]);
  float den = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float m = pml[(o0 + s * stride) * 2];
    if (m != -INFINITY) den += pml[(o0 + s * stride) * 2 + 1] * expf(m - M);
  }
  for (int c = threadIdx.x; c < dh; c += blockDim.x) {
    float num = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float m = pml[(o0 + s * stride) * 2];
      if (m != -INFINITY) num += po[(o0 + s * stride) * dh + c] * expf(m - M);
    }
    out[(size_t)r * n_heads * dh + h * dh + c] = from_f<T>(den > 0.f ? num / den : 0.f);
  }
}

template <typename T, int DH>
static void tree_attention_t(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, void* out,
                             int rows, int n_heads, int max_ctx, int splits, cudaStream_t st) {
  const size_t smem = sizeof(float) * (kAttRows * (DH + 4) + kAttTile * (DH + 4) + kAttTile * DH +
                                       kAttRows * (kAttTile + 1));
  cudaFuncSetAttribute(tree_attn_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  dim3 grid(n_heads, splits, (rows + kAttRows - 1) / kAttRows);
  launch_pdl(tree_attn_kernel<T, DH>, dim3(grid), dim3(kAttThreads), smem, st, (const T*)q, (const T*)kv.k, (const T*)kv.v, meta,
                                                          sc.o, sc.ml, rows, n_heads, max_ctx);
  launch_pdl(attn_combine_kernel<T>, dim3(dim3(rows, n_heads)), dim3(DH < 128 ? 64 : 128), 0, st, sc.o, sc.ml, (T*)out, splits, rows,
                                                                              n_heads, DH, 0);
}

void launch_attn_combine(AttnScratch sc, void* out, int dtype, int splits, int rows, int n_heads, int head_dim,
                         cudaStream_t st, int early) {
  AMPH_DISPATCH(dtype, launch_pdl(attn_combine_kernel<T>, dim3(dim3(rows, n_heads)), dim3(head_dim < 128 ? 64 : 128), 0, st, sc.o, sc.ml,
                                  (T*)out, splits, rows, n_heads, head_dim, early));
}

void launch_tree_attention(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, void* out, int dtype,
                           int rows, int n_heads, int head_dim, int max_ctx, int ctx_hi, int max_splits,
                           cudaStream_t st, int early, int separate_merge) {
  int splits = (ctx_hi + 127) / 128;
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  if (dtype == AMPH_DTYPE_BF16) {                    // tensor-core path; the kernel below serves fp32 caches
    if (launch_tree_attention_mma(q, kv, meta, sc, rows, n_heads, head_dim, max_ctx, splits, st,
                                  separate_merge ? nullptr : out))
      return;
    launch_pdl(attn_combine_kernel<bf16>, dim3(dim3(rows, n_heads)), dim3(head_dim < 128 ? 64 : 128), 0, st, sc.o, sc.ml, (bf16*)out, splits,
                                                                                        rows, n_heads, head_dim, early);
    return;
  }
  if (head_dim == 64) {
    AMPH_DISPATCH(dtype, (tree_attention_t<T, 64>(q, kv, meta, sc, out, rows, n_heads, max_ctx, splits, st)));
  } else {
    AMPH_DISPATCH(dtype, (tree_attention_t<T, 128>(q, kv, meta, sc, out, rows, n_heads, max_ctx, splits, st)));
  }
}

// --------------------------------------------------------------------------------------------
// SwiGLU on the fused gate / up projection: act = silu(gate) * up
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_kernel(PartialView P, T* __restrict__ act, int rows, int f, RowScale rs, int early) {
  if (early) pdl_launch_dependents();
  pdl_wait();
  if (!early) pdl_launch_dependents();
  const int r = blockIdx.x;
  const float sc = row_scale(rs, r);
  for (int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4; c < f; c += gridDim.y * blockDim.x * 4) {
    const float4 g = sum_partials4(P, r, c), u = sum_partials4(P, r, f + c);
    float4 o;
    float t;
    t = g.x * sc; o.x = t / (1.0f + expf(-t)) * (u.x * sc);
    t = g.y * sc; o.y = t / (1.0f + expf(-t)) * (u.y * sc);
    t = g.z * sc; o.z = t / (1.0f + expf(-t)) * (u.z * sc);
    t = g.w * sc; o.w = t / (1.0f + expf(-t)) * (u.w * sc);
    store4(act + (size_t)r * f + c, o);
  }
}

void launch_swiglu(PartialView P, void* act, int dtype, int rows, int f, cudaStream_t st, RowScale rs, int early) {
  int gy = (f / 4 + 255) / 256;
  if (gy > 16) gy = 16;
  AMPH_DISPATCH(dtype, launch_pdl(swiglu_kernel<T>, dim3(rows, gy), dim3(256), 0, st, P, (T*)act, rows, f, rs, early));
}

// --------------------------------------------------------------------------------------------
// Eq. 1's concatenation [feature ; embedding of the next token]
// --------------------------------------------------------------------------------------------
// emb == NULL: the ablation without the sampled token; the row is the feature alone (pitch d)
template <typename T>
__global__ void concat_kernel(const float* __restrict__ feat, const T* __restrict__ emb,
                              const int* __restrict__ next_tok, int vocab, T* __restrict__ cat, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = blockIdx.x;
  const size_t pitch = emb ? 2 * (size_t)d : (size_t)d;
  int t = next_tok[r];
  t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
  for (int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4; c < d; c += gridDim.y * blockDim.x * 4) {
    store4(cat + (size_t)r * pitch + c, load4(feat + (size_t)r * d + c));
    if (emb) store4(cat + (size_t)r * pitch + d + c, load4(emb + (size_t)t * d + c));
  }
}

void launch_concat(const float* feat, const void* tok_emb, const int* next_tok, int vocab, void* cat, int dtype,
                   int rows, int d, cudaStream_t st) {
  const int gy = (d / 4 + 255) / 256;
  AMPH_DISPATCH(dtype, launch_pdl(concat_kernel<T>, dim3(rows, gy), dim3(256), 0, st, feat, (const T*)tok_emb, next_tok, vocab, (T*)cat, d));
}

// --------------------------------------------------------------------------------------------
// Plain projection kernel: one warp per output feature, 128-bit weight loads, fp32 accumulate.
// Used for fp32 models, for shapes the tensor-core kernel does not cover, and as its A/B check.
// --------------------------------------------------------------------------------------------
template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<bf16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load16(const T* p, float* out);
template <>
__device__ __forceinline__ void load16<float>(const float* p, float* out) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void load16<bf16>(const bf16* p, float* out) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

template <typename T, int R>
__global__ void __launch_bounds__(256)
gemm_generic_kernel(const T* __restrict__ X, int ldx, const T* __restrict__ W, int out, int in,
                    float* __restrict__ P, int ldp, int col_off, int rows) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int V = Vec16<T>::N;
  const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (o >= out) return;
  const T* w = W + (size_t)o * in;
  for (int r0 = 0; r0 < rows; r0 += R) {
    float acc[R];
#pragma unroll
    for (int i = 0; i < R; ++i) acc[i] = 0.f;
    for (int k = lane * V; k < in; k += 32 * V) {
      float wv[V];
      load16<T>(w + k, wv);
#pragma unroll
      for (int i = 0; i < R; ++i) {
        if (r0 + i < rows) {
          float xv[V];
          load16<T>(X + (size_t)(r0 + i) * ldx + k, xv);
#pragma unroll
          for (int e = 0; e < V; ++e) acc[i] += wv[e] * xv[e];
        }
      }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
      float v = acc[i];
      for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
      if (lane == 0 && r0 + i < rows) P[(size_t)(r0 + i) * ldp + col_off + o] = v;
    }
  }
}

void launch_gemm_generic(const void* x, int ldx, const GemmSeg* segs, int n_seg, int out, int in, float* P,
                         int ldp, int rows, int dtype, cudaStream_t st) {
  const int blocks = (out + 7) / 8;
  for (int s = 0; s < n_seg; ++s) {
    AMPH_DISPATCH(dtype, launch_pdl(gemm_generic_kernel<T, 8>, dim3(blocks), dim3(256), 0, st, 
                             (const T*)x, ldx, (const T*)segs[s].w, out, in, P, ldp, s * out, rows));
  }
}

// --------------------------------------------------------------------------------------------
// draft module: last-row gather, head MLP epilogue (Eq. 2-4), fused K x K attention (Eq. 5)
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void gather_last_kernel(const float* __restrict__ h1, const float* __restrict__ h2,
                                   const DevState* __restrict__ s, float* __restrict__ last,
                                   T* __restrict__ last_act, int d) {
  pdl_wait();
  pdl_launch_dependents();
  int lr = s->n_pending - 1;
  lr = lr < 0 ? 0 : (lr >= kPendMax ? kPendMax - 1 : lr);
  const float* src = blockIdx.x == 0 ? h1 : h2;
  for (int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4; c < d; c += gridDim.y * blockDim.x * 4) {
    const float4 v = load4(src + (size_t)lr * d + c);
    store4(last + (size_t)blockIdx.x * d + c, v);
    store4(last_act + (size_t)blockIdx.x * d + c, v);
  }
}

void launch_gather_last(const float* h1, const float* h2, const DevState* st_dev, float* last, void* last_act,
                        int dtype, int d, cudaStream_t st) {
  const int gy = (d / 4 + 255) / 256;
  AMPH_DISPATCH(dtype, launch_pdl(gather_last_kernel<T>, dim3(2, gy), dim3(256), 0, st, h1, h2, st_dev, last, (T*)last_act, d));
}

template <typename T>
__global__ void gather_diag_kernel(PartialView P, T* __restrict__ out, int r) {
  pdl_wait();
  pdl_launch_dependents();
  const int k = blockIdx.x;
  for (int j = threadIdx.x; j < r; j += blockDim.x) out[(size_t)k * r + j] = from_f<T>(sum_partials(P, k, k * r + j));
}

void launch_gather_diag(PartialView P, void* out_act, int dtype, int K, int r, cudaStream_t st) {
  AMPH_DISPATCH(dtype, launch_pdl(gather_diag_kernel<T>, dim3(K), dim3(256), 0, st, P, (T*)out_act, r));
}

struct BiasPtrs { const void* b[kMaxK]; };

template <typename T>
__global__ void mlp_heads_kernel(PartialView P, const float* __restrict__ last, BiasPtrs bias,
                                 const T* __restrict__ pe, float* __restrict__ hp, float* __restrict__ ao,
                                 T* __restrict__ ao_act, int K, int n_sal, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const int k = blockIdx.x;
  const int row = (k < K / 2 || n_sal == 1) ? 0 : 1;       // Eq. 2: first half of the heads <- stage 1
  const T* b = (const T*)bias.b[k];
  for (int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4; c < d; c += gridDim.y * blockDim.x * 4) {
    const float4 w = sum_partials4(P, row, k * d + c), bb = load4(b + c), l = load4(last + (size_t)row * d + c),
                 e = load4(pe + (size_t)k * d + c);
    float4 v;
    float pre;
    pre = w.x + bb.x; v.x = l.x + pre / (1.0f + expf(-pre)) + e.x;
    pre = w.y + bb.y; v.y = l.y + pre / (1.0f + expf(-pre)) + e.y;
    pre = w.z + bb.z; v.z = l.z + pre / (1.0f + expf(-pre)) + e.z;
    pre = w.w + bb.w; v.w = l.w + pre / (1.0f + expf(-pre)) + e.w;
    store4(hp + (size_t)k * d + c, v);
    store4(ao + (size_t)k * d + c, v);          // the attention block updates this copy in place
    store4(ao_act + (size_t)k * d + c, v);
  }
}

void launch_mlp_heads(PartialView P, const float* last, const void* const* bias, const void* pe, float* hp,
                      float* ao, void* ao_act, int dtype, int K, int n_sal, int d, cudaStream_t st) {
  BiasPtrs bp;
  for (int k = 0; k < kMaxK; ++k) bp.b[k] = k < K ? bias[k] : nullptr;
  const int gy = (d / 4 + 127) / 128;
  AMPH_DISPATCH(dtype, launch_pdl(mlp_heads_kernel<T>, dim3(K, gy), dim3(128), 0, st, P, last, bp, (const T*)pe, hp, ao, (T*)ao_act,
                                                              K, n_sal, d));
}

// One block per attention head: the K x K score matrix, softmax and mixing stay in shared memory.
template <typename T>
__global__ void aeb_attention_kernel(PartialView P, T* __restrict__ out, int K, int n_heads, int dh) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) float sm[];
  float* qs = sm;                 // [K][dh]
  float* ks = qs + K * dh;
  float* vs = ks + K * dh;
  float* pr = vs + K * dh;        // [K][K]
  const int h = blockIdx.x, d = n_heads * dh;
  const int per = K * dh / 4;                            // float4 items per q / k / v block
  for (int i = threadIdx.x; i < 3 * per; i += blockDim.x) {
    const int which = i / per, j = (i - which * per) * 4;
    const int r = j / dh, c = j - r * dh;
    store4(sm + which * K * dh + j, sum_partials4(P, r, which * d + h * dh + c));
  }
  __syncthreads();
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int p = w; p < K * K; p += nw) {               // one warp per (i, j) score
    const int i = p / K, j = p - i * K;
    float dot = 0.f;
    for (int c = lane; c < dh; c += 32) dot += qs[i * dh + c] * ks[j * dh + c];
    for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
    if (lane == 0) pr[p] = dot / sqrtf((float)dh);
  }
  __syncthreads();
  if (threadIdx.x < K) {                              // bi-directional: every row sees every row
    const int i = threadIdx.x;
    float m = -INFINITY;
    for (int j = 0; j < K; ++j) m = fmaxf(m, pr[i * K + j]);
    float sum = 0.f;
    for (int j = 0; j < K; ++j) { const float e = expf(pr[i * K + j] - m); pr[i * K + j] = e; sum += e; }
    for (int j = 0; j < K; ++j) pr[i * K + j] /= sum;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < K * dh; idx += blockDim.x) {
    const int i = idx / dh, c = idx - i * dh;
    float acc = 0.f;
    for (int j = 0; j < K; ++j) acc += pr[i * K + j] * vs[j * dh + c];
    out[(size_t)i * d + h * dh + c] = from_f<T>(acc);
  }
}

void launch_aeb_attention(PartialView P, void* out_act, int dtype, int K, int n_heads, int head_dim,
                          cudaStream_t st) {
  const size_t smem = sizeof(float) * (3 * K * head_dim + K * K);
  AMPH_DISPATCH(dtype, launch_pdl(aeb_attention_kernel<T>, dim3(n_heads), dim3(128), smem, st, P, (T*)out_act, K, n_heads, head_dim));
}

// --------------------------------------------------------------------------------------------
// selection: top-k per drafting head (Eq. 6), greedy argmax per verified row
// order: value descending, equal values by ascending id
// --------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  return v > bv || (v == bv && i < bi);
}

__device__ void block_best(float& v, int& i, float* sv, int* si) {
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (better(ov, oi, v, i)) { v = ov; i = oi; }
  }
  const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) { sv[w] = v; si[w] = i; }
  __syncthreads();
  v = sv[0]; i = si[0];
  for (int k = 1; k < nw; ++k)
    if (better(sv[k], si[k], v, i)) { v = sv[k]; i = si[k]; }
}

struct TopkCounts { int c[kMaxK]; };

// Stage 1: block (head k, chunk j) reduces the split-K partials of its slice of the head's logits, stores
// them (debug tap) and selects the slice's own top-c_k in the order above.  Stage 2: one block per head
// merges the slices' candidates.  The global top-c_k are each among their slice's top-c_k, so the result is
// the exact top-c_k of the row, in order.
constexpr int kTopkChunks = kTopkCandChunks;
constexpr int kTopkThreads = 256;

__global__ void __launch_bounds__(kTopkThreads)
topk_slice_kernel(PartialView P, int vocab, int chunk, TopkCounts ck, float2* __restrict__ cand,
                  float* __restrict__ d_logits, int vec) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) float slice[];
  __shared__ float sv[32];
  __shared__ int si[32];
  const int k = blockIdx.x, j = blockIdx.y;
  const int lo = j * chunk, hi = lo + chunk < vocab ? lo + chunk : vocab;
  float* grow = d_logits + (size_t)k * vocab;
  for (int c = lo + threadIdx.x * 4; c < hi; c += blockDim.x * 4) {
    if (vec && c + 3 < hi) {
      const float4 v = sum_partials4(P, k, k * vocab + c);
      store4(grow + c, v);
      store4(slice + (c - lo), v);
    } else {
      for (int e = c; e < hi && e < c + 4; ++e) {
        const float v = sum_partials(P, k, k * vocab + e);
        grow[e] = v;
        slice[e - lo] = v;
      }
    }
  }
  __syncthreads();
  float pv = INFINITY;
  int pi = -1;
  for (int t = 0; t < ck.c[k]; ++t) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = lo + threadIdx.x; c < hi; c += blockDim.x) {
      const float v = slice[c - lo];
      const bool after_prev = v < pv || (v == pv && c > pi);       // strictly after the previous pick
      if (after_prev && better(v, c, bv, bi)) { bv = v; bi = c; }
    }
    block_best(bv, bi, sv, si);
    if (threadIdx.x == 0) cand[((size_t)k * gridDim.y + j) * kTopkStride + t] = make_float2(bv, __int_as_float(bi));
    pv = bv; pi = bi;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kTopkThreads)
topk_merge_kernel(const float2* __restrict__ cand, int n_chunks, TopkCounts ck, int* __restrict__ ids,
                  float* __restrict__ vals) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float sv[32];
  __shared__ int si[32];
  const int k = blockIdx.x, ckk = ck.c[k];
  const int n = n_chunks * ckk;                                    // candidates of this head
  float pv = INFINITY;
  int pi = -1;
  for (int t = 0; t < ckk; ++t) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = threadIdx.x; c < n; c += blockDim.x) {
      const float2 e = cand[((size_t)k * n_chunks + c / ckk) * kTopkStride + c % ckk];
      const int id = __float_as_int(e.y);
      const bool after_prev = e.x < pv || (e.x == pv && id > pi);
      if (id != 0x7fffffff && after_prev && better(e.x, id, bv, bi)) { bv = e.x; bi = id; }
    }
    block_best(bv, bi, sv, si);
    if (threadIdx.x == 0) { ids[k * kTopkStride + t] = bi; vals[k * kTopkStride + t] = bv; }
    pv = bv; pi = bi;
    __syncthreads();
  }
}

void launch_topk_heads(PartialView P, int vocab, int K, const int* ck, int* ids, float* vals, float* d_logits,
                       float* cand, cudaStream_t st) {
  TopkCounts c;
  for (int k = 0; k < kMaxK; ++k) c.c[k] = k < K ? ck[k] : 0;
  const int vec = vocab % 4 == 0 && P.ld % 4 == 0;
  int chunk = (vocab + kTopkChunks - 1) / kTopkChunks;
  chunk = (chunk + 3) / 4 * 4;
  const int n_chunks = (vocab + chunk - 1) / chunk;
  const size_t bytes = (size_t)chunk * sizeof(float);
  if (bytes > 48 * 1024) cudaFuncSetAttribute(topk_slice_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  launch_pdl(topk_slice_kernel, dim3(K, n_chunks), dim3(kTopkThreads), bytes, st, P, vocab, chunk, c,
             reinterpret_cast<float2*>(cand), d_logits, vec);
  launch_pdl(topk_merge_kernel, dim3(K), dim3(kTopkThreads), 0, st, reinterpret_cast<const float2*>(cand), n_chunks, c, ids, vals);
}

// Greedy choice per verified row in two stages, like the top-k above: block (row, slice) reduces the partials of
// its slice of the row, stores the logits (debug tap) and its best (value, id); one thread per row then merges the
// slices (ties -> lowest id, the same order as a single pass).
constexpr int kArgmaxSlices = 8;

__global__ void __launch_bounds__(256)
argmax_slice_kernel(PartialView P, int vocab, int chunk, float2* __restrict__ cand, float* __restrict__ logits_out, int vec) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float sv[32];
  __shared__ int si[32];
  const int r = blockIdx.x, j = blockIdx.y;
  const int lo = j * chunk, hi = lo + chunk < vocab ? lo + chunk : vocab;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = lo + threadIdx.x * 4; c < hi; c += blockDim.x * 4) {
    if (vec && c + 3 < hi) {
      const float4 v = sum_partials4(P, r, c);
      if (logits_out) store4(logits_out + (size_t)r * vocab + c, v);
      if (better(v.x, c, bv, bi)) { bv = v.x; bi = c; }
      if (better(v.y, c + 1, bv, bi)) { bv = v.y; bi = c + 1; }
      if (better(v.z, c + 2, bv, bi)) { bv = v.z; bi = c + 2; }
      if (better(v.w, c + 3, bv, bi)) { bv = v.w; bi = c + 3; }
    } else {
      for (int e = c; e < hi && e < c + 4; ++e) {
        const float v = sum_partials(P, r, e);
        if (logits_out) logits_out[(size_t)r * vocab + e] = v;
        if (better(v, e, bv, bi)) { bv = v; bi = e; }
      }
    }
  }
  block_best(bv, bi, sv, si);
  if (threadIdx.x == 0) cand[r * kArgmaxSlices + j] = make_float2(bv, __int_as_float(bi));
}

__global__ void argmax_merge_kernel(const float2* __restrict__ cand, int n_slices, int rows, int* __restrict__ amax) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int j = 0; j < n_slices; ++j) {
    const float2 e = cand[r * kArgmaxSlices + j];
    const int id = __float_as_int(e.y);
    if (better(e.x, id, bv, bi)) { bv = e.x; bi = id; }
  }
  amax[r] = bi;
}

void launch_argmax_rows(PartialView P, int vocab, int rows, int* amax, float* logits_out, float* cand, cudaStream_t st) {
  const int vec = vocab % 4 == 0 && P.ld % 4 == 0;
  int chunk = (vocab + kArgmaxSlices - 1) / kArgmaxSlices;
  chunk = (chunk + 3) / 4 * 4;
  const int n_slices = (vocab + chunk - 1) / chunk;
  launch_pdl(argmax_slice_kernel, dim3(rows, n_slices), dim3(256), 0, st, P, vocab, chunk, reinterpret_cast<float2*>(cand), logits_out, vec);
  launch_pdl(argmax_merge_kernel, dim3((rows + 127) / 128), dim3(128), 0, st, reinterpret_cast<const float2*>(cand), n_slices, rows, amax);
}

// --------------------------------------------------------------------------------------------
// control: row tables, tree tokens, acceptance, compaction
// --------------------------------------------------------------------------------------------
__device__ __forceinline__ void chain_mask(int r, u64* m) {       // bits 0..r
  m[0] = r >= 63 ? ~0ull : ((1ull << (r + 1)) - 1ull);
  m[1] = r < 64 ? 0ull : (r >= 127 ? ~0ull : ((1ull << (r - 63)) - 1ull));
}

__global__ void meta_chain_kernel(RowMeta* meta, int base, int n_rows) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = threadIdx.x;
  if (r == 0) { meta->base = base; meta->n_rows = n_rows; }
  meta->pos[r] = base + r;
  meta->slot[r] = base + r;
  chain_mask(r, meta->mask[r]);
}

void launch_meta_chain(RowMeta* meta, int base, int n_rows, cudaStream_t st) {
  launch_pdl(meta_chain_kernel, dim3(1), dim3(kMaxRows), 0, st, meta, base, n_rows);
}

__global__ void meta_pending_kernel(RowMeta* meta, const DevState* s) {
  pdl_wait();
  pdl_launch_dependents();
  const int r = threadIdx.x;
  int np = s->n_pending;
  np = np < 0 ? 0 : (np > kPendMax ? kPendMax : np);
  const int base = s->C - np;
  if (r == 0) { meta->base = base; meta->n_rows = np; }
  meta->pos[r] = base + r;
  meta->slot[r] = base + r;
  chain_mask(r, meta->mask[r]);
}

void launch_meta_pending(RowMeta* meta, const DevState* s, cudaStream_t st) {
  launch_pdl(meta_pending_kernel, dim3(1), dim3(kMaxRows), 0, st, meta, s);
}

// tok[0] = root; tok[n] = head depth[n]'s candidate of rank rank[n] (Appendix A.1); optional overrides;
// row table of the verification pass: position C + depth, slot C + n, mask = ancestors (Fig. 5).
__global__ void tree_build_kernel(const TreeDev* __restrict__ tree, DevState* s, const int* __restrict__ topk_ids,
                                  const int* __restrict__ override_tok, int* __restrict__ tok, RowMeta* meta) {
  pdl_wait();
  pdl_launch_dependents();
  const int n = threadIdx.x;
  const int N = tree->n_nodes;
  const int C = s->C;
  if (n == 0) { meta->base = C; meta->n_rows = N; }
  if (n < N) {
    if (n == 0) {
      tok[0] = s->root;
    } else {
      if (topk_ids) tok[n] = topk_ids[(tree->depth[n] - 1) * kTopkStride + tree->rank[n]];
      if (override_tok && override_tok[n] >= 0) tok[n] = override_tok[n];
    }
    meta->pos[n] = C + tree->depth[n];
    meta->slot[n] = C + n;
    meta->mask[n][0] = tree->anc[n][0];
    meta->mask[n][1] = tree->anc[n][1];
  } else {
    meta->pos[n] = C;
    meta->slot[n] = -1;
    meta->mask[n][0] = meta->mask[n][1] = 0ull;
  }
}

void launch_tree_build(const TreeDev* tree, DevState* s, const int* topk_ids, const int* override_tok, int* tok,
                       RowMeta* meta, cudaStream_t st) {
  launch_pdl(tree_build_kernel, dim3(1), dim3(kMaxRows), 0, st, tree, s, topk_ids, override_tok, tok, meta);
}

// Greedy acceptance: node n matches if its token equals the target's choice at its parent; it is
// accepted if every node on its root path matches; the deepest accepted node wins (lowest index
// among equals).  One block; the match set is a 128-bit mask tested against the ancestor masks.
__global__ void accept_kernel(const TreeDev* __restrict__ tree, DevState* s, const int* __restrict__ tok,
                              const int* __restrict__ amax) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ u64 match[2];
  __shared__ int best_key;
  const int n = threadIdx.x;
  const int N = tree->n_nodes;
  if (n < 2) match[n] = 0ull;
  if (n == 0) best_key = 0;
  __syncthreads();
  if (n < N) {
    const bool m = n == 0 || tok[n] == amax[tree->parent[n]];
    if (m) atomicOr(&match[n >> 6], 1ull << (n & 63));
  }
  __syncthreads();
  if (n < N) {
    const bool ok = ((tree->anc[n][0] & ~match[0]) | (tree->anc[n][1] & ~match[1])) == 0ull;
    if (ok) atomicMax(&best_key, tree->depth[n] * 256 + (255 - n));
  }
  __syncthreads();
  if (n == 0) {
    const int best = 255 - (best_key & 255);
    const int C = s->C;
    u64 a0 = tree->anc[best][0], a1 = tree->anc[best][1];
    int L = 0;
    while (a0 && L < kPendMax) { s->path[L++] = __ffsll((long long)a0) - 1; a0 &= a0 - 1; }
    while (a1 && L < kPendMax) { s->path[L++] = 64 + __ffsll((long long)a1) - 1; a1 &= a1 - 1; }
    const int nr = amax[best];
    for (int j = 0; j < L; ++j) {
      s->out_tok[j] = tok[s->path[j]];
      s->pend_tok[j] = j + 1 < L ? tok[s->path[j + 1]] : nr;
    }
    for (int j = L; j < kPendMax; ++j) { s->path[j] = -1; s->out_tok[j] = -1; }
    s->L = L;
    s->C_old = C;
    s->best = best;
    s->next_root = nr;
    s->C = C + L;
    s->root = nr;
    s->n_pending = L;
    s->step += 1;
  }
}

void launch_accept(const TreeDev* tree, DevState* s, const int* tok, const int* amax, cudaStream_t st) {
  launch_pdl(accept_kernel, dim3(1), dim3(kMaxRows), 0, st, tree, s, tok, amax);
}

// --------------------------------------------------------------------------------------------
// Sampling at a temperature (Table 2; Section 2, rejection sampling with point-mass proposals)
// --------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds; each multiplies counter words 0 and 2 by fixed odd constants,
// crosses the halves of the 64-bit products and mixes in the key, which is bumped by Weyl constants between rounds.
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
    c0 = n0; c1 = l1; c2 = n2; c3 = l0;
  }
  return c0;
}

constexpr int kSampleThreads = 1024;
constexpr int kSampleMaxChildren = 16;       // candidates a head keeps at most = children a node has at most

// One block per row.  w(v) = exp((l_v - max) / T); the row's uniform scaled by the sum of all weights is compared with
// running sums of w, so nothing is divided.  Sums are taken in a fixed order (deterministic).
__global__ void __launch_bounds__(kSampleThreads)
sample_rows_kernel(const float* __restrict__ logits, int vocab, int row0, const TreeDev* __restrict__ tree,
                   const int* __restrict__ tok, const DevState* __restrict__ s, int seq, int stream_id, float inv_t,
                   uint32_t k0, uint32_t k1, int* __restrict__ choice, float* __restrict__ uniforms_out) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float red[kSampleThreads / 32];
  __shared__ float part[kSampleThreads];
  __shared__ int kid_tok[kSampleMaxChildren];
  __shared__ int n_kids_s, result_s;
  __shared__ float target_s, base_s;
  const int r = blockIdx.x, row = row0 + r, tid = threadIdx.x;
  const float* l = logits + (size_t)row * vocab;
  // row maximum
  float m = -INFINITY;
  for (int v = tid; v < vocab; v += kSampleThreads) m = fmaxf(m, l[v]);
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  m = red[0];
  for (int i = 1; i < kSampleThreads / 32; ++i) m = fmaxf(m, red[i]);
  __syncthreads();
  // the distinct tokens of the row's children, in node order
  if (tid == 0) {
    int nk = 0;
    if (tree != nullptr && tok != nullptr) {
      const int N = tree->n_nodes;
      for (int c = r + 1; c < N && nk < kSampleMaxChildren; ++c) {
        if (tree->parent[c] != r) continue;
        const int x = tok[c];
        bool seen = x < 0 || x >= vocab;
        for (int j = 0; j < nk; ++j) seen = seen || kid_tok[j] == x;
        if (!seen) kid_tok[nk++] = x;
      }
    }
    n_kids_s = nk;
    result_s = -1;
  }
  __syncthreads();
  const int nk = n_kids_s;
  // every thread owns a contiguous range of ids; its weight sum leaves the children's tokens out
  const int chunk = (vocab + kSampleThreads - 1) / kSampleThreads;
  const int lo = tid * chunk, hi = lo + chunk < vocab ? lo + chunk : vocab;
  float mine = 0.f;
  for (int v = lo; v < hi; ++v) {
    bool kid = false;
    for (int j = 0; j < nk; ++j) kid = kid || kid_tok[j] == v;
    if (!kid) mine += __expf((l[v] - m) * inv_t);
  }
  part[tid] = mine;
  __syncthreads();
  if (tid == 0) {
    const uint32_t w = philox_first_word((uint32_t)r, (uint32_t)s->step, (uint32_t)seq, (uint32_t)stream_id, k0, k1);
    const float u = (float)(w >> 8) * (1.0f / 16777216.0f);
    if (uniforms_out) uniforms_out[r] = u;
    float kids = 0.f, rest = 0.f;
    float wk[kSampleMaxChildren];
    for (int j = 0; j < nk; ++j) { wk[j] = __expf((l[kid_tok[j]] - m) * inv_t); kids += wk[j]; }
    for (int i = 0; i < kSampleThreads; ++i) rest += part[i];
    const float target = u * (kids + rest);
    float acc = 0.f;
    int res = -1;
    for (int j = 0; j < nk && res < 0; ++j) {            // children first: accepted iff the running sum passes the target
      acc += wk[j];
      if (target < acc) res = kid_tok[j];
    }
    result_s = res;
    target_s = target;
    base_s = kids;
  }
  __syncthreads();
  if (result_s >= 0) {
    if (tid == 0) choice[row] = result_s;
    return;
  }
  // residual distribution: the first id, ascending, children's tokens left out, whose running sum exceeds the target
  if (tid == 0) {
    float acc = base_s;
    int owner = -1;
    for (int i = 0; i < kSampleThreads; ++i) {
      if (acc + part[i] > target_s && part[i] > 0.f) { owner = i; break; }
      acc += part[i];
    }
    if (owner < 0) {                                       // rounding left the target above the total: the last admissible id
      for (int i = kSampleThreads - 1; i >= 0 && owner < 0; --i)
        if (part[i] > 0.f) { owner = i; acc = -INFINITY; }   // its walk then ends on its last admissible id
    }
    n_kids_s = nk;
    result_s = -2 - owner;                                 // owner thread, encoded
    base_s = acc;
  }
  __syncthreads();
  const int owner = -2 - result_s;
  if (tid == owner) {
    float acc = base_s;
    int res = -1, last = -1;
    for (int v = lo; v < hi; ++v) {
      bool kid = false;
      for (int j = 0; j < nk; ++j) kid = kid || kid_tok[j] == v;
      if (kid) continue;
      last = v;
      acc += __expf((l[v] - m) * inv_t);
      if (acc > target_s) { res = v; break; }
    }
    choice[row] = res >= 0 ? res : last;
  }
}

void launch_sample_rows(const float* logits, int vocab, int row0, int n_rows, const TreeDev* tree, const int* tok,
                        const DevState* s, int seq, int stream_id, float temperature, unsigned long long seed, int* choice,
                        float* uniforms_out, cudaStream_t st) {
  launch_pdl(sample_rows_kernel, dim3(n_rows), dim3(kSampleThreads), 0, st, logits, vocab, row0, tree, tok, s, seq, stream_id,
             1.0f / temperature, (uint32_t)(seed & 0xffffffffull), (uint32_t)(seed >> 32), choice, uniforms_out);
}

// Block l < n_layers moves layer l's accepted key / value rows: slot C_old + j <- C_old + path[j].
// path is strictly increasing with path[j] >= j, so no source is overwritten before it is read and
// the moves are independent.  The extra last block queues the accepted hidden rows for the next draft.
template <typename T>
__global__ void compact_kernel(const DevState* __restrict__ s, const KvView* __restrict__ kv, int n_layers,
                               int n_heads, int dh, int max_ctx, const float* __restrict__ hidden,
                               float* __restrict__ pend_h, int d) {
  pdl_wait();
  pdl_launch_dependents();
  const int L = s->L, C0 = s->C_old;
  if ((int)blockIdx.x == n_layers) {
    for (int j = 0; j < L; ++j)
      for (int c = threadIdx.x; c < d; c += blockDim.x) pend_h[(size_t)j * d + c] = hidden[(size_t)s->path[j] * d + c];
    return;
  }
  T* kc = (T*)kv[blockIdx.x].k;
  T* vc = (T*)kv[blockIdx.x].v;
  for (int j = 1; j < L; ++j) {
    const int src = C0 + s->path[j], dst = C0 + j;
    if (src == dst || src >= max_ctx) continue;
    for (int i = threadIdx.x; i < n_heads * dh; i += blockDim.x) {
      const int h = i / dh, c = i - h * dh;
      const size_t so = ((size_t)h * max_ctx + src) * dh + c, dd = ((size_t)h * max_ctx + dst) * dh + c;
      kc[dd] = kc[so];
      vc[dd] = vc[so];
    }
  }
}

void launch_compact(const DevState* s, const KvView* kv_layers, int n_layers, int dtype, int n_heads,
                    int head_dim, int max_ctx, const float* hidden, float* pend_h, int d, cudaStream_t st) {
  AMPH_DISPATCH(dtype, launch_pdl(compact_kernel<T>, dim3(n_layers + 1), dim3(256), 0, st, s, kv_layers, n_layers, n_heads, head_dim,
                                                                       max_ctx, hidden, pend_h, d));
}

__global__ void reduce_partials_kernel(PartialView P, float* __restrict__ y, int rows, int cols) {
  pdl_wait();
  pdl_launch_dependents();
  const size_t n = (size_t)rows * cols;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / cols), c = (int)(i - (size_t)r * cols);
    y[i] = sum_partials(P, r, c);
  }
}

void launch_reduce_partials(PartialView P, float* y, int rows, int cols, cudaStream_t st) {
  const size_t n = (size_t)rows * cols;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  launch_pdl(reduce_partials_kernel, dim3(blocks), dim3(256), 0, st, P, y, rows, cols);
}

template <typename T>
__global__ void kv_export_kernel(const T* __restrict__ c, int row0, int n_heads, int dh, int max_ctx,
                                 float* __restrict__ dst) {
  pdl_wait();
  pdl_launch_dependents();
  const int slot = row0 + blockIdx.x;
  for (int i = threadIdx.x; i < n_heads * dh; i += blockDim.x) {
    const int h = i / dh, e = i - h * dh;
    dst[(size_t)blockIdx.x * n_heads * dh + i] = to_f(c[((size_t)h * max_ctx + slot) * dh + e]);
  }
}

void launch_kv_export(KvView kv, int which, int dtype, int row0, int rows, int n_heads, int head_dim, int max_ctx,
                      float* dst, cudaStream_t st) {
  if (rows <= 0) return;
  AMPH_DISPATCH(dtype, launch_pdl(kv_export_kernel<T>, dim3(rows), dim3(256), 0, st, (const T*)(which ? kv.v : kv.k), row0, n_heads,
                                                                 head_dim, max_ctx, dst));
}

// End of prefill: root = greedy choice after the last prompt token; the last prompt row stays
// pending so that the first draft runs the adaptation layers on it (Eq. 1).
__global__ void prefill_tail_kernel(DevState* s, const int* __restrict__ amax, int last_row,
                                    const float* __restrict__ hidden, float* __restrict__ pend_h, int d, int C) {
  pdl_wait();
  pdl_launch_dependents();
  for (int c = threadIdx.x; c < d; c += blockDim.x) pend_h[c] = hidden[(size_t)last_row * d + c];
  if (threadIdx.x == 0) {
    const int root = amax[last_row];
    s->C = C;
    s->root = root;
    s->n_pending = 1;
    s->pend_tok[0] = root;
    s->L = 0;
    s->C_old = C;
    s->best = 0;
    s->next_root = root;
    s->step = 0;
  }
}

void launch_prefill_tail(DevState* s, const int* amax, int last_row, const float* hidden, float* pend_h, int d,
                         int C, cudaStream_t st) {
  launch_pdl(prefill_tail_kernel, dim3(1), dim3(256), 0, st, s, amax, last_row, hidden, pend_h, d, C);
}

}  // namespace amph
