// Tensor-core projection path (tcgen05 MMA with TMEM accumulators, operands staged by TMA).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include "amph_internal.cuh"

namespace amph {

struct TcGemm;

// Work fused into the projection kernel.  Every CTA still leaves its split-K partial tile in P; the CTA that
// arrives last at a tile (a counter per tile, no waiting) sums the partials in split order and applies:
//   QKV_ROPE : three segments q, k, v of width n_heads * head_dim: deferred RMS division, rotary embedding,
//              q -> q buffer, k / v -> KV-cache slots of the row table;
//   RESIDUAL : x += y; xn = gain * x (not normalised); ss_part[row][tile] = sum of squares over the tile;
//   SWIGLU   : two segments gate, up: deferred RMS division, act = silu(gate) * up.
enum { TC_EPI_NONE = 0, TC_EPI_QKV_ROPE = 1, TC_EPI_RESIDUAL = 2, TC_EPI_SWIGLU = 3 };
constexpr int kTcCounterInts = 4096;

struct TcEpilogue {
  int mode = TC_EPI_NONE;
  int* counters = nullptr;        // kTcCounterInts ints, all zero between launches
  RowScale rs;                    // QKV_ROPE, SWIGLU: division left over from the norm that fed this projection
  float* x = nullptr;             // RESIDUAL: fp32 residual stream [rows][out]
  void* xn = nullptr;             //           bf16 gain * x
  const void* gain = nullptr;     //           bf16 [out], may be NULL (then xn / ss_part are not written)
  float* ss_part = nullptr;       //           [rows][out / 128]
  void* act = nullptr;            // SWIGLU: bf16 [rows][out]
  const RowMeta* meta = nullptr;  // QKV_ROPE
  const float2* rope = nullptr;
  void* q = nullptr;
  void* kc = nullptr;
  void* vc = nullptr;
  int n_heads = 0, head_dim = 0, max_ctx = 0;
};

// Registers the activation buffers (bf16, row-major [rows][cols]) projections may read from.
// err_flag: device int that a kernel sets to AMPH_ERR_TIMEOUT if a bounded pipeline wait gives up.
// Returns NULL if the driver entry point for tensor maps is unavailable.
TcGemm* tc_gemm_create(void* const* xbufs, const int* xrows, const int* xcols, int n, int* err_flag);

// P[s][row][seg*out + o] (fp32 partial sums over K-splits s) = X[row][:] . W_seg[o][:].
// Returns false (nothing launched) if the shape is not covered; the caller then uses the plain kernel.
bool tc_gemm_launch(TcGemm* g, int xb, const void* const* w, int n_seg, int out, int in, int rows, float* P,
                    size_t p_floats, int* splits, size_t* split_stride, cudaStream_t st,
                    const TcEpilogue* epi = nullptr);

void tc_gemm_destroy(TcGemm* g);

}  // namespace amph
