// Tensor-core projection path (tcgen05 MMA with TMEM accumulators, operands staged by TMA).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include "amph_internal.cuh"

namespace amph {

struct TcGemm;

// Registers the activation buffers (bf16, row-major [rows][cols]) projections may read from.
// err_flag: device int that a kernel sets to AMPH_ERR_TIMEOUT if a bounded pipeline wait gives up.
// Returns NULL if the driver entry point for tensor maps is unavailable.
TcGemm* tc_gemm_create(void* const* xbufs, const int* xrows, const int* xcols, int n, int* err_flag);

// P[s][row][seg*out + o] (fp32 partial sums over K-splits s) = X[row][:] . W_seg[o][:].
// Returns false (nothing launched) if the shape is not covered; the caller then uses the plain kernel.
bool tc_gemm_launch(TcGemm* g, int xb, const void* const* w, int n_seg, int out, int in, int rows, float* P,
                    size_t p_floats, int* splits, size_t* split_stride, cudaStream_t st);

// Gate / up projection with SwiGLU in the epilogue (no partial sums, no separate kernel):
//   act[row][o] = silu(g * s) * (u * s),  g = X[row] . W_gate[o],  u = X[row] . W_up[o],  s = the row's deferred RMSNorm scale.
// w_gate, w_up: bf16 [f, in]; act: bf16 [rows][f].  Takes at most 64 rows and needs the two matrices less than 1 TB
// apart (they are fetched through one tensor map); returns false, nothing launched, if the form is not available.
bool tc_gemm_launch_swiglu(TcGemm* g, int xb, const void* w_gate, const void* w_up, int f, int in, int rows, void* act,
                           const RowScale& rs, cudaStream_t st);

// q / k / v projection with the rotary embedding and the cache write in the epilogue (no partial sums, no separate kernel):
//   q[row] <- rope(s * X[row] . Wq^T),  K cache[slot[row]] <- rope(s * X[row] . Wk^T),  V cache[slot[row]] <- s * X[row] . Wv^T
// with s the row's deferred RMSNorm scale, rope the rotation of pairs (i, i + dh / 2) by the angles in `rope`
// ([rows][dh / 2] (cos, sin)).  Weights bf16 [n_heads * dh, in]; q bf16 [rows][n_heads * dh]; caches [head][slot][dh].
// Takes at most 64 rows and head_dim 64 or 128; returns false, nothing launched, if the form is not available.
bool tc_gemm_launch_qkv_rope(TcGemm* g, int xb, const void* wq, const void* wk, const void* wv, int n_heads, int dh, int in,
                             int rows, void* q, KvView kv, const RowMeta* meta, const float2* rope, int max_ctx,
                             const RowScale& rs, cudaStream_t st);

// Asks for the head of every gate / up weight tile (about budget_bytes in all: the first K blocks of all rows of both
// matrices) to be brought into L2.  A plain launch for a side stream: meant to run while the main stream's kernels leave
// HBM idle.  Returns false, nothing launched, if the two matrices cannot be described by one tensor map.
bool tc_gemm_prefetch_swiglu(TcGemm* g, const void* w_gate, const void* w_up, int f, int in, size_t budget_bytes, cudaStream_t st);
void tc_gemm_destroy(TcGemm* g);

// Points activation buffer `xb` of an existing plan set at another bf16 [rows][cols] buffer and the error flag at
// another device int (host-side bookkeeping only; tensor maps of buffers seen before stay cached, up to a bound).
void tc_gemm_rebind(TcGemm* g, int xb, void* ptr, int rows, int cols, int* err_flag);

// Failure-path self-test: every barrier wait of later launches gives up after wait_limit_ns, and the first stage's
// barrier of each CTA expects extra_tx bytes more than its copies deliver (so that wait can never complete).
void tc_gemm_set_selftest(TcGemm* g, unsigned long long wait_limit_ns, unsigned extra_tx);

}  // namespace amph
