// Tensor-core projection path (tcgen05 MMA with TMEM accumulators, operands staged by TMA).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

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

void tc_gemm_destroy(TcGemm* g);

}  // namespace amph
