// amph_project_noalloc: the projection primitive for callers that cannot allocate device memory.
//
// A serving engine that has already handed every free byte of the GPU to its own memory pool, or a
// latency-critical loop that must not risk the implicit synchronisation of an allocation, cannot call
// cudaMalloc (nor ask its framework for a tensor) just to give the projection its split-K scratch.
// This variant keeps that scratch in a fixed array inside the library image instead.  The array is part
// of the module: every GPU that loads the library holds these bytes until the process exits.
#include <stdarg.h>
#include <stdio.h>

#include <mutex>

#include "amph_internal.cuh"
#include "gemm_tc.cuh"

using namespace amph;

namespace {

constexpr size_t kStaticScratchBytes = AMPH_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Split-K partial sums (after a 256-byte header whose first int32 is the device error flag).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];     // device address of g_static_scratch, per device ordinal
TcGemm* g_plans[kMaxDevices];          // tensor-core plan set per device, created by the first tensor-core call and kept

// In host code `g_static_scratch` is only a handle of the symbol, not an address a kernel may
// dereference: the device address has to be looked up, once per device, with that device current.
void say(char* msg, size_t len, const char* fmt, ...) {
  if (!msg || !len) return;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(msg, len, fmt, ap);
  va_end(ap);
}

amph_status scratch_for_current_device(void** out, char* msg, size_t len) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    say(msg, len, "no usable current device (%s)", e == cudaSuccess ? "ordinal out of range" : cudaGetErrorString(e));
    return AMPH_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      say(msg, len, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      return AMPH_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return AMPH_OK;
}

}  // namespace

extern "C" {

amph_status amph_project_noalloc(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg,
                                 int32_t out, int32_t in, int32_t rows, int32_t dtype, int32_t use_tensor_core,
                                 float* y_dev, int32_t* status_dev, void* stream, char* err_msg, size_t err_len) {
  if (err_msg && err_len) err_msg[0] = 0;
  if (!x_dev || !w || !y_dev) { say(err_msg, err_len, "NULL pointer"); return AMPH_ERR_INVALID_ARG; }
  if (n_seg < 1 || n_seg > kMaxK || out < 1 || in < 8 || rows < 1 || rows > kMaxRows || x_rows_cap < rows) {
    say(err_msg, err_len, "bad projection shape");
    return AMPH_ERR_SHAPE;
  }
  if ((dtype != AMPH_DTYPE_F32 && dtype != AMPH_DTYPE_BF16) || in % (dtype == AMPH_DTYPE_F32 ? 4 : 8)) {
    say(err_msg, err_len, "unknown dtype, or a row of `in` elements is not a multiple of 16 bytes");
    return AMPH_ERR_SHAPE;
  }
  // One split of partial sums must fit: rows padded to 16 x all output features, fp32.
  const size_t ld = (size_t)n_seg * out;
  const size_t rows_pad = rows <= 16 ? 16 : (size_t)(rows + 15) / 16 * 16;
  const size_t need = 256 + rows_pad * ld * sizeof(float);
  if (need > kStaticScratchBytes) {
    say(err_msg, err_len,
        "projection too large for the built-in scratch: %zu rows x %zu features need %zu bytes, the limit is %zu "
        "(use amph_project with caller-provided scratch)", rows_pad, ld, need, kStaticScratchBytes);
    return AMPH_ERR_WORKSPACE;
  }
  void* base = nullptr;
  amph_status rc = scratch_for_current_device(&base, err_msg, err_len);
  if (rc != AMPH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  int* err = status_dev ? status_dev : (int*)base;
  float* P = (float*)((char*)base + 256);
  const size_t p_floats = (kStaticScratchBytes - 256) / sizeof(float);
  // The array keeps whatever the previous call left.  Only the status word must start at zero; the partial
  // sums are fully overwritten before anything reads them.
  if (cudaMemsetAsync(err, 0, sizeof(int), st) != cudaSuccess) {
    say(err_msg, err_len, "clearing the status word failed: %s", cudaGetErrorString(cudaGetLastError()));
    return AMPH_ERR_CUDA;
  }
  PartialView pv;
  pv.p = P;
  pv.ld = (int)ld;
  if (use_tensor_core) {
    if (dtype != AMPH_DTYPE_BF16) { say(err_msg, err_len, "the tensor-core kernel takes bf16 only"); return AMPH_ERR_SHAPE; }
    void* xb[1] = {const_cast<void*>(x_dev)};
    const int xr[1] = {x_rows_cap}, xc[1] = {in};
    // The plan set (driver entry point, kernel attributes, cached tensor maps: host-side bookkeeping only) is made
    // once per device and re-pointed at this call's activations, so a steady-state call encodes at most one new map.
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    TcGemm*& g = g_plans[dev];
    if (!g) g = tc_gemm_create(xb, xr, xc, 1, err);
    if (!g) { say(err_msg, err_len, "tensor-map encoder unavailable or not an sm_100 device"); return AMPH_ERR_CUDA; }
    tc_gemm_rebind(g, 0, xb[0], xr[0], xc[0], err);
    int splits = 0;
    size_t stride = 0;
    const bool ok = tc_gemm_launch(g, 0, w, n_seg, out, in, rows, P, p_floats, &splits, &stride, st);
    if (!ok) { say(err_msg, err_len, "shape not covered by the tensor-core kernel"); return AMPH_ERR_SHAPE; }
    pv.splits = splits;
    pv.split_stride = stride;
  } else {
    GemmSeg segs[kMaxK];
    for (int s = 0; s < n_seg; ++s) segs[s].w = w[s];
    launch_gemm_generic(x_dev, in, segs, n_seg, out, in, P, (int)ld, rows, dtype, st);
    pv.splits = 1;
    pv.split_stride = 0;
  }
  launch_reduce_partials(pv, y_dev, rows, (int)ld, st);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { say(err_msg, err_len, "launch failed: %s", cudaGetErrorString(e)); return AMPH_ERR_CUDA; }
  return AMPH_OK;
}

}  // extern "C"
