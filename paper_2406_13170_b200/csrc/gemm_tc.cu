#include "gemm_tc.cuh"
namespace amph {
struct TcGemm {};
TcGemm* tc_gemm_create(void* const*, const int*, const int*, int, int*) { return nullptr; }
bool tc_gemm_launch(TcGemm*, int, const void* const*, int, int, int, int, float*, size_t, int*, size_t*, cudaStream_t) { return false; }
void tc_gemm_destroy(TcGemm* g) { delete g; }
}
