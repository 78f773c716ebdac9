// GEMM dispatch.  (The tcgen05 path is added in this file.)
#include "common.cuh"
#include "kernels.cuh"

#include <atomic>

namespace rsd {

static std::atomic<uint64_t> g_launches{0};
cudaError_t launched(int n_kernels) {
  g_launches.fetch_add((uint64_t)n_kernels, std::memory_order_relaxed);
  return cudaGetLastError();
}
uint64_t launches_total() { return g_launches.load(std::memory_order_relaxed); }

bool gemm_tc_supported(int dtype, int M, int N, int K) { (void)dtype; (void)M; (void)N; (void)K; return false; }
size_t gemm_scratch_bytes(int M) { (void)M; return 4096; }

cudaError_t launch_gemm_tc(const void*, const void*, float*, int, int, int, int, void*, size_t, const int32_t*, cudaStream_t) {
  return cudaErrorNotSupported;
}

cudaError_t launch_gemm(int dtype, const void* W, const void* x, float* y, int M, int N, int K, int accumulate,
                        int impl, void* scratch, size_t scratch_bytes, const int32_t* n_active, cudaStream_t s) {
  if (impl == 2 || (impl == 0 && gemm_tc_supported(dtype, M, N, K)))
    return launch_gemm_tc(W, x, y, M, N, K, accumulate, scratch, scratch_bytes, n_active, s);
  return launch_gemm_simt(dtype, W, x, y, M, N, K, accumulate, n_active, s);
}

}  // namespace rsd
