// Gate + compaction for callers that must not allocate device memory.
//
// Some hosts of this library run where a cudaMalloc is not an option: inside a serving loop whose
// memory was carved up once at start-up and is fully spoken for, in a process that shares the GPU
// under a fixed memory budget, or in a latency-critical section where an allocation (which may
// synchronise the device) is forbidden.  rsd_k_gate_compact asks such a caller for a scratch
// buffer it may not be able to provide.  The variant below keeps that scratch inside the library
// image instead: a fixed array in device global memory that exists on every GPU that loads the
// library, from load until the process exits.
#include "../../include/rsd.h"

#include <mutex>
#include <string>

#include "kernels.cuh"

namespace {

// One int per block of 1024 rows: 1024 ints cover RSD_GATE_STATIC_MAX_ROWS = 2^20 rows (4 KiB).
constexpr int kStaticBlocks = RSD_GATE_STATIC_MAX_ROWS / 1024;
static __device__ __align__(256) int32_t g_gate_block_counts[kStaticBlocks];

// In host code `g_gate_block_counts` is only a handle for the runtime, not a device address, so
// the address is looked up once per device (with that device current) and remembered.
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
int32_t* g_scratch_ptr[kMaxDevices] = {};
std::string g_error;

}  // namespace

extern "C" {

// The text is copied under the lock into a buffer of the calling thread, so a failing call on another host
// thread cannot reallocate it under the reader; it stays valid until this thread asks again.
const char* rsd_k_gate_compact_static_error(void) {
  thread_local std::string copy;
  std::lock_guard<std::mutex> lock(g_mutex);
  copy = g_error;
  return copy.c_str();
}

int rsd_k_gate_compact_static(const float* rewards, const uint8_t* live, float delta, uint8_t* accept,
                              int32_t* rej_idx, int32_t* n_rej, int32_t B, void* cuda_stream) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!rewards || !live || !accept || !rej_idx || !n_rej) {
    g_error = "rsd_k_gate_compact_static: null pointer argument";
    return RSD_ERR_ARG;
  }
  if (B < 1 || B > RSD_GATE_STATIC_MAX_ROWS) {
    g_error = "rsd_k_gate_compact_static: B = " + std::to_string(B) + " is outside 1.." +
              std::to_string(RSD_GATE_STATIC_MAX_ROWS) +
              " (the built-in scratch holds one counter per 1024 rows); use rsd_k_gate_compact with "
              "caller-provided scratch for larger batches";
    return RSD_ERR_ARG;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    g_error = std::string("rsd_k_gate_compact_static: no usable current device: ") + cudaGetErrorString(e);
    return RSD_ERR_CUDA;
  }
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_gate_block_counts);
    if (e != cudaSuccess || p == nullptr) {
      g_error = std::string("rsd_k_gate_compact_static: cudaGetSymbolAddress failed: ") + cudaGetErrorString(e);
      return RSD_ERR_CUDA;
    }
    g_scratch_ptr[dev] = (int32_t*)p;
  }
  // Nothing in the scratch has to start at zero: the counting kernel overwrites the counter of
  // every block it launches before the scan reads it, so a previous call's contents are harmless.
  e = rsd::launch_gate_compact_large(rewards, live, delta, accept, rej_idx, n_rej, g_scratch_ptr[dev], B,
                                     (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) {
    g_error = std::string("rsd_k_gate_compact_static: launch failed: ") + cudaGetErrorString(e);
    return RSD_ERR_CUDA;
  }
  return RSD_OK;
}

}  // extern "C"
