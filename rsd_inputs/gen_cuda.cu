/* GPU side of the synthetic-weight generator: fills device arrays (fp32 or bfloat16) with
 * exactly the values gen_cpu.c produces for the same (seed, tensor id, element index). */
#include "weight_init.h"
#include <cuda_runtime.h>
#include <cuda_bf16.h>

namespace {

template <bool kBf16>
__global__ void fill_kernel(void* out, uint32_t seed, uint32_t tensor_id, uint64_t first_index,
                            uint64_t count, float scale) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) {
    float v = rsd_in_weight_value(seed, tensor_id, first_index + i, scale);
    if (kBf16) {
      reinterpret_cast<uint16_t*>(out)[i] = rsd_in_f32_to_bf16_bits(v);
    } else {
      reinterpret_cast<float*>(out)[i] = v;
    }
  }
}

template <bool kBf16>
__global__ void const_kernel(void* out, uint64_t count, float value) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) {
    if (kBf16) {
      reinterpret_cast<uint16_t*>(out)[i] = rsd_in_f32_to_bf16_bits(value);
    } else {
      reinterpret_cast<float*>(out)[i] = value;
    }
  }
}

int grid_for(uint64_t count) {
  uint64_t blocks = (count + 255) / 256;
  if (blocks > 148ull * 16) blocks = 148ull * 16;
  if (blocks == 0) blocks = 1;
  return (int)blocks;
}

}  // namespace

/* dtype: 0 = fp32, 1 = bfloat16.  `out` is a device pointer to `count` elements; element i
 * receives the value of logical index first_index + i.  Returns the cudaError_t of the launch. */
extern "C" int rsd_inputs_fill_device(void* out, int dtype, uint32_t seed, uint32_t tensor_id,
                                      uint64_t first_index, uint64_t count, float scale, void* stream) {
  if (count == 0) return 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (dtype == 1) fill_kernel<true><<<grid_for(count), 256, 0, s>>>(out, seed, tensor_id, first_index, count, scale);
  else fill_kernel<false><<<grid_for(count), 256, 0, s>>>(out, seed, tensor_id, first_index, count, scale);
  return (int)cudaGetLastError();
}

extern "C" int rsd_inputs_fill_const_device(void* out, int dtype, uint64_t count, float value, void* stream) {
  if (count == 0) return 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (dtype == 1) const_kernel<true><<<grid_for(count), 256, 0, s>>>(out, count, value);
  else const_kernel<false><<<grid_for(count), 256, 0, s>>>(out, count, value);
  return (int)cudaGetLastError();
}
