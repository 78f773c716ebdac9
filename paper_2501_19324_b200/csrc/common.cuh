// Shared device helpers of the RSD step-loop kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace rsd {

// ---- programmatic dependent launch ------------------------------------------------------------------
// Every kernel starts with RSD_PDL_SYNC(): it lets the next kernel in the stream be scheduled early
// (launch_dependents) and then waits until the kernels before it have completed and their writes
// are visible (wait).  Launched through launch_pdl, a kernel's blocks can therefore be resident and
// past their set-up while the previous kernel drains, instead of paying the launch gap after it.
// Without the launch attribute both instructions do nothing.
#define RSD_PDL_SYNC()                                             \
  do {                                                             \
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); \
    asm volatile("griddepcontrol.wait;" ::: "memory");             \
  } while (0)

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}
#define RSD_LAUNCH(kernel, grid, block, smem, stream, ...) \
  (void)::rsd::launch_pdl(kernel, dim3(grid), dim3(block), (size_t)(smem), stream, __VA_ARGS__)

// ---- element conversion ---------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// Stores v as a GEMM operand.  fp32 operands are stored as they are.  bf16 operands are stored as a
// pair hi = bf16(v), lo = bf16(v - hi) when a second array is given, so that the tensor-core product
// with bf16 weights sees the activation to about 16 mantissa bits (hi and lo are two rows of the same
// GEMM whose results are added).
template <typename T> __device__ __forceinline__ void store_operand(T* hi, T* lo, size_t i, float v);
template <> __device__ __forceinline__ void store_operand<float>(float* hi, float*, size_t i, float v) { hi[i] = v; }
template <> __device__ __forceinline__ void store_operand<__nv_bfloat16>(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float v) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  hi[i] = h;
  if (lo != nullptr) lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

// A single fp16 operand (the dense passes that run on fp16 copies of the weights): no low half.
template <> __device__ __forceinline__ void store_operand<__half>(__half* hi, __half*, size_t i, float v) { hi[i] = __float2half_rn(v); }

// 16-byte vector of elements of type T, unpacked to fp32.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  float v[4];
  __device__ __forceinline__ void load(const float* p) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ void load_stream(const float* p) {
    float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  float v[8];
  __device__ __forceinline__ void unpack(uint4 t) {
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { unpack(*reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void load_stream(const __nv_bfloat16* p) { unpack(__ldcs(reinterpret_cast<const uint4*>(p))); }
};

// ---- reductions ----------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

// Sum over a block of up to 1024 threads; every thread receives the total.  `smem` holds 33 floats.
__device__ __forceinline__ float block_sum(float v, float* smem) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? smem[lane] : 0.f;
  t = warp_sum(t);
  return t;
}

// Exclusive prefix sum of one int per thread over a block of up to 1024 threads (thread order);
// *total receives the block sum.  `smem` holds 33 ints.
__device__ __forceinline__ int block_exclusive_scan(int v, int* smem, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) smem[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = (lane < nw) ? smem[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xFFFFFFFFu, winc, o);
      if (lane >= o) winc += n;
    }
    smem[lane] = winc - w;            // exclusive offset of each warp
    if (lane == 31) smem[32] = winc;  // block total
  }
  __syncthreads();
  *total = smem[32];
  return smem[warp] + inc - v;
}

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) -----------------------------------------
// Ten rounds; each round multiplies words 0 and 2 by the two round multipliers, mixes the high
// halves with words 1 and 3 and the key, and the key advances by the two Weyl increments.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// 32 random bits -> uniform on (0,1): (2k+1) / 2^24 with k the top 23 bits (exact in fp32).
__device__ __forceinline__ float uniform_from_bits(uint32_t x) {
  return (float)(2u * (x >> 9) + 1u) * (1.0f / 16777216.0f);
}

}  // namespace rsd
