/* Seeded synthetic-weight generator shared by the CPU oracle's callers and the GPU callers.
 *
 * This header holds NO arithmetic of the decoding method: it only defines how a synthetic
 * weight value is derived from (seed, tensor id, logical element index), so that every
 * consumer sees bit-identical inputs.  It compiles as plain C and as CUDA.
 *
 * Value recipe ("weights N(0, sigma)", random init):
 *   - Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11),
 *     key = (seed, tensor id), counter = (index low, index high, 0, domain tag);
 *   - the 128 output bits are read as eight 16-bit uniforms whose sum S (an Irwin-Hall
 *     variate, exact in integers) is centred and scaled:  value = (2S - 8*65535) * scale,
 *     scale = sigma / (2 * sqrt(8 * (65536^2 - 1) / 12)) rounded once to fp32 by the caller.
 *     The integer 2S - 8*65535 is below 2^21, hence exact in fp32, and the single fp32
 *     multiply is correctly rounded on every IEEE machine: CPU and GPU agree bit for bit
 *     (no transcendental functions are involved, unlike Box-Muller).
 *   - for 16-bit storage the fp32 value is rounded to bfloat16, round-to-nearest-even,
 *     by integer bit manipulation.
 */
#ifndef RSD_INPUTS_WEIGHT_INIT_H
#define RSD_INPUTS_WEIGHT_INIT_H

#include <stdint.h>

#ifdef __CUDACC__
#define RSD_IN_HD __host__ __device__ static inline
#else
#define RSD_IN_HD static inline
#endif

#define RSD_IN_DOMAIN_WEIGHT 0x57454947u /* counter word 3 for weight draws */

RSD_IN_HD void rsd_in_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* fp32 value of logical element `idx` of tensor `tensor_id`. */
RSD_IN_HD float rsd_in_weight_value(uint32_t seed, uint32_t tensor_id, uint64_t idx, float scale) {
  uint32_t ctr[4] = {(uint32_t)idx, (uint32_t)(idx >> 32), 0u, RSD_IN_DOMAIN_WEIGHT};
  uint32_t key[2] = {seed, tensor_id};
  uint32_t o[4];
  rsd_in_philox4x32_10(ctr, key, o);
  int32_t s = 0;
  for (int i = 0; i < 4; ++i) s += (int32_t)(o[i] & 0xFFFFu) + (int32_t)(o[i] >> 16);
  int32_t centred = 2 * s - 8 * 65535;
  return (float)centred * scale;
}

/* Round an fp32 value to the nearest bfloat16 (ties to even); returns the 16 payload bits. */
RSD_IN_HD uint16_t rsd_in_f32_to_bf16_bits(float v) {
  union { float f; uint32_t u; } cvt;
  cvt.f = v;
  uint32_t u = cvt.u;
  uint32_t rounding = 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)((u + rounding) >> 16);
}

RSD_IN_HD float rsd_in_bf16_bits_to_f32(uint16_t b) {
  union { float f; uint32_t u; } cvt;
  cvt.u = (uint32_t)b << 16;
  return cvt.f;
}

#endif
