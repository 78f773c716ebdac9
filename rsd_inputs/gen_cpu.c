/* CPU side of the synthetic-weight generator: fills host fp32 arrays.
 * For 16-bit configurations the fp32 array holds the bfloat16-rounded values. */
#include "weight_init.h"
#include <stddef.h>

void rsd_inputs_fill_f32(float* out, uint32_t seed, uint32_t tensor_id, uint64_t first_index,
                         uint64_t count, float scale, int round_bf16) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < (int64_t)count; ++i) {
    float v = rsd_in_weight_value(seed, tensor_id, first_index + (uint64_t)i, scale);
    if (round_bf16) v = rsd_in_bf16_bits_to_f32(rsd_in_f32_to_bf16_bits(v));
    out[i] = v;
  }
}

void rsd_inputs_fill_const_f32(float* out, uint64_t count, float value) {
  for (uint64_t i = 0; i < count; ++i) out[i] = value;
}

/* Raw Philox block, exported so tests can pin the generator to known-answer vectors. */
void rsd_inputs_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  rsd_in_philox4x32_10(ctr, key, out);
}
