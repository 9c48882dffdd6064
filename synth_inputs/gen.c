/* Seeded synthetic-input generator (counter based, so any element can be
 * produced independently and in parallel).  It holds none of the decoding
 * method's arithmetic: it only fills buffers with reproducible random bits.
 *
 *   u64 stream : z = splitmix64_finalise(key + (idx + 1) * GOLDEN)
 *   normal     : Box-Muller (cosine branch) in double from the two 32-bit
 *                halves of z, scaled by `std`, rounded to nearest-even bf16
 *   token ids  : z mod vocab
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* out[i] = bf16(std * N(0,1)) for i in [0, count) */
void synth_normal_bf16(uint64_t key, double std, int64_t count, uint16_t *out) {
  const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    uint64_t z = mix64(key + (uint64_t)(i + 1) * GOLDEN);
    double u1 = ((double)(uint32_t)(z >> 32) + 1.0) * (1.0 / 4294967296.0); /* (0,1] */
    double u2 = (double)(uint32_t)z * (1.0 / 4294967296.0);                 /* [0,1) */
    double g = sqrt(-2.0 * log(u1)) * cos(two_pi * u2);
    out[i] = f32_to_bf16_rne((float)(std * g));
  }
}

/* out[i] = bf16(value) */
void synth_const_bf16(double value, int64_t count, uint16_t *out) {
  uint16_t v = f32_to_bf16_rne((float)value);
  for (int64_t i = 0; i < count; ++i) out[i] = v;
}

/* out[i] uniform in [0, modulus) */
void synth_uniform_i32(uint64_t key, int32_t modulus, int64_t count, int32_t *out) {
  for (int64_t i = 0; i < count; ++i) {
    uint64_t z = mix64(key + (uint64_t)(i + 1) * GOLDEN);
    out[i] = (int32_t)(z % (uint64_t)modulus);
  }
}
