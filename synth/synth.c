/*
 * Seeded synthetic input generators (test and benchmark infrastructure).
 *
 * This file holds no attention arithmetic: it only turns (seed, tensor id,
 * flat element index) into a number.  Both the CPU oracle's callers and the
 * CUDA path's callers fill their input tensors from here, so the two sides
 * see identical bit patterns.
 *
 * Generator: counter based.  For element i of tensor t under seed s two
 * 64-bit hashes are drawn with the splitmix64 finaliser (Steele, Lea, Flood,
 * "Fast splittable pseudorandom number generators", 2014), mapped to two
 * uniforms and combined with the Box-Muller transform in double precision.
 * Because a value depends only on (s, t, i), any slice of a long stream can
 * be produced on its own: a block of frames of a minute-long token stream is
 * the same whether the stream is generated whole or block by block.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

static inline uint64_t key_of(uint64_t seed, uint64_t tensor_id) {
  return mix64(mix64(seed) ^ (tensor_id * 0xD1B54A32D192ED03ull));
}

/* standard normal for counter i under key */
static inline double gauss_at(uint64_t key, uint64_t i) {
  uint64_t h1 = mix64(key ^ (2 * i));
  uint64_t h2 = mix64(key ^ (2 * i + 1));
  double u1 = ((double)(h1 >> 11) + 1.0) * (1.0 / 9007199254740992.0); /* (0,1] */
  double u2 = (double)(h2 >> 11) * (1.0 / 9007199254740992.0);         /* [0,1) */
  return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
}

/* float -> bfloat16 bits, round to nearest even (inputs here are finite) */
static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* out[j] = bf16( (float)(gauss(start + j) * scale) ), j in [0, count) */
void synth_gauss_bf16(uint16_t* out, int64_t count, uint64_t seed, uint64_t tensor_id,
                      int64_t start, double scale) {
  const uint64_t key = key_of(seed, tensor_id);
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < count; ++j)
    out[j] = f32_to_bf16_rne((float)(gauss_at(key, (uint64_t)(start + j)) * scale));
}

/* same stream, kept in fp32 (for the fp32 I/O path) */
void synth_gauss_f32(float* out, int64_t count, uint64_t seed, uint64_t tensor_id,
                     int64_t start, double scale) {
  const uint64_t key = key_of(seed, tensor_id);
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < count; ++j)
    out[j] = (float)(gauss_at(key, (uint64_t)(start + j)) * scale);
}

/* small integers in {-r, ..., r}, exactly representable in bf16 for r <= 128 */
void synth_smallint_bf16(uint16_t* out, int64_t count, uint64_t seed, uint64_t tensor_id,
                         int64_t start, int32_t r) {
  const uint64_t key = key_of(seed, tensor_id);
  const uint64_t span = (uint64_t)(2 * r + 1);
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < count; ++j) {
    uint64_t h = mix64(key ^ (uint64_t)(start + j));
    int32_t v = (int32_t)((h >> 20) % span) - r;
    out[j] = f32_to_bf16_rne((float)v);
  }
}

/* uniform integers in [0, n) (for one-hot feature indices and the like) */
void synth_index_i32(int32_t* out, int64_t count, uint64_t seed, uint64_t tensor_id,
                     int64_t start, int32_t n) {
  const uint64_t key = key_of(seed, tensor_id);
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < count; ++j) {
    uint64_t h = mix64(key ^ (uint64_t)(start + j));
    out[j] = (int32_t)((h >> 20) % (uint64_t)n);
  }
}
