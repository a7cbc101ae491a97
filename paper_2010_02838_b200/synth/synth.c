/*
 * synth.c -- seeded, counter-based synthetic input generator (host side).
 *
 * Holds none of the objective's arithmetic: it only turns (seed, stream, index) into standard
 * normal floats or uniform integers, so that tests, benchmark and oracle all see identical bits
 * and any slice of a tensor can be regenerated on its own.
 *
 * Mixing function: the 64-bit finaliser of SplitMix64 (Steele, Lea, Flood 2014), applied to a
 * Weyl sequence over the counter.  Normals: Box-Muller on two 53-bit uniforms per pair of
 * outputs (element 2k takes the cosine branch of pair k, element 2k+1 the sine branch).
 */
#include <math.h>
#include <stdint.h>

static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

static inline uint64_t draw(uint64_t seed, uint64_t stream, uint64_t counter, uint64_t lane) {
  uint64_t key = mix64(seed * 0x9E3779B97F4A7C15ULL + stream * 0xD1B54A32D192ED03ULL + 0x2545F4914F6CDD1DULL);
  return mix64(key + (2 * counter + lane + 1) * 0x9E3779B97F4A7C15ULL);
}

/* out[i] = standard normal number `first + i` of the (seed, stream) sequence, as float */
void synth_normal_f32(uint64_t seed, uint64_t stream, uint64_t first, uint64_t count, float* out) {
  const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < (int64_t)count; ++i) {
    const uint64_t e = first + (uint64_t)i;
    const uint64_t pair = e >> 1;
    const double u1 = ((double)(draw(seed, stream, pair, 0) >> 11) + 1.0) * (1.0 / 9007199254740992.0); /* (0,1] */
    const double u2 = (double)(draw(seed, stream, pair, 1) >> 11) * (1.0 / 9007199254740992.0);         /* [0,1) */
    const double rad = sqrt(-2.0 * log(u1));
    const double ang = two_pi * u2;
    out[i] = (float)((e & 1) ? rad * sin(ang) : rad * cos(ang));
  }
}

/* out[i] = uniform integer in [0, bound) number `first + i` of the (seed, stream) sequence */
void synth_uniform_i32(uint64_t seed, uint64_t stream, uint64_t first, uint64_t count, int32_t bound, int32_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < (int64_t)count; ++i) {
    const uint64_t v = draw(seed, stream, first + (uint64_t)i, 0);
    out[i] = (int32_t)(((v >> 32) * (uint64_t)(uint32_t)bound) >> 32);
  }
}

/* out[i] = raw 64-bit draw (used for seeded permutations) */
void synth_raw_u64(uint64_t seed, uint64_t stream, uint64_t first, uint64_t count, uint64_t* out) {
  for (uint64_t i = 0; i < count; ++i) out[i] = draw(seed, stream, first + i, 0);
}
