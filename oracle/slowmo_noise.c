/*
 * Oracle side of the counter-based synthetic-noise generator. TEST INFRASTRUCTURE:
 * see slowmo_oracle.h. The CUDA library has its own, separately written generator;
 * the two must agree bit for bit on the integer stream and on the binary32 normals.
 *
 * The paper (Eq. 1) only assumes a stochastic gradient oracle per worker; the concrete
 * stream below is this project's stand-in for it: a SplitMix64 hash of
 * (seed, outer t, local k, worker w, coordinate j) mapped to N(0,1) by Box-Muller, both
 * outputs of each Box-Muller pair being used (for coordinates 2q and 2q+1).
 *
 * Built with -ffp-contract=off: every rounding below is written out; fused operations
 * are explicit fmaf calls.
 */
#include "slowmo_oracle.h"

#include <math.h>

static const uint64_t GOLDEN_GAMMA = 0x9E3779B97F4A7C15ull; /* SplitMix64 increment */

/* SplitMix64's output function: xor-shift-multiply twice, final xor-shift. */
uint64_t oracle_mix64(uint64_t s) {
  s ^= s >> 30;
  s *= 0xBF58476D1CE4E5B9ull;
  s ^= s >> 27;
  s *= 0x94D049BB133111EBull;
  s ^= s >> 31;
  return s;
}

/*
 * A SplitMix64 generator adds GOLDEN_GAMMA to its state and then outputs mix64(state).
 * Its j-th output (j from 0) after starting at `key` is therefore mix64(key + (j+1)*gamma):
 * random access in j.
 */
uint64_t oracle_stream_word(uint64_t key, uint64_t j) {
  return oracle_mix64(key + GOLDEN_GAMMA * (j + 1));
}

/* Fold one more integer into a key: advance by (v+1) increments and mix. */
static uint64_t absorb(uint64_t s, uint64_t v) { return oracle_mix64(s + GOLDEN_GAMMA * (v + 1)); }

uint64_t oracle_stream_key(uint32_t tag, uint64_t seed, uint64_t t, uint32_t k, uint32_t w) {
  uint64_t s = seed;
  s = absorb(s, tag);
  s = absorb(s, t);
  s = absorb(s, k);
  s = absorb(s, w);
  s = absorb(s, 0);
  return s;
}

/* Top 24 bits of the word as U = k1 * 2^-24 in [0,1). */
float oracle_word_to_unit(uint64_t r) {
  uint32_t k1 = (uint32_t)(r >> 40);
  return ldexpf((float)k1, -24);
}

/*
 * ln(u) for u = n * 2^-24, n an integer in [1, 2^24], in binary32.
 * n = f * 2^E with f in [sqrt(1/2), sqrt(2)); ln f = 2 atanh(s), s = (f-1)/(f+1),
 * atanh series cut after s^9; ln u = (E-24) ln2 + ln f.
 */
static float ln_unit24(uint32_t n) {
  int E;
  float f = frexpf((float)n, &E); /* f in [0.5, 1), n = f * 2^E exactly */
  f = f * 2.0f;                   /* f in [1, 2)   */
  E = E - 1;
  if (f > 1.41421354f) { /* binary32 nearest to sqrt(2) */
    f = f * 0.5f;
    E = E + 1;
  }
  float s = (f - 1.0f) / (f + 1.0f);
  float w = s * s;
  float p = (float)(1.0 / 9.0);
  p = fmaf(w, p, (float)(1.0 / 7.0));
  p = fmaf(w, p, (float)(1.0 / 5.0));
  p = fmaf(w, p, (float)(1.0 / 3.0));
  p = fmaf(w, p, 1.0f);
  float lnf = (2.0f * s) * p;
  return fmaf((float)(E - 24), 0.693147182f, lnf);
}

/*
 * cos and sin of the angle 2 pi k2 / 2^24 for a 24-bit integer k2, in binary32.
 * The top two bits pick the quadrant; inside the quadrant the angle psi = (pi/2) r / 2^22
 * is reflected about pi/4 so that a Taylor polynomial is only ever evaluated on [0, pi/4].
 */
static void cos_sin_turn24(uint32_t k2, float *cos_out, float *sin_out) {
  uint32_t q = k2 >> 22;
  uint32_t r = k2 & 0x3FFFFFu;
  int reflected = r > 0x200000u;
  if (reflected) r = 0x400000u - r;                          /* psi' = pi/2 - psi */
  float theta = 3.14159274f * ldexpf((float)r, -23);         /* (pi/2) * r / 2^22 */
  float t2 = theta * theta;

  float sin_t; /* theta - theta^3/3! + ... + theta^9/9! */
  {
    float p = (float)(1.0 / 362880.0);
    p = fmaf(t2, p, (float)(-1.0 / 5040.0));
    p = fmaf(t2, p, (float)(1.0 / 120.0));
    p = fmaf(t2, p, (float)(-1.0 / 6.0));
    p = fmaf(t2, p, 1.0f);
    sin_t = theta * p;
  }
  float cos_t; /* 1 - theta^2/2! + ... - theta^10/10! */
  {
    float p = (float)(-1.0 / 3628800.0);
    p = fmaf(t2, p, (float)(1.0 / 40320.0));
    p = fmaf(t2, p, (float)(-1.0 / 720.0));
    p = fmaf(t2, p, (float)(1.0 / 24.0));
    p = fmaf(t2, p, (float)(-1.0 / 2.0));
    p = fmaf(t2, p, 1.0f);
    cos_t = p;
  }
  /* cos psi and sin psi of the un-reflected in-quadrant angle */
  float cos_psi = reflected ? sin_t : cos_t;
  float sin_psi = reflected ? cos_t : sin_t;
  switch (q) { /* angle = q pi/2 + psi */
    case 0: *cos_out = cos_psi;  *sin_out = sin_psi;  break;
    case 1: *cos_out = -sin_psi; *sin_out = cos_psi;  break;
    case 2: *cos_out = -cos_psi; *sin_out = -sin_psi; break;
    default: *cos_out = sin_psi; *sin_out = -cos_psi; break;
  }
}

/*
 * Box-Muller: one word gives the two independent normals
 *   z[0] = sqrt(-2 ln u1) cos(2 pi u2),  z[1] = sqrt(-2 ln u1) sin(2 pi u2),
 * with u1 = (k1+1) 2^-24 in (0,1] from bits 63..40 and u2 = k2 2^-24 in [0,1) from bits 39..16.
 */
void oracle_word_to_normal_pair(uint64_t r, float z[2]) {
  uint32_t k1 = (uint32_t)(r >> 40);
  uint32_t k2 = (uint32_t)(r >> 16) & 0xFFFFFFu;
  float radius = sqrtf(-2.0f * ln_unit24(k1 + 1));
  float c, s;
  cos_sin_turn24(k2, &c, &s);
  z[0] = radius * c;
  z[1] = radius * s;
}

/*
 * The normal of coordinate j in the stream `key`: coordinates 2q and 2q+1 share word q of
 * the stream and take the cosine and the sine output of its Box-Muller pair.
 */
float oracle_stream_normal(uint64_t key, uint64_t j) {
  float z[2];
  oracle_word_to_normal_pair(oracle_stream_word(key, j >> 1), z);
  return z[j & 1];
}

/* Bulk form of oracle_word_to_normal_pair for tests: out[2i], out[2i+1] from words[i]. */
void oracle_words_to_normals(const uint64_t *words, uint64_t n, float *out) {
  for (uint64_t i = 0; i < n; ++i) oracle_word_to_normal_pair(words[i], out + 2 * i);
}

void oracle_stream_export(uint32_t tag, uint64_t seed, uint64_t t, uint32_t k, uint32_t w,
                          uint64_t j0, uint64_t n, uint64_t *words, float *normals) {
  uint64_t key = oracle_stream_key(tag, seed, t, k, w);
  for (uint64_t i = 0; i < n; ++i) {
    if (words) words[i] = oracle_stream_word(key, j0 + i);
    if (normals) normals[i] = oracle_stream_normal(key, j0 + i);
  }
}

/* a_j = a_lo + (a_hi - a_lo) U, U from the curvature stream. */
float oracle_curvature(const oracle_config *cfg, uint64_t j) {
  uint64_t key = oracle_stream_key(ORACLE_TAG_CURVATURE, cfg->seed, 0, 0, 0);
  float U = oracle_word_to_unit(oracle_stream_word(key, j));
  return fmaf(cfg->a_hi - cfg->a_lo, U, cfg->a_lo);
}

/* c_{w,j} = c_std z, z from worker w's centre stream. */
float oracle_centre(const oracle_config *cfg, uint32_t w, uint64_t j) {
  uint64_t key = oracle_stream_key(ORACLE_TAG_CENTRE, cfg->seed, 0, 0, w);
  return cfg->c_std * oracle_stream_normal(key, j);
}

/* G_{w,j} = sigma z, z from worker w's supplied-gradient stream. */
float oracle_supplied_gradient(const oracle_config *cfg, uint32_t w, uint64_t j) {
  uint64_t key = oracle_stream_key(ORACLE_TAG_SUPPLIED, cfg->seed, 0, 0, w);
  return cfg->sigma * oracle_stream_normal(key, j);
}
