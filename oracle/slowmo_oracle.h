/*
 * CPU oracle for the SlowMo data-parallel hot path (Wang, Tantia, Ballas, Rabbat, ICLR 2020).
 *
 * THIS IS TEST INFRASTRUCTURE. It is a plain, slow, scalar restatement of the paper's
 * Algorithm 1 with the update directions of Table C.1, used to check the CUDA library.
 * It shares no code with the CUDA path and the CUDA path never calls it. Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * Every step of Algorithm 1 is elementwise in the parameter index j, so the oracle is
 * evaluated on any list of indices j independently: the whole T x tau trajectory of the m
 * replicas of one coordinate is run before moving to the next coordinate.
 *
 * Two arithmetic modes are built from the same source (slowmo_oracle.c):
 *   *_f32  every operation in IEEE binary32 in the stated order (the parity gate: the
 *          state of the method is fp32);
 *   *_f64  the same formulas in binary64 (used to pin the oracle against the identities,
 *          closed forms and library routines the paper's statements imply).
 * The synthetic noise z and the synthetic inputs a, c, G are fp32 values in both modes
 * (they are inputs of the method, produced by the counter-based generator in
 * slowmo_noise.c), widened exactly in the f64 mode.
 */
#ifndef SLOWMO_ORACLE_H
#define SLOWMO_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- counter-based noise (slowmo_noise.c) ------------------------------------------ */

/* Stream tags: which quantity a word of the stream is used for. */
enum {
  ORACLE_TAG_CURVATURE = 1, /* a_j      (t = k = w = 0)                  */
  ORACLE_TAG_CENTRE    = 2, /* c_{w,j}  (t = k = 0)                      */
  ORACLE_TAG_GRADNOISE = 3, /* z in the stochastic gradient at (t,k,w,j) */
  ORACLE_TAG_SUPPLIED  = 5  /* fixed supplied gradient G_{w,j}           */
};

/* SplitMix64 output function (Steele, Lea, Flood 2014) applied to one 64-bit word. */
uint64_t oracle_mix64(uint64_t s);
/* j-th output (j = 0, 1, ...) of a SplitMix64 generator whose state starts at `key`. */
uint64_t oracle_stream_word(uint64_t key, uint64_t j);
/* Key of the stream for (tag, seed, outer t, local k, worker w). */
uint64_t oracle_stream_key(uint32_t tag, uint64_t seed, uint64_t t, uint32_t k, uint32_t w);
/* Uniform in [0,1) with 24 bits from the top of a word; exact in binary32. */
float oracle_word_to_unit(uint64_t r);
/* Two independent N(0,1) draws from one word: Box-Muller (cosine, sine), binary32 arithmetic. */
void oracle_word_to_normal_pair(uint64_t r, float z[2]);
void oracle_words_to_normals(const uint64_t *words, uint64_t n, float *out); /* out[2i], out[2i+1] from words[i] */
/* Normal of coordinate j in a stream: output (j & 1) of the pair made from word j >> 1. */
float oracle_stream_normal(uint64_t key, uint64_t j);
/* Bulk export for tests, for j0 <= j < j0 + n: words[i] = word j0+i of the stream,
 * normals[i] = normal of coordinate j0+i (which is made from word (j0+i) >> 1). */
void oracle_stream_export(uint32_t tag, uint64_t seed, uint64_t t, uint32_t k, uint32_t w,
                          uint64_t j0, uint64_t n, uint64_t *words, float *normals);

/* ---- Algorithm 1 (slowmo_oracle.c) -------------------------------------------------- */

enum {
  ORACLE_BASE_NESTEROV = 0,     /* Table C.1, SGD row (local Nesterov momentum, no communication) */
  ORACLE_BASE_ADAM = 1,         /* Table C.1, Adam row                                             */
  ORACLE_BASE_SGP_NESTEROV = 2, /* Algorithm 2 (stochastic gradient push with Nesterov momentum)   */
  ORACLE_BASE_SGP_ADAM = 3      /* Table C.1, SGP (Adam) row                                       */
};
enum { ORACLE_BUF_RESET = 0, ORACLE_BUF_MAINTAIN = 1, ORACLE_BUF_AVERAGE = 2 };
enum {
  ORACLE_GRAD_GENERATED = 0,     /* noisy quadratic gradient, generated from the hash     */
  ORACLE_GRAD_SUPPLIED_HASH = 1, /* fixed G_{w,j} = sigma * z(tag 5), same at every step   */
  ORACLE_GRAD_SUPPLIED_ARRAY = 2 /* caller passes G for every step                        */
};

typedef struct {
  uint32_t m;   /* workers                                   */
  uint32_t tau; /* inner steps per outer iteration           */
  uint32_t T;   /* outer iterations                          */
  float alpha;  /* slow learning rate   (Algorithm 1)        */
  float beta;   /* slow momentum factor (Algorithm 1)        */
  float gamma;  /* base learning rate, used when gamma_t is NULL */
  int32_t base;          /* ORACLE_BASE_*                    */
  float mu;              /* beta_local of Table C.1 (SGD row) */
  float weight_decay;    /* L2 coefficient added to the gradient */
  float adam_b1, adam_b2, adam_eps; /* Table C.1 (Adam row)  */
  int32_t buffer_policy; /* ORACLE_BUF_*  (Algorithm 1, first statement of the outer loop) */
  int32_t grad_mode;     /* ORACLE_GRAD_*                    */
  uint64_t seed;
  float a_lo, a_hi;      /* curvature a_j ~ U[a_lo, a_hi)    */
  float c_std;           /* centre c_{w,j} ~ N(0, c_std^2)   */
  float sigma;           /* gradient-noise scale             */
  float x_init;          /* x_{0,0} in every coordinate      */
  int32_t no_average;    /* 0: Algorithm 1 as printed. 1: the variant of Section 6 that skips the
                            exact average: every worker applies Eq. (2), (3) to its own x_{t,tau},
                            with its own slow momentum u^{(i)} and its own outer iterate           */
} oracle_config;

/*
 * Run Algorithm 1 for the n coordinates j_idx[0..n-1] (or j0, j0+1, ... when j_idx is NULL).
 *
 *   gamma_t   NULL, or T base learning rates, one per outer iteration.
 *   G         only for ORACLE_GRAD_SUPPLIED_ARRAY: [T*tau][m][n] gradients, step-major.
 *   x, h, v   outputs [m][n] (row = worker); v may be NULL for Nesterov.
 *   anchor,u  outputs [n]: x_{T,0} and u_T; [m][n] (one row per worker) when no_average is set.
 *   dbar      optional [T][tau][n]: the worker-mean direction (1/m) sum_i d^{(i)}_{t,k}
 *             (always accumulated in binary64), for the identities of the paper's
 *             "Equivalent Updates" section.
 * Returns 0, or -1 on invalid arguments. Threads over coordinates with OpenMP.
 */
int slowmo_oracle_run_f32(const oracle_config *cfg, const float *gamma_t, const uint64_t *j_idx,
                          uint64_t j0, uint64_t n, const float *G, float *x, float *anchor,
                          float *u, float *h, float *v, double *dbar);
int slowmo_oracle_run_f64(const oracle_config *cfg, const float *gamma_t, const uint64_t *j_idx,
                          uint64_t j0, uint64_t n, const float *G, double *x, double *anchor,
                          double *u, double *h, double *v, double *dbar);

/* Hop distance 2^q of the directed exponential graph at global base-optimizer step s for m
 * workers: q cycles through 0 .. floor(log2(m-1)); 0 when m = 1 (no peer). */
uint32_t oracle_sgp_hops(uint32_t m, uint64_t s);

/* Synthetic inputs for coordinates, as the run above sees them (fp32 values). */
float oracle_curvature(const oracle_config *cfg, uint64_t j);
float oracle_centre(const oracle_config *cfg, uint32_t w, uint64_t j);
float oracle_supplied_gradient(const oracle_config *cfg, uint32_t w, uint64_t j);

int slowmo_oracle_threads(void); /* OpenMP threads a run will use */

#ifdef __cplusplus
}
#endif
#endif
