/*
 * Oracle: Algorithm 1 (Slow Momentum) with the base-optimizer directions of Table C.1,
 * one coordinate j at a time. TEST INFRASTRUCTURE: see slowmo_oracle.h.
 *
 * This file is compiled twice: with -DORACLE_F64=0 (binary32, the parity gate) and with
 * -DORACLE_F64=1 (binary64, for the pins). Built with -ffp-contract=off; every fused
 * operation is an explicit FMA(), every other operation rounds once in `real`.
 *
 * Readings where the paper leaves a choice (each also listed in the design notes):
 *  - Table C.1's Adam step count l: 1-based number of Adam steps since the buffers were
 *    last zeroed (the caption's l = k or l = t tau + k would divide by 1 - beta^0 = 0).
 *    Under the "average" policy buffers are not zeroed, so l keeps counting.
 *  - Weight decay is L2: added to the gradient before the momentum update.
 *  - The buffer policy of outer iteration t+1 is applied right after the outer update
 *    of iteration t (at t = 0 every policy is a no-op because the buffers are zero).
 *  - Stochastic gradient push (Algorithm 2; Table C.1, SGP rows): the graph is the
 *    time-varying directed exponential graph with one peer per step: at global step
 *    s = t tau + k worker i sends to worker (i + 2^q) mod m, q = s mod (floor(log2(m-1)) + 1),
 *    and keeps half: p^(i,i) = p^(i+2^q,i) = 1/2. The push-sum weights w start at 1 and are
 *    set back to 1 after each outer step (all workers then hold the same model). The
 *    gradient (and the L2 term) is taken at the de-biased z = x / w; the exact average of
 *    Algorithm 1 is over x.
 *  - Section 6's variant without the exact average (no_average): each worker keeps its own
 *    outer iterate x_{t,0}^{(i)} and slow momentum u^{(i)} and applies Eq. (2), (3) with its
 *    own x_{t,tau}^{(i)} in place of the average; the buffer policy "average" would need the
 *    communication the variant removes and is rejected. Push-sum weights are left alone.
 *  - 1/gamma_t and alpha*gamma_t are formed once per outer iteration (in binary64,
 *    rounded once to `real`); the worker sum runs in worker order 0..m-1 and is divided
 *    by m.
 */
#include "slowmo_oracle.h"

#include <math.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#if ORACLE_F64
typedef double real;
#define FMA(a, b, c) fma((a), (b), (c))
#define SQRT(a) sqrt(a)
#define RUN_NAME slowmo_oracle_run_f64
#else
typedef float real;
#define FMA(a, b, c) fmaf((a), (b), (c))
#define SQRT(a) sqrtf(a)
#define RUN_NAME slowmo_oracle_run_f32
#endif

/* Stochastic gradient of worker i at coordinate j, step (t,k), evaluated at x. */
static real gradient(const oracle_config *cfg, uint32_t i, uint64_t j, uint32_t t, uint32_t k,
                     real x, real a_j, real c_ij, real G_ij) {
  real g;
  if (cfg->grad_mode == ORACLE_GRAD_GENERATED) {
    /* F_i(x) = 1/2 sum_j a_j (x_j - c_{i,j})^2, gradient a_j (x_j - c_{i,j}), plus sigma z */
    uint64_t key = oracle_stream_key(ORACLE_TAG_GRADNOISE, cfg->seed, t, k, i);
    real z = (real)oracle_stream_normal(key, j);
    real noise = (real)cfg->sigma * z;
    real e = x - c_ij;
    g = FMA(a_j, e, noise);
  } else {
    g = G_ij;
  }
  if (cfg->weight_decay != 0.0f) g = FMA((real)cfg->weight_decay, x, g);
  return g;
}

#if !ORACLE_F64
uint32_t oracle_sgp_hops(uint32_t m, uint64_t s) {
  if (m < 2) return 0;
  uint32_t nq = 0; /* floor(log2(m-1)) + 1 */
  for (uint32_t r = m - 1; r > 0; r >>= 1) nq += 1;
  return 1u << (uint32_t)(s % nq);
}
#endif

static int valid(const oracle_config *c) {
  if (c->m == 0 || c->tau == 0) return 0;
  if (c->base < ORACLE_BASE_NESTEROV || c->base > ORACLE_BASE_SGP_ADAM) return 0;
  if (c->buffer_policy < ORACLE_BUF_RESET || c->buffer_policy > ORACLE_BUF_AVERAGE) return 0;
  if (c->grad_mode < ORACLE_GRAD_GENERATED || c->grad_mode > ORACLE_GRAD_SUPPLIED_ARRAY) return 0;
  if (c->no_average && c->buffer_policy == ORACLE_BUF_AVERAGE) return 0;
  return 1;
}

int RUN_NAME(const oracle_config *cfg, const float *gamma_t, const uint64_t *j_idx, uint64_t j0,
             uint64_t n, const float *G, real *x_out, real *anchor_out, real *u_out, real *h_out,
             real *v_out, double *dbar) {
  if (!cfg || !valid(cfg) || !x_out || !anchor_out || !u_out || !h_out) return -1;
  if (cfg->grad_mode == ORACLE_GRAD_SUPPLIED_ARRAY && !G) return -1;
  const uint32_t m = cfg->m, tau = cfg->tau, T = cfg->T;
  const int adam = cfg->base == ORACLE_BASE_ADAM || cfg->base == ORACLE_BASE_SGP_ADAM;
  const int sgp = cfg->base == ORACLE_BASE_SGP_NESTEROV || cfg->base == ORACLE_BASE_SGP_ADAM;
  const real mu = (real)cfg->mu;
  const real b1 = (real)cfg->adam_b1, b2 = (real)cfg->adam_b2, eps = (real)cfg->adam_eps;
  const real omb1 = (real)(1.0 - (double)cfg->adam_b1); /* 1 - beta_1 */
  const real omb2 = (real)(1.0 - (double)cfg->adam_b2); /* 1 - beta_2 */
  const real alpha = (real)cfg->alpha, beta = (real)cfg->beta;
  (void)alpha;

#pragma omp parallel
  {
    real *x = (real *)malloc(sizeof(real) * m);
    real *h = (real *)malloc(sizeof(real) * m);
    real *v = (real *)malloc(sizeof(real) * m);
    real *c = (real *)malloc(sizeof(real) * m);
    real *Gfix = (real *)malloc(sizeof(real) * m);
    real *w = (real *)malloc(sizeof(real) * m);     /* push-sum weights w^{(i)}      */
    real *x_half = (real *)malloc(sizeof(real) * m); /* x_{k+1/2}^{(i)} of Algorithm 2 */
    real *w_half = (real *)malloc(sizeof(real) * m);
    real *x0_own = (real *)malloc(sizeof(real) * m); /* no_average: x_{t,0}^{(i)} */
    real *u_own = (real *)malloc(sizeof(real) * m);  /* no_average: u^{(i)}       */

#pragma omp for schedule(static)
    for (uint64_t q = 0; q < n; ++q) {
      const uint64_t j = j_idx ? j_idx[q] : j0 + q;

      /* synthetic problem data of this coordinate */
      real a_j = 0;
      for (uint32_t i = 0; i < m; ++i) c[i] = Gfix[i] = 0;
      if (cfg->grad_mode == ORACLE_GRAD_GENERATED) {
        a_j = (real)oracle_curvature(cfg, j);
        for (uint32_t i = 0; i < m; ++i) c[i] = (real)oracle_centre(cfg, i, j);
      } else if (cfg->grad_mode == ORACLE_GRAD_SUPPLIED_HASH) {
        for (uint32_t i = 0; i < m; ++i) Gfix[i] = (real)oracle_supplied_gradient(cfg, i, j);
      }

      /* Algorithm 1, input line: all workers start at x_{0,0}; u_0 = 0; buffers are zero */
      real x0 = (real)cfg->x_init; /* anchor x_{t,0} */
      real u = 0;
      for (uint32_t i = 0; i < m; ++i) {
        x[i] = x0;
        h[i] = 0;
        v[i] = 0;
        w[i] = 1;
        x0_own[i] = x0;
        u_own[i] = 0;
      }
      uint64_t l = 0;            /* Adam steps since the buffers were last zero */
      double pow_b1 = 1.0, pow_b2 = 1.0; /* beta_1^l, beta_2^l */

      for (uint32_t t = 0; t < T; ++t) {
        const double gam_d = (double)(gamma_t ? gamma_t[t] : cfg->gamma);
        const real gam = (real)gam_d;
        const real inv_gam = (real)(1.0 / gam_d);
        const real alpha_gam = (real)((double)cfg->alpha * gam_d);

        for (uint32_t k = 0; k < tau; ++k) {
          l += 1;
          pow_b1 *= (double)cfg->adam_b1;
          pow_b2 *= (double)cfg->adam_b2;
          const real ibc1 = (real)(1.0 / (1.0 - pow_b1)); /* 1 / (1 - beta_1^l) */
          const real ibc2 = (real)(1.0 / (1.0 - pow_b2)); /* 1 / (1 - beta_2^l) */
          double dsum = 0.0;

          for (uint32_t i = 0; i < m; ++i) {
            real G_ij = Gfix[i];
            if (cfg->grad_mode == ORACLE_GRAD_SUPPLIED_ARRAY)
              G_ij = (real)G[(((uint64_t)t * tau + k) * m + i) * n + q];
            /* SGP evaluates the gradient at the de-biased parameters z = x / w */
            const real at = sgp ? x[i] / w[i] : x[i];
            const real g = gradient(cfg, i, j, t, k, at, a_j, c[i], G_ij);
            real d;
            if (!adam) {
              /* Table C.1, SGD row: h <- mu h + g ; d = mu h + g (Nesterov momentum) */
              h[i] = FMA(mu, h[i], g);
              d = FMA(mu, h[i], g);
            } else {
              /* Table C.1, Adam row */
              h[i] = FMA(b1, h[i], omb1 * g);
              v[i] = FMA(b2, v[i], omb2 * (g * g));
              const real h_hat = h[i] * ibc1;
              const real v_hat = v[i] * ibc2;
              d = h_hat / (SQRT(v_hat) + eps);
            }
            /* Algorithm 1, base optimizer step: x_{t,k+1} = x_{t,k} - gamma_t d */
            x[i] = FMA(-gam, d, x[i]);
            dsum += (double)d;
          }
          if (dbar) dbar[((uint64_t)t * tau + k) * n + q] = dsum / (double)m;

          if (sgp && m > 1) {
            /* Algorithm 2: the step above gave x_{k+1/2}; every worker keeps half of
             * (x_{k+1/2}, w) and receives half of its in-neighbour's */
            const uint32_t hops = oracle_sgp_hops(m, (uint64_t)t * tau + k);
            for (uint32_t i = 0; i < m; ++i) {
              x_half[i] = x[i];
              w_half[i] = w[i];
            }
            for (uint32_t i = 0; i < m; ++i) {
              const uint32_t from = (i + m - hops % m) % m; /* the worker that sends to i */
              x[i] = (real)0.5 * x_half[i] + (real)0.5 * x_half[from];
              w[i] = (real)0.5 * w_half[i] + (real)0.5 * w_half[from];
            }
          }
        }

        if (!cfg->no_average) {
          /* Algorithm 1, exact average over the workers */
          real s = x[0];
          for (uint32_t i = 1; i < m; ++i) s = s + x[i];
          const real xbar = s / (real)m;
          /* Eq. (2): u_{t+1} = beta u_t + (x_{t,0} - xbar_{t,tau}) / gamma_t */
          u = FMA(beta, u, (x0 - xbar) * inv_gam);
          /* Eq. (3): x_{t+1,0} = x_{t,0} - alpha gamma_t u_{t+1} */
          x0 = FMA(-alpha_gam, u, x0);
          /* every worker continues from x_{t+1,0} */
          for (uint32_t i = 0; i < m; ++i) {
            x[i] = x0;
            w[i] = 1;
          }
        } else {
          /* Section 6: the same two updates per worker, on its own x_{t,tau}^{(i)} */
          for (uint32_t i = 0; i < m; ++i) {
            u_own[i] = FMA(beta, u_own[i], (x0_own[i] - x[i]) * inv_gam);
            x0_own[i] = FMA(-alpha_gam, u_own[i], x0_own[i]);
            x[i] = x0_own[i];
          }
        }

        /* buffer policy for the next outer iteration */
        if (cfg->buffer_policy == ORACLE_BUF_RESET) {
          for (uint32_t i = 0; i < m; ++i) h[i] = v[i] = 0;
          l = 0;
          pow_b1 = pow_b2 = 1.0;
        } else if (cfg->buffer_policy == ORACLE_BUF_AVERAGE) {
          real sh = h[0], sv = v[0];
          for (uint32_t i = 1; i < m; ++i) {
            sh = sh + h[i];
            sv = sv + v[i];
          }
          const real hbar = sh / (real)m, vbar = sv / (real)m;
          for (uint32_t i = 0; i < m; ++i) {
            h[i] = hbar;
            v[i] = vbar;
          }
        } /* maintain: nothing */
      }

      for (uint32_t i = 0; i < m; ++i) {
        x_out[(uint64_t)i * n + q] = x[i];
        h_out[(uint64_t)i * n + q] = h[i];
        if (v_out) v_out[(uint64_t)i * n + q] = v[i];
      }
      if (!cfg->no_average) {
        anchor_out[q] = x0;
        u_out[q] = u;
      } else {
        for (uint32_t i = 0; i < m; ++i) {
          anchor_out[(uint64_t)i * n + q] = x0_own[i];
          u_out[(uint64_t)i * n + q] = u_own[i];
        }
      }
    }
    free(x);
    free(h);
    free(v);
    free(c);
    free(Gfix);
    free(w);
    free(x_half);
    free(w_half);
    free(x0_own);
    free(u_own);
  }
  return 0;
}

#if !ORACLE_F64
int slowmo_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
#endif
