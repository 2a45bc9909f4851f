// Host side of libslowmo: argument checking, the state machine of Algorithm 1 (outer
// iteration t, inner step k, Adam count l) and kernel launches. See include/slowmo.h for
// the contract of every entry point.
#include "../../include/slowmo.h"

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "kernels.cuh"
#include "outer_fused.cuh"
#include "outer_sharded.cuh"
#include "outer_staged.cuh"
#include "sgp_step.cuh"

using namespace slowmo;

struct slowmo_ctx {
  slowmo_config cfg;
  slowmo_buffers buf;
  cudaStream_t stream;
  uint32_t nvec;             // 4-element column groups per row: ceil(P/4)
  uint32_t win_vec0, win_nvec;  // column window that launches cover (whole vector except inside slowmo_iteration_host)
  cudaStream_t copy_in, copy_out;  // created on first use by slowmo_iteration_host
  uint64_t t;                // outer iteration
  uint32_t k;                // inner steps taken in this outer iteration
  uint64_t l;                // Adam steps since the buffers were last zero
  double pow_b1, pow_b2;     // beta_1^l, beta_2^l
  float gamma;               // gamma_t in force
  std::vector<uint64_t> tensor_offsets;  // n_tensors + 1 prefix sums, or empty
  int outer_variant;
  int local_variant;         // SLOWMO_VARIANT_DEFAULT, SLOWMO_LOCAL_ROW_TILES or SLOWMO_LOCAL_COLUMN_OWNER
  int virt;                  // lazy variant: 0, or how the next local step must read the (virtual) replicas
  bool pending_last;         // fused variant: the last inner step waits to run inside the outer step
  LocalArgs pending;         // its arguments (counters k, l already include it)
  int *status_dev;           // device status block: [0] = timeout flag, [1] = where
  int cuda_error;
  int num_sms;
};

namespace {

// NVTX range around a library call, visible on a profiler's timeline; a no-op costing two
// indirect calls when no tool is attached.
struct TraceRange {
  explicit TraceRange(const char *name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange &) = delete;
  TraceRange &operator=(const TraceRange &) = delete;
};

bool is_adam(int base) { return base == SLOWMO_BASE_ADAM || base == SLOWMO_BASE_SGP_ADAM; }
bool is_sgp(int base) { return base == SLOWMO_BASE_SGP_NESTEROV || base == SLOWMO_BASE_SGP_ADAM; }
bool finite_pos(float v) { return std::isfinite(v) && v > 0.0f; }
bool unit_interval(float v) { return std::isfinite(v) && v >= 0.0f && v < 1.0f; }
bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(slowmo_ctx *ctx, cudaError_t e) {
  if (e == cudaSuccess) return SLOWMO_OK;
  if (ctx && ctx->cuda_error == 0) ctx->cuda_error = (int)e;
  return SLOWMO_ECUDA;
}

int check_launch(slowmo_ctx *ctx) { return cuda_fail(ctx, cudaGetLastError()); }

// Grid of the creation-time fills: blockIdx.x strides over the columns, blockIdx.y over the rows
// (at most 65535 of them at a time, the grid's limit), enough blocks to cover the machine a few times.
dim3 fill_grid(const slowmo_ctx *ctx, uint32_t rows) {
  const uint32_t grid_rows = rows < 65535u ? rows : 65535u;
  uint64_t want = (uint64_t)ctx->num_sms * 16;
  uint64_t per_row = (want + grid_rows - 1) / grid_rows;
  uint64_t need = ((uint64_t)ctx->nvec + kThreads - 1) / kThreads;
  if (per_row > need) per_row = need;
  if (per_row < 1) per_row = 1;
  return dim3((uint32_t)per_row, grid_rows);
}

// Layout of the local step (both compute every element with the same base_step).
bool use_column_owner(const slowmo_ctx *ctx) {
  if (ctx->local_variant == SLOWMO_LOCAL_ROW_TILES) return false;
  if (ctx->local_variant == SLOWMO_LOCAL_COLUMN_OWNER) return true;
  if (SLOWMO_LOCAL_LAYOUT == 1) return false;
  if (SLOWMO_LOCAL_LAYOUT == 2) return true;
  // measured on B200: with a generated gradient the column owner wins (the curvature is read
  // once per column: +3-4 % at m = 8 and m = 32); with a supplied gradient the two are equal
  return ctx->cfg.grad_mode == SLOWMO_GRAD_GENERATED;
}

#ifndef SLOWMO_VIRT_ROWS_DIV
#define SLOWMO_VIRT_ROWS_DIV 2   // the virtual-replica form keeps ROWS / this many rows in flight
#endif
template <int BASE, int GRAD, bool DERIVE>
void launch_local_cols(slowmo_ctx *ctx, const LocalArgs &A) {
  constexpr int ROWS = BASE == 1 ? SLOWMO_LOCAL_COL_ROWS / 2 : SLOWMO_LOCAL_COL_ROWS;
  const uint32_t blocks = (A.nvec + kThreads - 1) / kThreads;
  if (A.virt)
    local_step_cols_kernel<BASE, GRAD, (SLOWMO_VIRT_ROWS_DIV > 1 && ROWS > 1) ? ROWS / SLOWMO_VIRT_ROWS_DIV : ROWS, true, DERIVE>
        <<<blocks, kThreads, 0, ctx->stream>>>(A);
  else
    local_step_cols_kernel<BASE, GRAD, ROWS, false, DERIVE><<<blocks, kThreads, 0, ctx->stream>>>(A);
}

template <int BASE, int GRAD>
void launch_local(slowmo_ctx *ctx, const LocalArgs &A) {
  // the first step after a lazy outer step must be the column owner: only it can read virtual replicas
  if (A.virt || use_column_owner(ctx)) {
    // the row keys travel in the arguments up to kInlineKeys workers and are derived in the kernel beyond
    if (GRAD == 0 && A.m > kInlineKeys) launch_local_cols<BASE, GRAD, GRAD == 0>(ctx, A);
    else launch_local_cols<BASE, GRAD, false>(ctx, A);
    return;
  }
  const uint32_t per_tile = kThreads * kLocalUnroll;
  const uint32_t tiles = (A.nvec + per_tile - 1) / per_tile;
  local_step_kernel<BASE, GRAD, kLocalUnroll><<<tiles * ctx->cfg.m, kThreads, 0, ctx->stream>>>(A);
}

template <int NBUF>
void launch_outer_direct(slowmo_ctx *ctx, const OuterArgs &A) {
  const uint32_t blocks = (A.nvec + kThreads - 1) / kThreads;
  switch (ctx->cfg.buffer_policy) {
    case SLOWMO_BUF_RESET: outer_step_direct_kernel<NBUF, 0><<<blocks, kThreads, 0, ctx->stream>>>(A); break;
    case SLOWMO_BUF_MAINTAIN: outer_step_direct_kernel<NBUF, 1><<<blocks, kThreads, 0, ctx->stream>>>(A); break;
    default: outer_step_direct_kernel<NBUF, 2><<<blocks, kThreads, 0, ctx->stream>>>(A); break;
  }
}

void launch_local_any(slowmo_ctx *ctx, const LocalArgs &A) {
  const bool generated = ctx->cfg.grad_mode == SLOWMO_GRAD_GENERATED;
  if (is_sgp(ctx->cfg.base)) {
    // Algorithm 2: the graph's hop distance follows the global step count t*tau + k
    launch_sgp_step(A, sgp_hops(A.m, A.t * ctx->cfg.tau + A.k), is_adam(ctx->cfg.base), generated, ctx->stream);
  } else if (ctx->cfg.base == SLOWMO_BASE_NESTEROV) {
    if (generated) launch_local<0, 0>(ctx, A); else launch_local<0, 1>(ctx, A);
  } else {
    if (generated) launch_local<1, 0>(ctx, A); else launch_local<1, 1>(ctx, A);
  }
}

// Fused variant: run the deferred last inner step on its own (state is about to be read or
// written from outside).
int flush_pending(slowmo_ctx *ctx) {
  if (ctx->pending_last) {
    ctx->pending_last = false;
    launch_local_any(ctx, ctx->pending);
    if (int rc = check_launch(ctx)) return rc;
  }
  if (ctx->virt) {
    // lazy variant: write out the virtual replicas and buffers
    const uint32_t blocks = (ctx->nvec + kThreads - 1) / kThreads;
    const slowmo_buffers &b = ctx->buf;
    if (is_adam(ctx->cfg.base))
      materialize_kernel<2><<<blocks, kThreads, 0, ctx->stream>>>(b.x, b.h, b.v, b.anchor, b.pitch, ctx->nvec, ctx->cfg.m, ctx->virt);
    else
      materialize_kernel<1><<<blocks, kThreads, 0, ctx->stream>>>(b.x, b.h, b.v, b.anchor, b.pitch, ctx->nvec, ctx->cfg.m, ctx->virt);
    ctx->virt = 0;
    return check_launch(ctx);
  }
  return SLOWMO_OK;
}

// Resolve a tensor id to (base pointer, rows); NULL if the tensor does not exist here.
float *tensor_base(slowmo_ctx *ctx, int which, uint32_t *rows) {
  const slowmo_buffers &b = ctx->buf;
  const uint32_t outer_rows = ctx->cfg.no_average ? ctx->cfg.m : 1;  // per-worker anchor and u without the average
  switch (which) {
    case SLOWMO_T_X: *rows = ctx->cfg.m; return b.x;
    case SLOWMO_T_ANCHOR: *rows = outer_rows; return b.anchor;
    case SLOWMO_T_U: *rows = outer_rows; return b.u;
    case SLOWMO_T_H: *rows = ctx->cfg.m; return b.h;
    case SLOWMO_T_V: *rows = ctx->cfg.m; return b.v;
    case SLOWMO_T_A: *rows = 1; return b.a;
    case SLOWMO_T_C: *rows = ctx->cfg.m; return b.c;
    default: *rows = 0; return nullptr;
  }
}

int copy_params(slowmo_ctx *ctx, int which, int32_t replica, uint64_t offset, uint64_t count, float *user,
                int user_on_device, bool to_user) {
  if (!ctx || !user) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  uint32_t rows = 0;
  float *base = tensor_base(ctx, which, &rows);
  if (!base) return SLOWMO_EINVAL;
  if (replica < -1 || (replica >= 0 && (uint32_t)replica >= rows)) return SLOWMO_EINVAL;
  if (offset > ctx->cfg.P || count > ctx->cfg.P - offset) return SLOWMO_EINVAL;
  if (count == 0) return SLOWMO_OK;
  if (int rc = flush_pending(ctx)) return rc;
  const uint32_t nrows = replica < 0 ? rows : 1;
  float *dev = base + (replica < 0 ? 0 : (uint64_t)replica * ctx->buf.pitch) + offset;
  const size_t width = count * sizeof(float), dpitch = ctx->buf.pitch * sizeof(float);
  cudaError_t e;
  if (to_user) {
    e = cudaMemcpy2DAsync(user, width, dev, dpitch, width, nrows,
                          user_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, ctx->stream);
  } else {
    e = cudaMemcpy2DAsync(dev, dpitch, user, width, width, nrows,
                          user_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, ctx->stream);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (!user_on_device) return cuda_fail(ctx, cudaStreamSynchronize(ctx->stream));
  return SLOWMO_OK;
}

}  // namespace

extern "C" {

int slowmo_create(const slowmo_config *cfg, const slowmo_buffers *buf, void *cuda_stream, slowmo_ctx **out) {
  if (!cfg || !buf || !out) return SLOWMO_EINVAL;
  *out = nullptr;
  const bool adam = is_adam(cfg->base);
  const bool generated = cfg->grad_mode == SLOWMO_GRAD_GENERATED;
  if (cfg->P == 0 || cfg->m == 0 || cfg->tau == 0) return SLOWMO_EINVAL;
  if (cfg->base < SLOWMO_BASE_NESTEROV || cfg->base > SLOWMO_BASE_SGP_ADAM) return SLOWMO_EINVAL;
  if (cfg->no_average != 0 && cfg->no_average != 1) return SLOWMO_EINVAL;
  if (cfg->no_average && cfg->buffer_policy == SLOWMO_BUF_AVERAGE) return SLOWMO_EINVAL;
  if (cfg->P > SLOWMO_MAX_P) return SLOWMO_EINVAL;  // 4-column groups are indexed with 32 bits
  if (!finite_pos(cfg->alpha) || !unit_interval(cfg->beta) || !finite_pos(cfg->gamma)) return SLOWMO_EINVAL;
  if (cfg->buffer_policy < SLOWMO_BUF_RESET || cfg->buffer_policy > SLOWMO_BUF_AVERAGE) return SLOWMO_EINVAL;
  if (!generated && cfg->grad_mode != SLOWMO_GRAD_SUPPLIED) return SLOWMO_EINVAL;
  if (!std::isfinite(cfg->weight_decay) || cfg->weight_decay < 0.0f || !std::isfinite(cfg->x_init)) return SLOWMO_EINVAL;
  if (!adam && !unit_interval(cfg->mu)) return SLOWMO_EINVAL;
  if (adam && (!unit_interval(cfg->adam_b1) || !unit_interval(cfg->adam_b2) || !finite_pos(cfg->adam_eps)))
    return SLOWMO_EINVAL;
  if (!std::isfinite(cfg->sigma) || cfg->sigma < 0.0f) return SLOWMO_EINVAL;
  if (generated && (!std::isfinite(cfg->a_lo) || !std::isfinite(cfg->a_hi) || cfg->a_hi < cfg->a_lo ||
                    !std::isfinite(cfg->c_std) || cfg->c_std < 0.0f))
    return SLOWMO_EINVAL;
  if (!buf->x || !buf->h || !buf->anchor || !buf->u) return SLOWMO_EINVAL;
  if (adam && !buf->v) return SLOWMO_EINVAL;
  if (generated && (!buf->a || !buf->c)) return SLOWMO_EINVAL;
  if ((cfg->n_tensors != 0) != (cfg->tensor_sizes != nullptr)) return SLOWMO_EINVAL;
  if (buf->pitch % 4 != 0) return SLOWMO_EALIGN;
  if (buf->pitch < cfg->P) return SLOWMO_EINVAL;
  const void *ptrs[] = {buf->x, buf->h, buf->v, buf->anchor, buf->u, buf->a, buf->c};
  for (const void *p : ptrs)
    if (p && !aligned16(p)) return SLOWMO_EALIGN;
  const uint64_t nvec = (cfg->P + 3) / 4;
  const uint64_t per_tile = (uint64_t)kThreads * kLocalUnroll;
  if (((nvec + per_tile - 1) / per_tile) * cfg->m >= (1ull << 31)) return SLOWMO_EINVAL;  // grid limit

  slowmo_ctx *ctx = new (std::nothrow) slowmo_ctx();
  if (!ctx) return SLOWMO_ENOMEM;
  ctx->cfg = *cfg;
  ctx->cfg.tensor_sizes = nullptr;
  ctx->buf = *buf;
  ctx->stream = (cudaStream_t)cuda_stream;
  ctx->nvec = (uint32_t)nvec;
  ctx->win_vec0 = 0;
  ctx->win_nvec = (uint32_t)nvec;
  ctx->copy_in = ctx->copy_out = nullptr;
  ctx->t = 0;
  ctx->k = 0;
  ctx->l = 0;
  ctx->pow_b1 = ctx->pow_b2 = 1.0;
  ctx->gamma = cfg->gamma;
  ctx->outer_variant = SLOWMO_VARIANT_DEFAULT;
  ctx->local_variant = SLOWMO_VARIANT_DEFAULT;
  ctx->virt = 0;
  ctx->pending_last = false;
  ctx->status_dev = nullptr;
  ctx->cuda_error = 0;
  if (cfg->n_tensors) {
    try {
      ctx->tensor_offsets.resize((size_t)cfg->n_tensors + 1);
    } catch (...) {
      delete ctx;
      return SLOWMO_ENOMEM;
    }
    uint64_t acc = 0;
    for (uint32_t i = 0; i < cfg->n_tensors; ++i) {
      ctx->tensor_offsets[i] = acc;
      if (cfg->tensor_sizes[i] == 0 || cfg->tensor_sizes[i] > cfg->P - acc) {
        delete ctx;
        return SLOWMO_EINVAL;
      }
      acc += cfg->tensor_sizes[i];
    }
    ctx->tensor_offsets[cfg->n_tensors] = acc;
    if (acc != cfg->P) {
      delete ctx;
      return SLOWMO_EINVAL;
    }
  }

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->status_dev, 4 * sizeof(int));
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status_dev, 0, 4 * sizeof(int), ctx->stream);
  if (e == cudaSuccess) e = outer_staged_configure();
  if (e != cudaSuccess) {
    if (ctx->status_dev) cudaFree(ctx->status_dev);
    delete ctx;
    return SLOWMO_ECUDA;
  }

  // Algorithm 1, input line: x^{(i)} = x_{0,0}, u_0 = 0, buffers zero; synthetic problem data.
  const uint32_t m = cfg->m;
  const size_t row_bytes = (size_t)ctx->nvec * 4 * sizeof(float);
  const size_t pitch_bytes = buf->pitch * sizeof(float);
  fill_value_rows_kernel<<<fill_grid(ctx, m), kThreads, 0, ctx->stream>>>(buf->x, buf->pitch, ctx->nvec, m, cfg->x_init);
  const uint32_t outer_rows = cfg->no_average ? m : 1;
  fill_value_rows_kernel<<<fill_grid(ctx, outer_rows), kThreads, 0, ctx->stream>>>(buf->anchor, buf->pitch, ctx->nvec,
                                                                                   outer_rows, cfg->x_init);
  e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaMemset2DAsync(buf->u, pitch_bytes, 0, row_bytes, outer_rows, ctx->stream);
  if (e == cudaSuccess) e = cudaMemset2DAsync(buf->h, pitch_bytes, 0, row_bytes, m, ctx->stream);
  if (e == cudaSuccess && buf->v) e = cudaMemset2DAsync(buf->v, pitch_bytes, 0, row_bytes, m, ctx->stream);
  if (e == cudaSuccess && generated) {
    fill_curvature_kernel<<<fill_grid(ctx, 1).x, kThreads, 0, ctx->stream>>>(buf->a, ctx->nvec, cfg->seed, cfg->a_lo, cfg->a_hi);
    fill_normal_rows_kernel<<<fill_grid(ctx, m), kThreads, 0, ctx->stream>>>(buf->c, buf->pitch, ctx->nvec, m, kTagCentre,
                                                                             cfg->seed, cfg->c_std, cfg->worker_offset);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    cudaFree(ctx->status_dev);
    delete ctx;
    return SLOWMO_ECUDA;
  }
  *out = ctx;
  return SLOWMO_OK;
}

int slowmo_destroy(slowmo_ctx *ctx) {
  if (!ctx) return SLOWMO_EINVAL;
  flush_pending(ctx);
  cudaStreamSynchronize(ctx->stream);
  if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
  if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
  if (ctx->status_dev) cudaFree(ctx->status_dev);
  delete ctx;
  return SLOWMO_OK;
}

int slowmo_local_steps(slowmo_ctx *ctx, uint32_t n, const float *grad) {
  TraceRange trace("slowmo_local_steps");
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  const slowmo_config &c = ctx->cfg;
  const bool generated = c.grad_mode == SLOWMO_GRAD_GENERATED;
  if (generated ? grad != nullptr : grad == nullptr) return SLOWMO_EINVAL;
  if (grad && !aligned16(grad)) return SLOWMO_EALIGN;
  if ((uint64_t)ctx->k + n > c.tau) return SLOWMO_ESTATE;

  const uint64_t woff = 4ull * ctx->win_vec0;  // first column of the window
  LocalArgs A;
  A.x = ctx->buf.x + woff;
  A.h = ctx->buf.h + woff;
  A.v = ctx->buf.v ? ctx->buf.v + woff : nullptr;
  A.src = (generated ? ctx->buf.c : grad) + woff;
  A.a = ctx->buf.a ? ctx->buf.a + woff : nullptr;
  A.anchor = ctx->buf.anchor + woff;
  A.virt = 0;
  A.pitch = ctx->buf.pitch;
  A.nvec = ctx->win_nvec;
  A.vec0 = ctx->win_vec0;
  A.m = c.m;
  A.worker0 = c.worker_offset;
  A.seed = c.seed;
  A.neg_gamma = -ctx->gamma;
  A.mu = c.mu;
  A.wd = c.weight_decay;
  A.sigma = c.sigma;
  A.b1 = c.adam_b1;
  A.b2 = c.adam_b2;
  A.omb1 = (float)(1.0 - (double)c.adam_b1);
  A.omb2 = (float)(1.0 - (double)c.adam_b2);
  A.eps = c.adam_eps;

  for (uint32_t s = 0; s < n; ++s) {
    // Table C.1: bias corrections use the 1-based count l of Adam steps since the buffers were zero
    ctx->l += 1;
    ctx->pow_b1 *= (double)c.adam_b1;
    ctx->pow_b2 *= (double)c.adam_b2;
    A.ibc1 = (float)(1.0 / (1.0 - ctx->pow_b1));
    A.ibc2 = (float)(1.0 / (1.0 - ctx->pow_b2));
    A.t = ctx->t;
    A.k = ctx->k;
    if (generated && c.m <= kInlineKeys)
      for (uint32_t i = 0; i < c.m; ++i)
        A.keys[i] = stream_key(kTagGradNoise, c.seed, ctx->t, ctx->k, c.worker_offset + i);
    // lazy variant: the first step of an outer iteration reads the anchor in place of the rows
    A.virt = ctx->virt;
    ctx->virt = 0;
    ctx->k += 1;
    // fused and lazy variants: step tau-1 is taken inside the outer-step kernel
    if ((ctx->outer_variant == SLOWMO_OUTER_FUSED || ctx->outer_variant == SLOWMO_OUTER_LAZY) && ctx->k == c.tau &&
        !is_sgp(c.base) && !c.no_average && A.virt == 0) {
      ctx->pending = A;
      ctx->pending_last = true;
      break;
    }
    launch_local_any(ctx, A);
    int rc = check_launch(ctx);
    if (rc != SLOWMO_OK) return rc;
  }
  return SLOWMO_OK;
}

int slowmo_outer_step(slowmo_ctx *ctx) {
  TraceRange trace("slowmo_outer_step");
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  const slowmo_config &c = ctx->cfg;
  if (ctx->k != c.tau) return SLOWMO_ESTATE;

  const uint64_t woff = 4ull * ctx->win_vec0;
  OuterArgs A;
  A.x = ctx->buf.x + woff;
  A.h = ctx->buf.h + woff;
  A.v = ctx->buf.v ? ctx->buf.v + woff : nullptr;
  A.anchor = ctx->buf.anchor + woff;
  A.u = ctx->buf.u + woff;
  A.pitch = ctx->buf.pitch;
  A.nvec = ctx->win_nvec;
  A.m = c.m;
  A.beta = c.beta;
  A.inv_gamma = (float)(1.0 / (double)ctx->gamma);
  A.neg_alpha_gamma = -(float)((double)c.alpha * (double)ctx->gamma);
  A.m_float = (float)c.m;
  const int nbuf = is_adam(c.base) ? 2 : 1;

  int variant = ctx->outer_variant;
  if (variant == SLOWMO_VARIANT_DEFAULT) variant = SLOWMO_OUTER_DIRECT;
  if ((ctx->pending_last && variant != SLOWMO_OUTER_FUSED && variant != SLOWMO_OUTER_LAZY) || ctx->virt) {
    if (int rc = flush_pending(ctx)) return rc;
  }
  if (c.no_average) {
    const uint32_t per_tile = kThreads * kLocalUnroll;
    const uint32_t blocks = ((A.nvec + per_tile - 1) / per_tile) * c.m;
    const bool reset = c.buffer_policy == SLOWMO_BUF_RESET;
    if (nbuf == 1) {
      if (reset) outer_step_noaverage_kernel<1, 0, kLocalUnroll><<<blocks, kThreads, 0, ctx->stream>>>(A);
      else outer_step_noaverage_kernel<1, 1, kLocalUnroll><<<blocks, kThreads, 0, ctx->stream>>>(A);
    } else {
      if (reset) outer_step_noaverage_kernel<2, 0, kLocalUnroll><<<blocks, kThreads, 0, ctx->stream>>>(A);
      else outer_step_noaverage_kernel<2, 1, kLocalUnroll><<<blocks, kThreads, 0, ctx->stream>>>(A);
    }
  } else if (ctx->pending_last) {
    ctx->pending_last = false;
    // lazy: leave broadcast and buffer policy to the next local step (needs tau >= 2, so that this
    // next step is not itself a deferred one)
    const bool lazy = variant == SLOWMO_OUTER_LAZY && c.tau >= 2;
    launch_last_step_outer(ctx->pending, A, c.base == SLOWMO_BASE_ADAM, c.grad_mode == SLOWMO_GRAD_GENERATED,
                           c.buffer_policy, lazy, ctx->stream);
    if (lazy) ctx->virt = c.buffer_policy == SLOWMO_BUF_MAINTAIN ? 1 : (c.buffer_policy == SLOWMO_BUF_RESET ? 2 : 3);
  } else if (variant == SLOWMO_OUTER_STAGED) {
    launch_outer_staged(A, nbuf, c.buffer_policy, ctx->num_sms, ctx->status_dev, ctx->stream);
  } else {
    if (nbuf == 1) launch_outer_direct<1>(ctx, A); else launch_outer_direct<2>(ctx, A);
  }
  int rc = check_launch(ctx);
  if (rc != SLOWMO_OK) return rc;

  ctx->t += 1;
  ctx->k = 0;
  if (c.buffer_policy == SLOWMO_BUF_RESET) {
    ctx->l = 0;
    ctx->pow_b1 = ctx->pow_b2 = 1.0;
  }
  return SLOWMO_OK;
}

}  // extern "C"

namespace {

// One whole outer iteration with host input and output, pipelined over column windows. The
// per-worker input `in_host` [m, P] goes to the device tensor `in_dev` [m, pitch] (the centres c in
// generated mode, a gradient buffer in supplied mode) window by window; `grad` is what the local
// steps are given (NULL in generated mode, in_dev in supplied mode).
int iteration_host(slowmo_ctx *ctx, const float *in_host, float *in_dev, const float *grad, float *anchor_host,
                   uint32_t chunks) {
  TraceRange trace("slowmo_iteration_host");
  if (!ctx || !in_host || !in_dev || !anchor_host || chunks == 0 || chunks > 1024) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  const slowmo_config &c = ctx->cfg;
  if (ctx->k != 0 || ctx->pending_last) return SLOWMO_ESTATE;
  cudaError_t e = cudaSuccess;
  if (!ctx->copy_in) e = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking);
  if (e == cudaSuccess && !ctx->copy_out) e = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking);
  if (e != cudaSuccess) return cuda_fail(ctx, e);

  // windows of whole 2048-column tiles so that every window start keeps the 16-byte (and tile) alignment
  uint32_t win = (ctx->nvec + chunks - 1) / chunks;
  win = (win + 511u) / 512u * 512u;
  const uint32_t nwin = (ctx->nvec + win - 1) / win;
  const uint32_t outer_rows = c.no_average ? c.m : 1;
  const size_t dpitch = ctx->buf.pitch * sizeof(float), hpitch = (size_t)c.P * sizeof(float);
  std::vector<cudaEvent_t> ev(2 * (size_t)nwin + 1, nullptr);
  for (auto &x : ev)
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&x, cudaEventDisableTiming);
  int rc = SLOWMO_OK;
  // uploads must not overtake earlier work of this context that still reads the input tensor
  if (e == cudaSuccess) e = cudaEventRecord(ev[2 * nwin], ctx->stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_in, ev[2 * nwin], 0);

  const uint64_t t0 = ctx->t, l0 = ctx->l;
  const double p1 = ctx->pow_b1, p2 = ctx->pow_b2;
  const int virt0 = ctx->virt;
  for (uint32_t w = 0; w < nwin && e == cudaSuccess && rc == SLOWMO_OK; ++w) {
    const uint32_t vec0 = w * win, nv = ctx->nvec - vec0 < win ? ctx->nvec - vec0 : win;
    const uint64_t col0 = 4ull * vec0;
    const uint64_t cols = c.P - col0 < 4ull * nv ? c.P - col0 : 4ull * nv;  // host arrays have no padding
    e = cudaMemcpy2DAsync(in_dev + col0, dpitch, in_host + col0, hpitch, cols * sizeof(float), c.m,
                          cudaMemcpyHostToDevice, ctx->copy_in);
    if (e == cudaSuccess) e = cudaEventRecord(ev[2 * w], ctx->copy_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->stream, ev[2 * w], 0);
    if (e != cudaSuccess) break;
    // the whole outer iteration on this window; every window sees the same counters
    ctx->t = t0;
    ctx->k = 0;
    ctx->l = l0;
    ctx->pow_b1 = p1;
    ctx->pow_b2 = p2;
    ctx->virt = virt0;
    ctx->win_vec0 = vec0;
    ctx->win_nvec = nv;
    rc = slowmo_local_steps(ctx, c.tau, grad);
    if (rc == SLOWMO_OK) rc = slowmo_outer_step(ctx);
    if (rc != SLOWMO_OK) break;
    e = cudaEventRecord(ev[2 * w + 1], ctx->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_out, ev[2 * w + 1], 0);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync(anchor_host + col0, hpitch, ctx->buf.anchor + col0, dpitch, cols * sizeof(float), outer_rows,
                            cudaMemcpyDeviceToHost, ctx->copy_out);
  }
  ctx->win_vec0 = 0;
  ctx->win_nvec = ctx->nvec;
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->copy_out);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  for (auto x : ev)
    if (x) cudaEventDestroy(x);
  if (rc != SLOWMO_OK) return rc;
  return cuda_fail(ctx, e);
}

}  // namespace

extern "C" {

int slowmo_iteration_host(slowmo_ctx *ctx, const float *c_host, float *anchor_host, uint32_t chunks) {
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cfg.grad_mode != SLOWMO_GRAD_GENERATED) return SLOWMO_ENOTIMPL;
  return iteration_host(ctx, c_host, ctx->buf.c, nullptr, anchor_host, chunks);
}

int slowmo_iteration_host_supplied(slowmo_ctx *ctx, const float *grad_host, float *grad_dev, float *anchor_host,
                                   uint32_t chunks) {
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cfg.grad_mode != SLOWMO_GRAD_SUPPLIED) return SLOWMO_ENOTIMPL;
  if (grad_dev && !aligned16(grad_dev)) return SLOWMO_EALIGN;
  return iteration_host(ctx, grad_host, grad_dev, grad_dev, anchor_host, chunks);
}

int slowmo_outer_step_external(slowmo_ctx *ctx) {
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  if (ctx->k != ctx->cfg.tau) return SLOWMO_ESTATE;
  if (int rc = flush_pending(ctx)) return rc;  // a deferred last step must have run before the rows are used
  ctx->t += 1;
  ctx->k = 0;
  if (ctx->cfg.buffer_policy == SLOWMO_BUF_RESET) {
    ctx->l = 0;
    ctx->pow_b1 = ctx->pow_b2 = 1.0;
  }
  return SLOWMO_OK;
}

int slowmo_outer_step_sharded(const slowmo_shard_args *a, void *cuda_stream) {
  TraceRange trace("slowmo_outer_step_sharded");
  if (!a) return SLOWMO_EINVAL;
  const bool adam = a->base == SLOWMO_BASE_ADAM || a->base == SLOWMO_BASE_SGP_ADAM;
  if (a->base < SLOWMO_BASE_NESTEROV || a->base > SLOWMO_BASE_SGP_ADAM) return SLOWMO_EINVAL;
  if (a->buffer_policy < SLOWMO_BUF_RESET || a->buffer_policy > SLOWMO_BUF_AVERAGE) return SLOWMO_EINVAL;
  if (a->world == 0 || a->world > kMaxShardGpus || a->rank >= a->world || a->m_local == 0) return SLOWMO_EINVAL;
  if (a->P == 0 || a->P > SLOWMO_MAX_P || a->pitch < a->P) return SLOWMO_EINVAL;
  if (a->pitch % 4 != 0) return SLOWMO_EALIGN;
  if (!finite_pos(a->alpha) || !unit_interval(a->beta) || !finite_pos(a->gamma_t)) return SLOWMO_EINVAL;
  if (!a->x || !a->h || !a->anchor || !a->u || (adam && !a->v)) return SLOWMO_EINVAL;
  ShardArgs A;
  for (uint32_t r = 0; r < a->world; ++r) {
    A.x[r] = a->x[r];
    A.h[r] = a->h[r];
    A.v[r] = adam ? a->v[r] : nullptr;
    A.anchor[r] = a->anchor[r];
    A.u[r] = a->u[r];
    const void *ptrs[] = {A.x[r], A.h[r], A.anchor[r], A.u[r]};
    for (const void *p : ptrs) {
      if (!p) return SLOWMO_EINVAL;
      if (!aligned16(p)) return SLOWMO_EALIGN;
    }
    if (adam && (!A.v[r] || !aligned16(A.v[r]))) return A.v[r] ? SLOWMO_EALIGN : SLOWMO_EINVAL;
  }
  A.pitch = a->pitch;
  A.world = a->world;
  A.rank = a->rank;
  A.m_local = a->m_local;
  shard_slice((uint32_t)((a->P + 3) / 4), a->world, a->rank, &A.vec_begin, &A.vec_end);
  A.beta = a->beta;
  A.inv_gamma = (float)(1.0 / (double)a->gamma_t);
  A.neg_alpha_gamma = -(float)((double)a->alpha * (double)a->gamma_t);
  A.m_float = (float)((uint64_t)a->world * a->m_local);
  launch_outer_sharded(A, adam ? 2 : 1, a->buffer_policy, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? SLOWMO_OK : SLOWMO_ECUDA;
}

int slowmo_materialize(slowmo_ctx *ctx) {
  TraceRange trace("slowmo_materialize");
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  return flush_pending(ctx);
}

int slowmo_set_gamma(slowmo_ctx *ctx, float gamma_t) {
  if (!ctx || !finite_pos(gamma_t)) return SLOWMO_EINVAL;
  if (ctx->k != 0) return SLOWMO_ESTATE;
  ctx->gamma = gamma_t;
  return SLOWMO_OK;
}

int slowmo_get_params(slowmo_ctx *ctx, int which, int32_t replica, uint64_t offset, uint64_t count, float *dst,
                      int dst_on_device) {
  return copy_params(ctx, which, replica, offset, count, dst, dst_on_device, true);
}

int slowmo_set_params(slowmo_ctx *ctx, int which, int32_t replica, uint64_t offset, uint64_t count,
                      const float *src, int src_on_device) {
  return copy_params(ctx, which, replica, offset, count, const_cast<float *>(src), src_on_device, false);
}

int slowmo_get_counters(slowmo_ctx *ctx, uint64_t *t, uint32_t *k, uint64_t *l) {
  if (!ctx) return SLOWMO_EINVAL;
  if (t) *t = ctx->t;
  if (k) *k = ctx->k;
  if (l) *l = ctx->l;
  return SLOWMO_OK;
}

int slowmo_get_state(slowmo_ctx *ctx, slowmo_state *out) {
  if (!ctx || !out) return SLOWMO_EINVAL;
  out->t = ctx->t;
  out->l = ctx->l;
  out->k = ctx->k;
  out->gamma_t = ctx->gamma;
  return SLOWMO_OK;
}

int slowmo_set_state(slowmo_ctx *ctx, const slowmo_state *in) {
  if (!ctx || !in) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  const slowmo_config &c = ctx->cfg;
  if (in->k > c.tau || !finite_pos(in->gamma_t) || in->l < in->k) return SLOWMO_EINVAL;
  // Table C.1's caption: with buffers zeroed at every outer step the count restarts there, l = k
  if (c.buffer_policy == SLOWMO_BUF_RESET && in->l != in->k) return SLOWMO_EINVAL;
  // what the context still owes the tensors (a deferred last step, virtual replicas) belongs to the
  // position being left: write it out before the counters change
  if (int rc = flush_pending(ctx)) return rc;
  ctx->t = in->t;
  ctx->k = in->k;
  ctx->l = in->l;
  ctx->gamma = in->gamma_t;
  // beta^l exactly as the step loop forms it: l successive binary64 multiplications (a power that
  // has underflowed to zero stays zero, so the loop can stop there)
  double p1 = 1.0, p2 = 1.0;
  for (uint64_t s = 0; s < in->l && (p1 != 0.0 || p2 != 0.0); ++s) {
    p1 *= (double)c.adam_b1;
    p2 *= (double)c.adam_b2;
  }
  ctx->pow_b1 = p1;
  ctx->pow_b2 = p2;
  return SLOWMO_OK;
}

int slowmo_fill_gradient(slowmo_ctx *ctx, float *grad) {
  if (!ctx || !grad) return SLOWMO_EINVAL;
  if (!aligned16(grad)) return SLOWMO_EALIGN;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  const uint32_t m = ctx->cfg.m;
  fill_normal_rows_kernel<<<fill_grid(ctx, m), kThreads, 0, ctx->stream>>>(
      grad, ctx->buf.pitch, ctx->nvec, m, kTagSupplied, ctx->cfg.seed, ctx->cfg.sigma, ctx->cfg.worker_offset);
  return check_launch(ctx);
}

int slowmo_debug_noise(slowmo_ctx *ctx, uint32_t tag, uint64_t t, uint32_t k, uint32_t w, uint64_t j0, uint64_t n,
                       uint64_t *words, float *normals) {
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  if (n == 0) return SLOWMO_OK;
  if (!words && !normals) return SLOWMO_EINVAL;
  const uint64_t key = stream_key(tag, ctx->cfg.seed, t, k, w);
  uint64_t blocks = (n + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)ctx->num_sms * 16;
  if (blocks > cap) blocks = cap;
  export_stream_kernel<<<(uint32_t)blocks, kThreads, 0, ctx->stream>>>(key, j0, n, words, normals);
  return check_launch(ctx);
}

int slowmo_debug_words_to_normals(slowmo_ctx *ctx, const uint64_t *words, uint64_t n, float *out) {
  if (!ctx || (n && (!words || !out))) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  if (n == 0) return SLOWMO_OK;
  uint64_t blocks = (n + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)ctx->num_sms * 16;
  if (blocks > cap) blocks = cap;
  words_to_normals_kernel<<<(uint32_t)blocks, kThreads, 0, ctx->stream>>>(words, n, out);
  return check_launch(ctx);
}

int slowmo_tensor_range(slowmo_ctx *ctx, uint32_t idx, uint64_t *offset, uint64_t *count) {
  if (!ctx || !offset || !count) return SLOWMO_EINVAL;
  if (ctx->tensor_offsets.empty() || idx >= ctx->cfg.n_tensors) return SLOWMO_EINVAL;
  *offset = ctx->tensor_offsets[idx];
  *count = ctx->tensor_offsets[idx + 1] - ctx->tensor_offsets[idx];
  return SLOWMO_OK;
}

int slowmo_set_variant(slowmo_ctx *ctx, int kernel, int variant) {
  if (!ctx) return SLOWMO_EINVAL;
  if (kernel == SLOWMO_K_OUTER) {
    if (variant != SLOWMO_VARIANT_DEFAULT && variant != SLOWMO_OUTER_DIRECT && variant != SLOWMO_OUTER_STAGED &&
        variant != SLOWMO_OUTER_FUSED && variant != SLOWMO_OUTER_LAZY)
      return SLOWMO_EINVAL;
    if (int rc = flush_pending(ctx)) return rc;
    ctx->outer_variant = variant;
    return SLOWMO_OK;
  }
  if (kernel == SLOWMO_K_LOCAL) {
    if (variant != SLOWMO_VARIANT_DEFAULT && variant != SLOWMO_LOCAL_ROW_TILES && variant != SLOWMO_LOCAL_COLUMN_OWNER)
      return SLOWMO_EINVAL;
    ctx->local_variant = variant;
    return SLOWMO_OK;
  }
  return SLOWMO_EINVAL;
}

int slowmo_sync_status(slowmo_ctx *ctx) {
  if (!ctx) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  if (int rc = flush_pending(ctx)) return rc;
  int host[4] = {0, 0, 0, 0};
  cudaError_t e = cudaMemcpyAsync(host, ctx->status_dev, sizeof(host), cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (host[0] != 0) {
    e = cudaMemsetAsync(ctx->status_dev, 0, sizeof(host), ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return SLOWMO_ETIMEOUT;
  }
  return SLOWMO_OK;
}

int slowmo_debug_wait_timeout(slowmo_ctx *ctx, uint32_t tries) {
  if (!ctx || tries == 0 || tries > (1u << 20)) return SLOWMO_EINVAL;
  if (ctx->cuda_error) return SLOWMO_ECUDA;
  bounded_wait_probe_kernel<<<1, 32, 0, ctx->stream>>>(ctx->status_dev, tries);
  return check_launch(ctx);
}

const char *slowmo_strerror(int status) {
  switch (status) {
    case SLOWMO_OK: return "ok";
    case SLOWMO_EINVAL: return "invalid argument";
    case SLOWMO_ESTATE: return "call not legal at this point of the outer/inner loop";
    case SLOWMO_EALIGN: return "pointer not 16-byte aligned or pitch not a multiple of 4";
    case SLOWMO_ECUDA: return "CUDA error (see slowmo_last_cuda_error)";
    case SLOWMO_ENOMEM: return "out of host memory";
    case SLOWMO_ETIMEOUT: return "a bounded device-side wait gave up";
    case SLOWMO_ENOTIMPL: return "not implemented";
    default: return "unknown status";
  }
}

int slowmo_last_cuda_error(slowmo_ctx *ctx) { return ctx ? ctx->cuda_error : 0; }

}  // extern "C"

// ---------------------------------------------------------------------------------------
// Allocation-free outer step (see slowmo_outer_step_static in include/slowmo.h).
//
// The staged outer-step kernel needs a few words of global scratch for its bounded-wait
// record. A context gets them from cudaMalloc; callers that may not allocate get them from
// this array, which is part of the library image on every device that loads it.
//
// In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// the address is looked up once per device with cudaGetSymbolAddress and that pointer is
// what the kernel receives.
// ---------------------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr int kStaticScratchInts = 64;  // 256 bytes; the kernel uses the first 4
static __device__ __align__(256) int g_static_scratch[kStaticScratchInts];

constexpr int kMaxDevices = 64;
struct StaticDeviceState {
  int *scratch = nullptr;  // device address of g_static_scratch on this device
  int num_sms = 0;
};
StaticDeviceState g_static_state[kMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the scratch address, raise the staged
// kernel's dynamic shared-memory limit, read the SM count. Allocates nothing.
cudaError_t static_setup(int dev, StaticDeviceState **out) {
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticDeviceState &st = g_static_state[dev];
  if (!st.scratch) {
    int *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = outer_staged_configure();
    if (e != cudaSuccess) return e;
    st.num_sms = sms;
    st.scratch = ptr;
  }
  *out = &st;
  return cudaSuccess;
}

}  // namespace

extern "C" int slowmo_outer_step_static(float *x, float *h, float *v, float *anchor, float *u, uint64_t pitch,
                                        uint64_t P, uint32_t m, int32_t base, int32_t buffer_policy, float alpha,
                                        float beta, float gamma_t, void *cuda_stream, int wait) {
  const bool adam = base == SLOWMO_BASE_ADAM;
  if (base != SLOWMO_BASE_NESTEROV && !adam) return SLOWMO_EINVAL;
  if (buffer_policy < SLOWMO_BUF_RESET || buffer_policy > SLOWMO_BUF_AVERAGE) return SLOWMO_EINVAL;
  if (P == 0 || P > SLOWMO_STATIC_MAX_P || m == 0 || m > SLOWMO_STATIC_MAX_M) return SLOWMO_EINVAL;
  if (!finite_pos(alpha) || !unit_interval(beta) || !finite_pos(gamma_t)) return SLOWMO_EINVAL;
  if (!x || !h || !anchor || !u || (adam && !v)) return SLOWMO_EINVAL;
  if (pitch % 4 != 0) return SLOWMO_EALIGN;
  if (pitch < P) return SLOWMO_EINVAL;
  const void *ptrs[] = {x, h, v, anchor, u};
  for (const void *p : ptrs)
    if (p && !aligned16(p)) return SLOWMO_EALIGN;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SLOWMO_ECUDA;
  StaticDeviceState *st = nullptr;
  if (static_setup(dev, &st) != cudaSuccess) return SLOWMO_ECUDA;
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  OuterArgs A;
  A.x = x;
  A.h = h;
  A.v = v;
  A.anchor = anchor;
  A.u = u;
  A.pitch = pitch;
  A.nvec = (uint32_t)((P + 3) / 4);
  A.m = m;
  A.beta = beta;
  A.inv_gamma = (float)(1.0 / (double)gamma_t);
  A.neg_alpha_gamma = -(float)((double)alpha * (double)gamma_t);
  A.m_float = (float)m;

  // the scratch keeps the previous call's record: clear the words the kernel reads
  if (cudaMemsetAsync(st->scratch, 0, 4 * sizeof(int), stream) != cudaSuccess) return SLOWMO_ECUDA;
  launch_outer_staged(A, adam ? 2 : 1, buffer_policy, st->num_sms, st->scratch, stream);
  if (cudaGetLastError() != cudaSuccess) return SLOWMO_ECUDA;
  if (!wait) return SLOWMO_OK;

  int host[4] = {0, 0, 0, 0};
  if (cudaMemcpyAsync(host, st->scratch, sizeof(host), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SLOWMO_ECUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SLOWMO_ECUDA;
  return host[0] != 0 ? SLOWMO_ETIMEOUT : SLOWMO_OK;
}
