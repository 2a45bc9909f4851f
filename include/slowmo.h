/*
 * libslowmo: the data-parallel hot path of Slow Momentum (SlowMo; Wang, Tantia, Ballas,
 * Rabbat, ICLR 2020) for m simulated workers held as an [m, P] fp32 replica tensor on one
 * NVIDIA B200 (sm_100a).
 *
 * The library runs the two phases of the paper's Algorithm 1:
 *   - the inner loop: tau steps x <- x - gamma_t d of the base optimizer on every replica,
 *     with the directions d of Table C.1 (SGD with Nesterov momentum, or Adam);
 *   - the outer step: exact average over the replicas, slow-momentum update (Eq. 2),
 *     outer-iterate update (Eq. 3), broadcast to all replicas, and the reset / maintain /
 *     average policy for the base-optimizer buffers (first statement of the outer loop).
 *
 * Conventions for every entry point
 *   Memory     All tensors are DEVICE pointers owned by the caller and borrowed for the
 *              life of the context. The library never allocates or frees tensor memory.
 *              slowmo_create makes one small device allocation (a status block of a few
 *              words) that slowmo_destroy releases.
 *   Layout     Row-major fp32. 2-D tensors are [m, pitch]: row i (worker i) starts at
 *              base + i*pitch elements; columns P..pitch-1 are padding. 1-D tensors have
 *              pitch elements. pitch is a multiple of 4 and >= P; every base pointer is
 *              16-byte aligned. Kernels process whole 4-element column groups, so padding
 *              columns below the next multiple of 4 are computed on and hold unspecified
 *              finite-or-not values; they are never returned by slowmo_get_params.
 *   Stream     Work is enqueued on the CUDA stream given at creation; calls return without
 *              waiting unless stated. One context per stream; a context is not thread-safe.
 *   Errors     Every call returns a SLOWMO_* status; nothing aborts or throws. CUDA
 *              failures are sticky in the context (SLOWMO_ECUDA; the cudaError_t is
 *              available from slowmo_last_cuda_error).
 *   Tracing    slowmo_local_steps, slowmo_outer_step, slowmo_iteration_host*, slowmo_materialize
 *              and slowmo_outer_step_sharded each open an NVTX range of their own name for the
 *              duration of the call (a no-op unless a profiler is attached).
 *   Numerics   All arithmetic is IEEE binary32 with the operation order documented at each
 *              call; the same configuration and seed give bit-identical state on every run.
 */
#ifndef SLOWMO_H
#define SLOWMO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct slowmo_ctx slowmo_ctx;

/* Largest parameter count per replica: the kernels index 4-column groups with 32 bits. */
#define SLOWMO_MAX_P ((1ull << 34) - 16384)

enum {
  SLOWMO_OK = 0,
  SLOWMO_EINVAL = -1,   /* bad argument (value, enum, NULL)                         */
  SLOWMO_ESTATE = -2,   /* call not legal at this point of Algorithm 1              */
  SLOWMO_EALIGN = -3,   /* pointer not 16-byte aligned or pitch not a multiple of 4 */
  SLOWMO_ECUDA = -4,    /* a CUDA call failed; sticky                               */
  SLOWMO_ENOMEM = -5,   /* host allocation failed                                   */
  SLOWMO_ETIMEOUT = -6, /* a bounded device-side wait gave up                       */
  SLOWMO_ENOTIMPL = -7
};
enum {
  SLOWMO_BASE_NESTEROV = 0,     /* Table C.1, SGD row: local Nesterov momentum, no communication   */
  SLOWMO_BASE_ADAM = 1,         /* Table C.1, Adam row                                              */
  SLOWMO_BASE_SGP_NESTEROV = 2, /* Algorithm 2: stochastic gradient push with Nesterov momentum     */
  SLOWMO_BASE_SGP_ADAM = 3      /* Table C.1, SGP (Adam) row                                        */
};
enum { SLOWMO_BUF_RESET = 0, SLOWMO_BUF_MAINTAIN = 1, SLOWMO_BUF_AVERAGE = 2 };
enum { SLOWMO_GRAD_GENERATED = 0, SLOWMO_GRAD_SUPPLIED = 1 };
/* tensors addressable by slowmo_get_params / slowmo_set_params */
enum {
  SLOWMO_T_X = 0,      /* replicas x^{(i)}            [m, pitch] */
  SLOWMO_T_ANCHOR = 1, /* x_{t,0}                     [pitch]    */
  SLOWMO_T_U = 2,      /* slow momentum u_t           [pitch]    */
  SLOWMO_T_H = 3,      /* first buffer h^{(i)}        [m, pitch] */
  SLOWMO_T_V = 4,      /* Adam second moment v^{(i)}  [m, pitch] */
  SLOWMO_T_A = 5,      /* curvature a_j               [pitch]    (generated mode) */
  SLOWMO_T_C = 6       /* centres c_{i,j}             [m, pitch] (generated mode) */
};
/* kernels whose implementation can be selected with slowmo_set_variant */
enum { SLOWMO_K_LOCAL = 0, SLOWMO_K_OUTER = 1 };
enum {
  SLOWMO_VARIANT_DEFAULT = 0,
  SLOWMO_OUTER_DIRECT = 1, /* vector loads straight to registers                      */
  SLOWMO_OUTER_STAGED = 2, /* bulk-copy (TMA) staging of row tiles through shared mem  */
  SLOWMO_OUTER_FUSED = 3,  /* the last inner step of each outer iteration runs inside the
                              outer-step kernel (same results, fewer HBM bytes); see
                              slowmo_local_steps for what this changes for the caller       */
  SLOWMO_OUTER_LAZY = 4,   /* SLOWMO_OUTER_FUSED, and in addition the outer step does not write
                              the m broadcast rows (nor the reset / averaged buffer rows): the
                              first inner step of the next iteration reads the anchor (and zero,
                              or the mean kept in row 0) instead of the rows. Same results through
                              the API; the caller's raw x, h, v tensors are up to date only after
                              slowmo_materialize or any call that reads state. Needs tau >= 2,
                              otherwise it behaves as SLOWMO_OUTER_FUSED                     */
  /* SLOWMO_K_LOCAL: layout of the fused local-step kernel (identical arithmetic per element) */
  SLOWMO_LOCAL_ROW_TILES = 5,    /* one block = one 2048-column tile of one replica row            */
  SLOWMO_LOCAL_COLUMN_OWNER = 6  /* one thread = one 4-column group of all m rows (reads the
                                    curvature once per column); the default with a generated
                                    gradient                                                      */
};

/*
 * Problem statement, after the "Input" line of Algorithm 1 (base optimizer with learning
 * rate gamma_t, tau, alpha, beta, m, x_{0,0}; u_0 = 0) plus the synthetic objective used in
 * generated-gradient mode: worker i minimises 1/2 sum_j a_j (x_j - c_{i,j})^2 and sees the
 * stochastic gradient a_j (x_j - c_{i,j}) + sigma z, z ~ N(0,1) from a counter-based hash of
 * (seed, t, k, i, j). a_j ~ U[a_lo, a_hi), c_{i,j} ~ N(0, c_std^2) are drawn from the same
 * hash at creation.
 */
typedef struct {
  uint64_t P;   /* parameters per replica (> 0, <= SLOWMO_MAX_P)                 */
  uint32_t m;   /* workers / replicas (> 0)                                      */
  uint32_t tau; /* base-optimizer steps per outer iteration (> 0)                */
  float alpha;  /* slow learning rate (> 0)                                      */
  float beta;   /* slow momentum factor, in [0, 1)                               */
  float gamma;  /* base learning rate gamma_0 (> 0, finite); see slowmo_set_gamma */
  int32_t base; /* SLOWMO_BASE_*                                                 */
  float mu;           /* beta_local of Table C.1 (SGD row), in [0, 1)            */
  float weight_decay; /* L2 coefficient, added to the gradient: g <- g + wd x    */
  float adam_b1, adam_b2, adam_eps; /* Table C.1 (Adam row); betas in [0,1), eps > 0 */
  int32_t buffer_policy;            /* SLOWMO_BUF_*                              */
  int32_t grad_mode;                /* SLOWMO_GRAD_*                             */
  uint64_t seed;
  float a_lo, a_hi, c_std, sigma; /* generator constants (sigma also scales slowmo_fill_gradient) */
  float x_init;                   /* x_{0,0} in every coordinate                 */
  uint32_t n_tensors;             /* optional segment table: number of parameter tensors */
  const uint64_t *tensor_sizes;   /* HOST array of n_tensors sizes summing to P, or NULL */
  int32_t no_average;             /* 0: Algorithm 1 as printed. 1: the variant of the paper's Section 6
                                     that skips the exact average: every worker applies Eq. (2), (3) to
                                     its own x_{t,tau}; anchor and u are then [m, pitch], one row per
                                     worker, and SLOWMO_BUF_AVERAGE is refused (EINVAL)                */
  uint32_t worker_offset;         /* global index of this context's first worker: row i is worker
                                     worker_offset + i for the noise and centre streams. 0 unless the m
                                     workers of a job are spread over several contexts (several GPUs)     */
} slowmo_config;

/* Device tensors borrowed from the caller (see "Layout" above). */
typedef struct {
  float *x;       /* [m, pitch]                                         */
  float *h;       /* [m, pitch]                                         */
  float *v;       /* [m, pitch]; required for Adam, may be NULL else    */
  float *anchor;  /* [pitch]; [m, pitch] with no_average                */
  float *u;       /* [pitch]; [m, pitch] with no_average                */
  float *a;       /* [pitch];    required in generated mode, else NULL  */
  float *c;       /* [m, pitch]; required in generated mode, else NULL  */
  uint64_t pitch; /* row length in elements                             */
} slowmo_buffers;

/*
 * Create a context and initialise the state of Algorithm 1's input line on the stream:
 * x^{(i)} = anchor = x_init, u = 0, h = v = 0, and in generated mode a and c from the hash.
 * `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).
 * Errors: EINVAL (any constraint listed beside the fields, unknown enum, NULL pointer,
 * sizes not summing to P), EALIGN, ENOMEM, ECUDA.
 */
int slowmo_create(const slowmo_config *cfg, const slowmo_buffers *buf, void *cuda_stream,
                  slowmo_ctx **out);

/* Release the context (never the caller's tensors). Waits for the stream first. */
int slowmo_destroy(slowmo_ctx *ctx);

/*
 * Inner loop of Algorithm 1: n base-optimizer steps on all m replicas, one fused kernel
 * launch per step. With k the steps already taken in this outer iteration, k + n <= tau is
 * required (ESTATE otherwise).
 *
 * Per element (worker i, coordinate j), in binary32:
 *   gradient   generated: e = x - c ; g = fma(a, e, sigma*z(t,k,i,j))   supplied: g = grad[i,j]
 *              then, if weight_decay != 0, g = fma(wd, x, g)
 *   Nesterov   h = fma(mu, h, g) ; d = fma(mu, h, g)                       (Table C.1, SGD)
 *   Adam       h = fma(b1, h, (1-b1)*g) ; v = fma(b2, v, (1-b2)*(g*g)) ;
 *              d = (h * 1/(1-b1^l)) / (sqrt(v * 1/(1-b2^l)) + eps)         (Table C.1, Adam)
 *              l = Adam steps since the buffers were last zero (1-based)
 *   step       x = fma(-gamma_t, d, x)                                     (Algorithm 1)
 *
 *   SGP bases  the step above yields x_{k+1/2}; then the push-sum mixing of Algorithm 2 on the
 *              time-varying directed exponential graph, one peer per step: with
 *              hops = 2^q, q = (t*tau + k) mod (floor(log2(m-1)) + 1), worker i keeps half and
 *              receives half from worker (i - hops) mod m:
 *              x_i = 0.5*x_{k+1/2,i} + 0.5*x_{k+1/2,(i-hops) mod m}.
 *              This mixing matrix is doubly stochastic, so the push-sum weights stay exactly 1
 *              and the de-biased z equals x; the gradient is therefore evaluated at x.
 *              SGP bases ignore SLOWMO_OUTER_FUSED and SLOWMO_OUTER_LAZY.
 *
 * `grad` is a device [m, pitch] tensor in supplied mode (read by each of the n steps) and
 * must be NULL in generated mode (EINVAL otherwise).
 *
 * With the SLOWMO_OUTER_FUSED variant selected, the step that completes the outer iteration
 * (k = tau-1) is not launched here: it is taken inside slowmo_outer_step's kernel. Until
 * then the caller's x, h, v tensors hold the state before that step, and in supplied mode
 * `grad` must stay valid and unchanged until slowmo_outer_step has been enqueued. Every
 * library call that reads or writes state (slowmo_get_params, slowmo_set_params,
 * slowmo_sync_status, slowmo_set_variant, slowmo_materialize, slowmo_destroy) first runs the
 * deferred step, so
 * results seen through the API are the same as without the variant.
 */
int slowmo_local_steps(slowmo_ctx *ctx, uint32_t n, const float *grad);

/*
 * Outer step of Algorithm 1 in one fused kernel; legal only after exactly tau local steps
 * (ESTATE otherwise). Per coordinate j, in binary32, with the gamma_t of this iteration:
 *   average    s = x^{(0)} ; s = s + x^{(i)} for i = 1..m-1 in order ; xbar = s / m
 *   Eq. (2)    u = fma(beta, u, (anchor - xbar) * (1/gamma_t))
 *   Eq. (3)    anchor = fma(-(alpha*gamma_t), u, anchor)
 *   broadcast  x^{(i)} = anchor for every i
 *   buffers    reset: h = v = 0 and l = 0; maintain: untouched;
 *              average: h^{(i)} = (sum over i in order) / m for every i, same for v
 * 1/gamma_t and alpha*gamma_t are formed in binary64 on the host and rounded once.
 * With no_average set there is no average and no broadcast: per worker i,
 *   u^{(i)} = fma(beta, u^{(i)}, (anchor^{(i)} - x^{(i)}) * (1/gamma_t)) ;
 *   anchor^{(i)} = fma(-(alpha*gamma_t), u^{(i)}, anchor^{(i)}) ; x^{(i)} = anchor^{(i)}.
 * Advances the outer counter t and sets k = 0.
 */
int slowmo_outer_step(slowmo_ctx *ctx);

/*
 * One whole outer iteration of Algorithm 1 (tau local steps, then the outer step) with HOST
 * input and output, pipelined over column windows: the per-worker problem data c [m, P]
 * (dense, no padding; pinned memory for the copies to overlap) is uploaded window by window on
 * a copy stream while the windows already on the device run their tau + 1 kernels on the
 * context's stream, and each window's new outer iterate is written to anchor_host ([P], or
 * [m, P] with no_average) on a second copy stream. Every statement of Algorithm 1 is elementwise
 * in the coordinate, so the windows are independent and the result is bit-identical to
 * slowmo_set_params(c) + slowmo_local_steps(tau) + slowmo_outer_step + slowmo_get_params(anchor).
 * `chunks` (1..1024) is the number of windows asked for; windows are whole 2048-column tiles.
 * Generated-gradient mode only (ENOTIMPL otherwise); legal only at k = 0 (ESTATE). Waits for
 * completion before returning.
 */
int slowmo_iteration_host(slowmo_ctx *ctx, const float *c_host, float *anchor_host, uint32_t chunks);

/*
 * The same for supplied-gradient mode (ENOTIMPL otherwise): the stochastic gradients of the
 * iteration, grad_host [m, P] (dense, host, pinned for overlap), are uploaded window by window into
 * the caller's DEVICE staging tensor grad_dev [m, pitch] (16-byte aligned, borrowed for the call),
 * and each window's tau local steps read it there, as slowmo_local_steps(tau, grad_dev) would: the
 * same gradient at each of the tau steps (Algorithm 1's stochastic gradient, held fixed over the
 * iteration). Bit-identical to copying grad_host into grad_dev and calling
 * slowmo_local_steps(tau, grad_dev) + slowmo_outer_step + slowmo_get_params(anchor).
 */
int slowmo_iteration_host_supplied(slowmo_ctx *ctx, const float *grad_host, float *grad_dev, float *anchor_host,
                                   uint32_t chunks);

/*
 * Outer step of Algorithm 1 for workers sharded over several GPUs of one node: the exact average
 * (the paper's AllReduce) fused with Eq. (2), Eq. (3), the broadcast and the buffer policy in
 * one kernel per GPU that reads and writes the other GPUs' memory directly.
 *
 * GPU r (0 <= r < world <= 16) holds the rows of global workers r*m_local .. r*m_local+m_local-1
 * in x[r], h[r] (v[r] for Adam bases), each [m_local, pitch], and full [pitch] copies anchor[r],
 * u[r] of the outer iterate and the slow momentum; the arrays x, h, v, anchor, u are HOST arrays
 * of `world` device pointers valid on the calling GPU (peer-mapped). The call made on GPU `rank`
 * handles that GPU's contiguous slice of the columns: it adds the rows of all GPUs in global
 * worker order (so the result is bit-identical to slowmo_outer_step on one GPU holding all
 * world*m_local workers), updates u and the anchor, and stores the slice into every GPU's
 * copies and rows, with the buffer policy. Every GPU makes the call with the same arguments
 * except `rank`.
 * Ordering is the caller's: all GPUs' local steps must have finished before any of these
 * kernels starts, and all of these kernels before anyone's next local step (for instance a
 * stream-ordered collective on each GPU's stream before and after). The kernels themselves
 * never wait for one another. Contexts that ran the local steps are told with
 * slowmo_outer_step_external. The local steps of sharded workers must use a communication-free
 * base (the SGP bases mix only the rows of one context). Errors as for slowmo_outer_step_static.
 * The call has no context, so a CUDA failure is returned as SLOWMO_ECUDA but recorded nowhere:
 * ask the CUDA runtime (cudaGetLastError) for the code.
 */
typedef struct {
  uint32_t world, rank;
  uint32_t m_local;              /* workers (rows) per GPU; m = world * m_local                     */
  uint64_t P, pitch;
  float *const *x, *const *h, *const *v;  /* [world] device pointers each; v may be NULL for Nesterov bases */
  float *const *anchor, *const *u;         /* [world] device pointers to the [pitch] copies                  */
  int32_t base, buffer_policy;   /* SLOWMO_BASE_* (tells whether v exists), SLOWMO_BUF_*             */
  float alpha, beta, gamma_t;
} slowmo_shard_args;
int slowmo_outer_step_sharded(const slowmo_shard_args *args, void *cuda_stream);

/* Tell a context that the outer step of the current iteration was carried out on its tensors by
 * other means (slowmo_outer_step_sharded): legal after exactly tau local steps (ESTATE
 * otherwise); runs a deferred last step if there is one, advances t, sets k = 0 and, under the
 * reset policy, restarts the Adam count. Launches nothing else. */
int slowmo_outer_step_external(slowmo_ctx *ctx);

/* Bring the caller's x, h, v tensors up to date: runs a deferred last inner step
 * (SLOWMO_OUTER_FUSED) and writes out virtual replicas and buffers (SLOWMO_OUTER_LAZY).
 * A no-op with the other variants. Enqueued on the stream. */
int slowmo_materialize(slowmo_ctx *ctx);

/* Change the base learning rate: the gamma_t of a learning-rate schedule. Algorithm 1 indexes
 * gamma by the outer iteration t only, and Section 2 (the remark under Eq. (3)) divides by
 * gamma_t in Eq. (2) precisely so that the slow momentum buffer does not depend on the
 * schedule; so the call is legal only between outer iterations, i.e. when k = 0 (ESTATE
 * otherwise), and the new value is used by the local steps, Eq. (2) and Eq. (3) of the
 * iteration that follows. EINVAL unless gamma > 0 and finite. */
int slowmo_set_gamma(slowmo_ctx *ctx, float gamma_t);

/*
 * Copy out part of a tensor: columns [offset, offset+count) of row `replica` (or of every
 * row when replica = -1, giving a dense [m, count] result; replica must be -1 or 0 for 1-D
 * tensors). offset + count <= P. `dst` is a host pointer (the call then waits for the
 * stream) or, with dst_on_device != 0, a device pointer (the copy is enqueued).
 */
int slowmo_get_params(slowmo_ctx *ctx, int which, int32_t replica, uint64_t offset, uint64_t count,
                      float *dst, int dst_on_device);

/* Inverse of slowmo_get_params: overwrite part of a tensor from host or device memory.
 * Used to restore a checkpoint and to upload per-worker problem data. */
int slowmo_set_params(slowmo_ctx *ctx, int which, int32_t replica, uint64_t offset, uint64_t count,
                      const float *src, int src_on_device);

/* Position in Algorithm 1: the loop indices t (outer iterations completed) and k (base-optimizer
 * steps taken in the current one), and Table C.1's step count l of the bias corrections (Adam
 * steps since the buffers were last zero). Any pointer may be NULL. */
int slowmo_get_counters(slowmo_ctx *ctx, uint64_t *t, uint32_t *k, uint64_t *l);

/*
 * Checkpoint and restore of everything Algorithm 1 carries besides the tensors: its loop indices
 * t and k, Table C.1's step count l (the caption's l = k with buffers reset, l = t tau + k with
 * buffers kept, counted from 1 here) and the gamma_t in force. Together with the tensors
 * x, anchor, u, h (and v), read with slowmo_get_params and written with slowmo_set_params, this
 * is the whole state: a context created with the same configuration, given the tensors and this
 * record, continues bit-identically to the run the checkpoint was taken from -- the noise of
 * step (t, k), the hop distance of the SGP graph and the bias corrections 1/(1 - beta^l) all
 * follow from the record. (beta_1^l and beta_2^l are re-formed by l successive binary64
 * multiplications, exactly as the step loop forms them.)
 *
 * slowmo_get_state may be called at any time. slowmo_set_state first writes out whatever the
 * context still owes its tensors (a deferred last inner step, virtual replicas), then moves to
 * the given position; call it BEFORE slowmo_set_params of the tensors when restoring. A state
 * with k = tau is legal (the outer step is then due). EINVAL: k > tau, gamma_t not finite and
 * positive, l < k, or l != k under SLOWMO_BUF_RESET.
 */
typedef struct {
  uint64_t t;    /* outer iterations completed                                    */
  uint64_t l;    /* base-optimizer steps since the buffers were last zero         */
  uint32_t k;    /* inner steps taken in the current outer iteration, 0 .. tau    */
  float gamma_t; /* base learning rate in force                                   */
} slowmo_state;
int slowmo_get_state(slowmo_ctx *ctx, slowmo_state *out);
int slowmo_set_state(slowmo_ctx *ctx, const slowmo_state *in);

/* Fill a device [m, pitch] tensor with the fixed synthetic gradient G[i,j] = sigma * z from
 * the hash (stream tag 5, worker i). For supplied-mode benchmarks; enqueued on the stream. */
int slowmo_fill_gradient(slowmo_ctx *ctx, float *grad);

/*
 * Export n consecutive draws of one noise stream, coordinates j0 <= j < j0 + n: the raw
 * 64-bit words (SplitMix64 outputs) and/or the binary32 normals derived from them.
 * Either device pointer may be NULL. Tags: 1 curvature, 2 centres, 3 gradient noise,
 * 5 supplied gradient. Test hook for the bit-exact comparison of the integer stream.
 */
int slowmo_debug_noise(slowmo_ctx *ctx, uint32_t tag, uint64_t t, uint32_t k, uint32_t w, uint64_t j0,
                       uint64_t n, uint64_t *words, float *normals);

/* Test hook: the two Box-Muller normals of each of n arbitrary 64-bit words (device arrays):
 * out[2i] (cosine output) and out[2i+1] (sine output) from words[i]. Lets a test sweep every
 * value of the 24-bit radius field and of the 24-bit angle field. */
int slowmo_debug_words_to_normals(slowmo_ctx *ctx, const uint64_t *words, uint64_t n, float *out);

/* Segment idx of the optional parameter-tensor table: first coordinate and length. The method
 * treats the model as one vector x in R^d (Eq. (1)); a network's parameter tensors are contiguous
 * segments of it, and this table only records where they lie. EINVAL without a table or for
 * idx >= n_tensors. */
int slowmo_tensor_range(slowmo_ctx *ctx, uint32_t idx, uint64_t *offset, uint64_t *count);

/* Select the implementation of a kernel: SLOWMO_K_OUTER with SLOWMO_VARIANT_DEFAULT or a
 * SLOWMO_OUTER_* value, SLOWMO_K_LOCAL with SLOWMO_VARIANT_DEFAULT or a SLOWMO_LOCAL_* value
 * (EINVAL otherwise). All variants compute identical results. */
int slowmo_set_variant(slowmo_ctx *ctx, int kernel, int variant);

/* Wait for the stream and report SLOWMO_ETIMEOUT if any kernel recorded that one of its
 * bounded waits ran out (the record is then cleared), SLOWMO_ECUDA on a CUDA failure. */
int slowmo_sync_status(slowmo_ctx *ctx);

/*
 * Outer step without a context and without any allocation. (The paper has no counterpart:
 * this entry point exists for callers that must not allocate device memory.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework whose
 * caching allocator owns all device memory and forbids raw allocations, in a process whose
 * memory budget was fixed up front, or in a latency-critical loop where an allocation's
 * implicit device synchronisation is unacceptable. slowmo_create cannot serve them,
 * because it allocates the small status block that the staged (bulk-copy) outer-step
 * kernel writes its bounded-wait record into. Here that scratch lives in a fixed 256-byte
 * array inside the library image instead (every GPU that loads the library holds those 256
 * bytes until the process exits), and all parameters that a context would remember are
 * passed in.
 *
 * Computes exactly what slowmo_outer_step computes (same kernel, same arithmetic, same
 * order): average of the m rows of x, Eq. (2), Eq. (3), broadcast, buffer policy, on the
 * caller's device tensors x, h [m, pitch], v [m, pitch] (Adam only, else NULL), anchor,
 * u [pitch], with the layout rules at the top of this file. base is SLOWMO_BASE_NESTEROV or
 * SLOWMO_BASE_ADAM (it only tells whether v exists); buffer_policy is SLOWMO_BUF_*.
 *
 * Limits: the scratch does not grow with the problem, so the only size limits are the
 * kernel's index range: 1 <= P <= SLOWMO_STATIC_MAX_P and 1 <= m <= SLOWMO_STATIC_MAX_M;
 * anything larger is refused with SLOWMO_EINVAL before any GPU work. Other errors as for
 * slowmo_create / slowmo_outer_step (EINVAL, EALIGN, ECUDA).
 *
 * Set-up: the first call on each device (with that device current) looks up the scratch
 * array's device address and raises the kernel's shared-memory limit. That first call
 * should come before any stream capture. No call allocates or frees memory.
 *
 * Sharing: every call on a device uses the same scratch and clears it on the stream before
 * its kernel. Calls that overlap on the GPU (different streams, or several host threads)
 * race on it: their results stay correct, but a timeout record may be lost or attributed to
 * the wrong call. Serialise calls if the record matters.
 *
 * wait != 0: the call waits for the stream and returns SLOWMO_ETIMEOUT if the kernel
 * recorded that a bounded wait ran out (results are then invalid). wait == 0: the call
 * returns once the work is enqueued.
 */
#define SLOWMO_STATIC_MAX_P ((1ull << 32) - 4096)
#define SLOWMO_STATIC_MAX_M 65536u
int slowmo_outer_step_static(float *x, float *h, float *v, float *anchor, float *u, uint64_t pitch,
                             uint64_t P, uint32_t m, int32_t base, int32_t buffer_policy, float alpha,
                             float beta, float gamma_t, void *cuda_stream, int wait);

/*
 * Test hook for the error path of the bounded device-side waits: enqueues a one-block kernel
 * that waits, with the pipeline's own try loop limited to `tries` (1 .. 2^20) attempts, on a
 * barrier that nothing completes, and records the timeout. The next slowmo_sync_status
 * returns SLOWMO_ETIMEOUT once and clears the record; the context and the GPU stay usable.
 */
int slowmo_debug_wait_timeout(slowmo_ctx *ctx, uint32_t tries);

const char *slowmo_strerror(int status);
int slowmo_last_cuda_error(slowmo_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif
