// sm_100a kernels of the SlowMo hot path: synthetic-input fills, the fused multi-replica
// base-optimizer step (Algorithm 1's inner statement with Table C.1's directions) and the
// fused outer step (exact average, Eq. 2, Eq. 3, broadcast, buffer policy).
//
// All of them are HBM-bound streams over [m, pitch] fp32 tensors: one 128-bit access per
// thread per tensor, full-line coalescing across the warp, several independent loads in
// flight per thread, and grids of many short blocks so the tail is negligible.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "noise.cuh"

namespace slowmo {

constexpr int kThreads = 256;

// Tunables (overridable at compile time for parameter sweeps).
#ifndef SLOWMO_LOCAL_UNROLL
#define SLOWMO_LOCAL_UNROLL 2   // 128-bit column groups per thread in the local-step kernel
#endif
#ifndef SLOWMO_LOCAL_MIN_BLOCKS
#define SLOWMO_LOCAL_MIN_BLOCKS 1  // __launch_bounds__ minimum resident blocks per SM
#endif
#ifndef SLOWMO_LOCAL_LAYOUT
#define SLOWMO_LOCAL_LAYOUT 0   // 0: choose by m; 1: always row tiles; 2: column owner whenever possible
#endif
#ifndef SLOWMO_LOCAL_COL_ROWS
#define SLOWMO_LOCAL_COL_ROWS 4  // rows in flight per thread in the column-owner layout (Nesterov; Adam half)
#endif
#ifndef SLOWMO_STREAM_HINT
#define SLOWMO_STREAM_HINT 0    // 1: evict-first (.cs) loads and stores, 0: default policy
#endif
constexpr int kLocalUnroll = SLOWMO_LOCAL_UNROLL;

// ---- streaming 128-bit accesses --------------------------------------------------------
// Tensors are far larger than L2 and every line is used exactly once per launch. The
// evict-first policy (.cs) measured equal or slightly slower than the default on B200, so
// the default policy is used; the hint stays selectable for sweeps.
#if SLOWMO_STREAM_HINT
__device__ __forceinline__ float4 ld_stream(const float *p) { return __ldcs(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ void st_stream(float *p, float4 v) { __stcs(reinterpret_cast<float4 *>(p), v); }
#else
__device__ __forceinline__ float4 ld_stream(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st_stream(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
#endif
// `a` is shared by the m rows of a column tile: keep it cacheable so the blocks of the other
// rows, which run next to this one, find it in L2.
__device__ __forceinline__ float4 ld_shared_row(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

// The two kernels that are bound by instruction issue keep few loads in flight per thread (two rows
// at a time, then some hundred instructions of arithmetic per row). Asking L2 for the next rows
// while the current ones are worked on costs one instruction per row and no register. Measured on
// B200 (resnet50 / transformer shapes): the virtual-replica first step gains 5 % with the Nesterov
// base and loses 2 % with Adam; the fused outer step gains 5 % with Adam and loses 6 % with
// Nesterov. Hence the defaults below (1: Nesterov only, 2: Adam only, 0: never, 3: always).
// With a supplied gradient these kernels wait on HBM, not on issue slots, and the extra requests
// only get in the way (virtual-replica first step at P = 1e9, m = 4: 8.3 ms with, 7.7 ms without),
// so the prefetch is compiled in for the generated gradient only.
#ifndef SLOWMO_PREFETCH_VIRT
#define SLOWMO_PREFETCH_VIRT 1
#endif
#ifndef SLOWMO_PREFETCH_FUSED
#define SLOWMO_PREFETCH_FUSED 2
#endif
__device__ __forceinline__ void prefetch_l2(const float *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
template <int BASE, int GRAD>
__device__ __forceinline__ constexpr bool prefetch_on(int mode) { return GRAD == 0 && ((mode >> BASE) & 1); }

__device__ __forceinline__ float &comp(float4 &v, int e) { return reinterpret_cast<float *>(&v)[e]; }
__device__ __forceinline__ float comp(const float4 &v, int e) { return reinterpret_cast<const float *>(&v)[e]; }

// ---- K0: fills ---------------------------------------------------------------------------

// dst[i, j] = scale * z(tag, seed, 0, 0, i, j) for every row i < rows and column j < 4*nvec
// (blockIdx.y strides over the rows, so the row count is not limited by the grid).
__global__ void __launch_bounds__(kThreads)
fill_normal_rows_kernel(float *dst, uint64_t pitch, uint32_t nvec, uint32_t rows, uint32_t tag, uint64_t seed,
                        float scale, uint32_t worker0) {
  for (uint32_t row = blockIdx.y; row < rows; row += gridDim.y) {
    const uint64_t key = stream_key(tag, seed, 0, 0, worker0 + row);  // row i holds global worker worker0 + i
    float *p = dst + (uint64_t)row * pitch;
    for (uint64_t vi = (uint64_t)blockIdx.x * kThreads + threadIdx.x; vi < nvec; vi += (uint64_t)gridDim.x * kThreads) {
      // columns 4vi..4vi+3 are the pairs 2vi and 2vi+1 of the row's stream
      const uint64_t s = key + kGoldenGamma * (2 * vi + 1);
      const float4 z = two_words_to_normals(mix64(s), mix64(s + kGoldenGamma));
      st_stream(p + 4 * vi, make_float4(__fmul_rn(scale, z.x), __fmul_rn(scale, z.y), __fmul_rn(scale, z.z),
                                        __fmul_rn(scale, z.w)));
    }
  }
}

// a[j] = fma(a_hi - a_lo, U_j, a_lo), U_j from the curvature stream.
__global__ void __launch_bounds__(kThreads)
fill_curvature_kernel(float *a, uint32_t nvec, uint64_t seed, float a_lo, float a_hi) {
  const uint64_t key = stream_key(kTagCurvature, seed, 0, 0, 0);
  const float span = __fsub_rn(a_hi, a_lo);
  for (uint64_t vi = (uint64_t)blockIdx.x * kThreads + threadIdx.x; vi < nvec; vi += (uint64_t)gridDim.x * kThreads) {
    uint64_t s = key + kGoldenGamma * (4 * vi + 1);
    float4 o;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      comp(o, e) = __fmaf_rn(span, word_to_unit(mix64(s)), a_lo);
      s += kGoldenGamma;
    }
    st_stream(a + 4 * vi, o);
  }
}

// dst[i, j] = value for every row i < rows and column j < 4*nvec.
__global__ void __launch_bounds__(kThreads)
fill_value_rows_kernel(float *dst, uint64_t pitch, uint32_t nvec, uint32_t rows, float value) {
  const float4 o = make_float4(value, value, value, value);
  for (uint32_t row = blockIdx.y; row < rows; row += gridDim.y) {
    float *p = dst + (uint64_t)row * pitch;
    for (uint64_t vi = (uint64_t)blockIdx.x * kThreads + threadIdx.x; vi < nvec; vi += (uint64_t)gridDim.x * kThreads)
      st_stream(p + 4 * vi, o);
  }
}

// Export of one stream for the bit-exact test, j0 <= j < j0 + n: word j of the stream and/or
// the normal of coordinate j.
__global__ void __launch_bounds__(kThreads)
export_stream_kernel(uint64_t key, uint64_t j0, uint64_t n, uint64_t *words, float *normals) {
  for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (uint64_t)gridDim.x * kThreads) {
    const uint64_t r = stream_word(key, j0 + i);
    if (words) words[i] = r;
    if (normals) normals[i] = stream_normal(key, j0 + i);
  }
}

// Test hook: both normals of arbitrary words, out[2i], out[2i+1] from words[i]. The kernels make
// their normals two words at a time, one word in each half of the packed registers; so every
// word goes through here in both halves (paired with its neighbour, then the other way round),
// and a word whose two evaluations differ in any bit is reported as NaN.
__global__ void __launch_bounds__(kThreads)
words_to_normals_kernel(const uint64_t *words, uint64_t n, float *out) {
  for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (uint64_t)gridDim.x * kThreads) {
    const uint64_t w = words[i], other = words[i + 1 < n ? i + 1 : 0];
    const float4 first = two_words_to_normals(w, other);   // w in the low half
    const float4 second = two_words_to_normals(other, w);  // w in the high half
    const bool same = __float_as_uint(first.x) == __float_as_uint(second.z) &&
                      __float_as_uint(first.y) == __float_as_uint(second.w);
    out[2 * i] = same ? first.x : __uint_as_float(0x7FC00000u);
    out[2 * i + 1] = same ? first.y : __uint_as_float(0x7FC00000u);
  }
}

// ---- K1: fused multi-replica base-optimizer step ------------------------------------------

constexpr uint32_t kInlineKeys = 64;  // noise keys of up to this many rows travel in the kernel arguments

struct LocalArgs {
  float *x, *h, *v;       // [m, pitch]
  const float *src;       // generated mode: centres c [m, pitch]; supplied mode: gradient G [m, pitch]
  const float *a;         // [pitch], generated mode
  const float *anchor;    // [pitch]: x_{t,0}, read in place of the x rows when the replicas are virtual
  int virt;               // 0: rows hold the state. Else the outer step left the broadcast (and the buffer
                          // policy) to this launch: x_i = anchor for every i, and the buffers are
                          // 1: as stored (maintain), 2: zero (reset), 3: the mean kept in row 0 (average)
  uint64_t pitch;
  uint32_t nvec;          // 4-element column groups per row (of the column window being processed)
  uint32_t vec0;          // index of the window's first column group in the whole vector (noise index)
  uint32_t m;
  uint32_t worker0;       // global index of row 0's worker (non-zero when the workers are sharded over GPUs)
  uint64_t seed, t;       // outer iteration, for the noise key
  uint32_t k;             // inner step, for the noise key
  float neg_gamma, mu, wd, sigma;
  float b1, b2, omb1, omb2, ibc1, ibc2, eps;  // Adam: betas, 1-betas, 1/(1-beta^l), epsilon
  uint64_t keys[kInlineKeys];  // generated mode, m <= kInlineKeys: stream key of (t, k, row), host-computed
};

// One element of the base-optimizer step (Table C.1 direction, then Algorithm 1's update).
template <int BASE>
__device__ __forceinline__ void base_step(const LocalArgs &A, float g, float &x, float &h, float &v) {
  if (A.wd != 0.0f) g = __fmaf_rn(A.wd, x, g);
  float d;
  if (BASE == 0) {
    h = __fmaf_rn(A.mu, h, g);
    d = __fmaf_rn(A.mu, h, g);
  } else {
    h = __fmaf_rn(A.b1, h, __fmul_rn(A.omb1, g));
    v = __fmaf_rn(A.b2, v, __fmul_rn(A.omb2, __fmul_rn(g, g)));
    d = __fdiv_rn(__fmul_rn(h, A.ibc1), __fadd_rn(__fsqrt_rn(__fmul_rn(v, A.ibc2)), A.eps));
  }
  x = __fmaf_rn(A.neg_gamma, d, x);
}

// Position of a 4-column group in a row's noise stream: columns 4v..4v+3 take the Box-Muller
// pairs of words 2v and 2v+1, i.e. the generator states key + G(2v+1) and key + G(2v+2). The
// term G(2v+1) does not depend on the row, so a thread that walks several rows forms it once.
__device__ __forceinline__ uint64_t noise_counter(uint64_t vec_index) { return kGoldenGamma * (2ull * vec_index + 1); }

// Stochastic gradient of the synthetic objective for one 4-column group of one worker:
// g = fma(a, x - c, sigma * z), z from the worker's noise stream (key) at `counter`.
//
// PACKED selects between two bit-identical evaluations. false: the scalar normal map and scalar
// arithmetic, used by the kernels that wait on HBM anyway (there the shorter instruction stream
// measured 0.4-2 % slower). true: the two-word packed map and packed arithmetic (about a quarter
// fewer instructions per update), used by the kernels that are bound by instruction issue: the
// virtual-replica first step, the outer step with the last inner step fused in, and the SGP step.
template <bool PACKED>
__device__ __forceinline__ float4 generated_gradient(uint64_t key, uint64_t counter, const float4 &a, const float4 &x,
                                                     const float4 &c, float sigma) {
  const uint64_t st = key + counter;
  if (PACKED) {
    const float4 z = two_words_to_normals(mix64(st), mix64(st + kGoldenGamma));
    const float2 s2 = splat2(sigma);
    const float2 lo = fma2(make_float2(a.x, a.y), add2(make_float2(x.x, x.y), neg2(make_float2(c.x, c.y))),
                           mul2(s2, make_float2(z.x, z.y)));
    const float2 hi = fma2(make_float2(a.z, a.w), add2(make_float2(x.z, x.w), neg2(make_float2(c.z, c.w))),
                           mul2(s2, make_float2(z.z, z.w)));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  }
  float4 z, g;
  word_to_normal_pair(mix64(st), z.x, z.y);
  word_to_normal_pair(mix64(st + kGoldenGamma), z.z, z.w);
#pragma unroll
  for (int e = 0; e < 4; ++e)
    comp(g, e) = __fmaf_rn(comp(a, e), __fsub_rn(comp(x, e), comp(c, e)), __fmul_rn(sigma, comp(z, e)));
  return g;
}

// The base-optimizer step on a 4-column group. PACKED: Nesterov momentum is all fused
// multiply-adds and runs on packed pairs; Adam's division and square root are scalar, so it goes
// element by element either way.
template <int BASE, bool PACKED>
__device__ __forceinline__ void base_step4(const LocalArgs &A, const float4 &g, float4 &x, float4 &h, float4 &v) {
  if (BASE == 0 && PACKED) {
    float2 g0 = make_float2(g.x, g.y), g1 = make_float2(g.z, g.w);
    float2 x0 = make_float2(x.x, x.y), x1 = make_float2(x.z, x.w);
    float2 h0 = make_float2(h.x, h.y), h1 = make_float2(h.z, h.w);
    if (A.wd != 0.0f) {
      g0 = fma2(splat2(A.wd), x0, g0);
      g1 = fma2(splat2(A.wd), x1, g1);
    }
    const float2 mu = splat2(A.mu), ng = splat2(A.neg_gamma);
    h0 = fma2(mu, h0, g0);
    h1 = fma2(mu, h1, g1);
    x0 = fma2(ng, fma2(mu, h0, g0), x0);
    x1 = fma2(ng, fma2(mu, h1, g1), x1);
    x = make_float4(x0.x, x0.y, x1.x, x1.y);
    h = make_float4(h0.x, h0.y, h1.x, h1.y);
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) base_step<BASE>(A, comp(g, e), comp(x, e), comp(h, e), comp(v, e));
  }
}

// Noise keys of the rows a thread walks (column-owner kernels). Up to kInlineKeys rows the keys
// come with the kernel arguments. Beyond that (DERIVE) the warp derives them itself, 32 at a
// time: at every 32nd position of the walk lane l computes the key of the row at position
// base + l (five mix64), and a shuffle hands the key of the current position to all lanes.
// No memory is involved, so the worker count is unlimited. All 32 lanes of a warp must stay in
// the walk (no early exit) because the shuffles name the full warp.
template <bool DERIVE>
struct RowKeys {
  uint64_t lane_key = 0;
  // call when (position & 31) == 0, with the row this lane's position base + lane maps to
  __device__ __forceinline__ void refill(const LocalArgs &A, uint32_t row_of_lane) {
    if (DERIVE) lane_key = stream_key(kTagGradNoise, A.seed, A.t, A.k, A.worker0 + row_of_lane);
  }
  __device__ __forceinline__ uint64_t at(const LocalArgs &A, uint32_t position, uint32_t row) const {
    if (DERIVE) return __shfl_sync(0xFFFFFFFFu, lane_key, (int)(position & 31u));
    return A.keys[row];
  }
};

// One block = one tile of kThreads*U column groups of one row. Consecutive blocks are the m
// rows of the same tile, so the shared curvature tile is read from DRAM once and from L2
// m-1 times. Each thread issues all its loads (3 or 4 tensors x U) before any arithmetic.
// The noise key of the row comes with the kernel arguments (computed on the host, the same
// integer arithmetic) so that no issue slot is spent on it; beyond kInlineKeys rows one lane
// per warp derives it while the loads are in flight.
template <int BASE, int GRAD, int U>
__global__ void __launch_bounds__(kThreads, SLOWMO_LOCAL_MIN_BLOCKS)
local_step_kernel(const LocalArgs A) {
  const uint32_t row = blockIdx.x % A.m;
  const uint32_t tile = blockIdx.x / A.m;
  const uint32_t v0 = tile * (uint32_t)(kThreads * U) + threadIdx.x;
  const uint64_t roff = (uint64_t)row * A.pitch;

  float4 x[U], h[U], v[U], s[U], a[U];
  bool ok[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const uint32_t vi = v0 + u * kThreads;
    ok[u] = vi < A.nvec;
    if (ok[u]) {
      const uint64_t off = roff + 4ull * vi;
      x[u] = ld_stream(A.x + off);
      h[u] = ld_stream(A.h + off);
      if (BASE == 1) v[u] = ld_stream(A.v + off);
      s[u] = ld_stream(A.src + off);
      if (GRAD == 0) a[u] = ld_shared_row(A.a + 4ull * vi);
    }
  }

  uint64_t key = 0;
  if (GRAD == 0) {
    if (A.m <= kInlineKeys) {
      key = A.keys[row];
    } else {  // many workers: one lane per warp derives the key while the loads are in flight
      if ((threadIdx.x & 31u) == 0) key = stream_key(kTagGradNoise, A.seed, A.t, A.k, A.worker0 + row);
      key = __shfl_sync(0xFFFFFFFFu, key, 0);
    }
  }

#pragma unroll
  for (int u = 0; u < U; ++u) {
    if (!ok[u]) continue;
    const uint32_t vi = v0 + u * kThreads;
    float4 g;
    if (GRAD == 0) g = generated_gradient<false>(key, noise_counter(A.vec0 + vi), a[u], x[u], s[u], A.sigma);
    else g = s[u];
    base_step4<BASE, false>(A, g, x[u], h[u], v[u]);
    const uint64_t off = roff + 4ull * vi;
    st_stream(A.x + off, x[u]);
    st_stream(A.h + off, h[u]);
    if (BASE == 1) st_stream(A.v + off, v[u]);
  }
}

// Column-owner layout of the same step: one thread owns a 4-column group and walks all m rows,
// ROWS at a time. The curvature is loaded once per column (instead of once per row from L2)
// and consecutive rows of a thread's loads are independent, so fewer threads keep as many
// bytes in flight. Same arithmetic per element as local_step_kernel: results are identical.
// DERIVE: more rows than noise keys fit the kernel arguments (see RowKeys); threads past the end
// of the row then stay in the loop, with their loads and stores switched off.
#ifndef SLOWMO_VIRT_MIN_BLOCKS
#define SLOWMO_VIRT_MIN_BLOCKS 4   // resident blocks per SM asked of the virtual-replica form
#endif
#ifndef SLOWMO_COLS_MIN_BLOCKS
#define SLOWMO_COLS_MIN_BLOCKS 3   // same for the ordinary form (80 registers; unbounded it took 110 and ran 10 % slower)
#endif
template <int BASE, int GRAD, int ROWS, bool VIRT, bool DERIVE>
__global__ void __launch_bounds__(kThreads, VIRT ? SLOWMO_VIRT_MIN_BLOCKS : SLOWMO_COLS_MIN_BLOCKS)
local_step_cols_kernel(const LocalArgs A) {
  static_assert(32 % ROWS == 0, "key refills happen at multiples of 32 rows");
  const uint32_t vi = blockIdx.x * kThreads + threadIdx.x;
  if (!DERIVE && vi >= A.nvec) return;
  const bool ok = DERIVE ? vi < A.nvec : true;
  const uint64_t col = ok ? 4ull * vi : 0;  // switched-off threads of the last warp point at column 0 and touch nothing
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  if (GRAD == 0 && ok) a = ld_shared_row(A.a + col);
  const uint64_t counter = noise_counter(A.vec0 + vi);
  RowKeys<DERIVE> keys;
  // virtual replicas: every row starts from the anchor; buffers from zero or from the mean in row 0
  float4 x_all = a, h_all = make_float4(0.f, 0.f, 0.f, 0.f), v_all = h_all;
  if (VIRT && ok) {
    x_all = ld_stream(A.anchor + col);
    if (A.virt == 3) {
      h_all = ld_stream(A.h + col);
      if (BASE == 1) v_all = ld_stream(A.v + col);
    }
  }
  for (uint32_t i0 = 0; i0 < A.m; i0 += ROWS) {
    if (GRAD == 0 && (i0 & 31u) == 0) keys.refill(A, i0 + (threadIdx.x & 31u));
    float4 x[ROWS], h[ROWS], v[ROWS], s[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      if (ok && i0 + q < A.m) {
        const uint64_t off = (uint64_t)(i0 + q) * A.pitch + col;
        if (!VIRT) {
          x[q] = ld_stream(A.x + off);
          h[q] = ld_stream(A.h + off);
          if (BASE == 1) v[q] = ld_stream(A.v + off);
        } else {
          x[q] = x_all;
          if (A.virt == 1) {
            h[q] = ld_stream(A.h + off);
            if (BASE == 1) v[q] = ld_stream(A.v + off);
          } else {
            h[q] = h_all;
            v[q] = v_all;
          }
        }
        s[q] = ld_stream(A.src + off);
        if (VIRT && prefetch_on<BASE, GRAD>(SLOWMO_PREFETCH_VIRT) && i0 + q + ROWS < A.m)
          prefetch_l2(A.src + off + (uint64_t)ROWS * A.pitch);
      }
    }
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      const uint32_t i = i0 + q;
      if (i >= A.m) break;
      uint64_t key = 0;
      if (GRAD == 0) key = keys.at(A, i, i);
      if (!ok) continue;
      float4 g;
      // the virtual-replica form moves fewer bytes per update and is bound by instruction issue
      if (GRAD == 0) g = generated_gradient<VIRT>(key, counter, a, x[q], s[q], A.sigma);
      else g = s[q];
      base_step4<BASE, VIRT && GRAD == 0>(A, g, x[q], h[q], v[q]);
      const uint64_t off = (uint64_t)i * A.pitch + col;
      st_stream(A.x + off, x[q]);
      st_stream(A.h + off, h[q]);
      if (BASE == 1) st_stream(A.v + off, v[q]);
    }
  }
}

// ---- K2: fused outer step, direct variant ---------------------------------------------------

struct OuterArgs {
  float *x, *h, *v;   // [m, pitch]
  float *anchor, *u;  // [pitch]
  uint64_t pitch;
  uint32_t nvec, m;
  float beta, inv_gamma, neg_alpha_gamma, m_float;
};

// Sum of the m rows of one column group in row order, then division by m. ROWS loads are issued
// together, the last batch with the rows past m switched off, so that no row is fetched only
// after the previous one has arrived; the additions stay in index order. The sum starts from -0,
// the one value for which s + v == v bit for bit whatever v is (signed zeros included), so the
// result equals x_0 + x_1 + ... added left to right.
#ifndef SLOWMO_OUTER_ROWS
#define SLOWMO_OUTER_ROWS 4   // rows loaded together (4 and 8 measured alike at m = 16, 32; 4 is 3 % faster at m = 8)
#endif
template <int ROWS>
__device__ __forceinline__ float4 ordered_row_mean(const float *base, uint64_t pitch, uint32_t m, float m_float) {
  float4 s = make_float4(-0.0f, -0.0f, -0.0f, -0.0f);
  for (uint32_t i = 0; i < m; i += ROWS) {
    float4 r[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q)
      if (i + q < m) r[q] = ld_stream(base + (uint64_t)(i + q) * pitch);
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      if (i + q >= m) break;
      s.x = __fadd_rn(s.x, r[q].x);
      s.y = __fadd_rn(s.y, r[q].y);
      s.z = __fadd_rn(s.z, r[q].z);
      s.w = __fadd_rn(s.w, r[q].w);
    }
  }
  return make_float4(__fdiv_rn(s.x, m_float), __fdiv_rn(s.y, m_float), __fdiv_rn(s.z, m_float),
                     __fdiv_rn(s.w, m_float));
}

__device__ __forceinline__ void store_rows(float *base, uint64_t pitch, uint32_t m, float4 val) {
#pragma unroll 4
  for (uint32_t i = 0; i < m; ++i) st_stream(base + (uint64_t)i * pitch, val);
}

// One thread = one 4-element column group: rows in, (u, anchor) update, rows out.
// NBUF = number of base-optimizer buffers (1: h, 2: h and v); POLICY as SLOWMO_BUF_*.
template <int NBUF, int POLICY>
__global__ void __launch_bounds__(kThreads)
outer_step_direct_kernel(const OuterArgs A) {
  const uint32_t vi = blockIdx.x * kThreads + threadIdx.x;
  if (vi >= A.nvec) return;
  const uint64_t col = 4ull * vi;

  const float4 x0 = ld_stream(A.anchor + col);
  const float4 u0 = ld_stream(A.u + col);
  const float4 xbar = ordered_row_mean<SLOWMO_OUTER_ROWS>(A.x + col, A.pitch, A.m, A.m_float);
  float4 un, xn;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    // Eq. (2): u <- beta u + (x_{t,0} - xbar)/gamma ; Eq. (3): x_{t+1,0} <- x_{t,0} - alpha gamma u
    const float ue = __fmaf_rn(A.beta, comp(u0, e), __fmul_rn(__fsub_rn(comp(x0, e), comp(xbar, e)), A.inv_gamma));
    comp(un, e) = ue;
    comp(xn, e) = __fmaf_rn(A.neg_alpha_gamma, ue, comp(x0, e));
  }
  st_stream(A.u + col, un);
  st_stream(A.anchor + col, xn);
  store_rows(A.x + col, A.pitch, A.m, xn);

  if (POLICY == 0) {  // reset
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    store_rows(A.h + col, A.pitch, A.m, zero);
    if (NBUF == 2) store_rows(A.v + col, A.pitch, A.m, zero);
  } else if (POLICY == 2) {  // average
    const float4 hbar = ordered_row_mean<SLOWMO_OUTER_ROWS>(A.h + col, A.pitch, A.m, A.m_float);
    store_rows(A.h + col, A.pitch, A.m, hbar);
    if (NBUF == 2) {
      const float4 vbar = ordered_row_mean<SLOWMO_OUTER_ROWS>(A.v + col, A.pitch, A.m, A.m_float);
      store_rows(A.v + col, A.pitch, A.m, vbar);
    }
  }
}

// Writes out what a lazy outer step left virtual: x_i = anchor for every row, and the buffer
// rows per policy (2: zeros, 3: copies of row 0; 1: nothing to do).
template <int NBUF>
__global__ void __launch_bounds__(kThreads)
materialize_kernel(float *x, float *h, float *v, const float *anchor, uint64_t pitch, uint32_t nvec, uint32_t m,
                   int virt) {
  const uint32_t vi = blockIdx.x * kThreads + threadIdx.x;
  if (vi >= nvec) return;
  const uint64_t col = 4ull * vi;
  const float4 x0 = ld_stream(anchor + col);
  for (uint32_t i = 0; i < m; ++i) st_stream(x + (uint64_t)i * pitch + col, x0);
  if (virt == 2) {
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t i = 0; i < m; ++i) {
      st_stream(h + (uint64_t)i * pitch + col, zero);
      if (NBUF == 2) st_stream(v + (uint64_t)i * pitch + col, zero);
    }
  } else if (virt == 3) {
    const float4 hb = ld_stream(h + col);
    for (uint32_t i = 1; i < m; ++i) st_stream(h + (uint64_t)i * pitch + col, hb);
    if (NBUF == 2) {
      const float4 vb = ld_stream(v + col);
      for (uint32_t i = 1; i < m; ++i) st_stream(v + (uint64_t)i * pitch + col, vb);
    }
  }
}

// ---- K2 without the exact average (Section 6 of the paper) -----------------------------------

// Every worker applies Eq. (2) and Eq. (3) to its own model: u, anchor and x are all
// [m, pitch] and the kernel is a plain elementwise stream, laid out like the local step
// (one block = one tile of one row). POLICY: 0 reset (h, v zeroed), 1 maintain.
template <int NBUF, int POLICY, int U>
__global__ void __launch_bounds__(kThreads)
outer_step_noaverage_kernel(const OuterArgs A) {
  const uint32_t row = blockIdx.x % A.m;
  const uint32_t tile = blockIdx.x / A.m;
  const uint32_t v0 = tile * (uint32_t)(kThreads * U) + threadIdx.x;
  const uint64_t roff = (uint64_t)row * A.pitch;
  float4 x[U], x0[U], u0[U];
  bool ok[U];
#pragma unroll
  for (int q = 0; q < U; ++q) {
    const uint32_t vi = v0 + q * kThreads;
    ok[q] = vi < A.nvec;
    if (ok[q]) {
      const uint64_t off = roff + 4ull * vi;
      x[q] = ld_stream(A.x + off);
      x0[q] = ld_stream(A.anchor + off);
      u0[q] = ld_stream(A.u + off);
    }
  }
#pragma unroll
  for (int q = 0; q < U; ++q) {
    if (!ok[q]) continue;
    float4 un, xn;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      // Eq. (2), (3) with the worker's own x_{t,tau} in place of the average
      const float ue = __fmaf_rn(A.beta, comp(u0[q], e), __fmul_rn(__fsub_rn(comp(x0[q], e), comp(x[q], e)), A.inv_gamma));
      comp(un, e) = ue;
      comp(xn, e) = __fmaf_rn(A.neg_alpha_gamma, ue, comp(x0[q], e));
    }
    const uint64_t off = roff + 4ull * (v0 + q * kThreads);
    st_stream(A.u + off, un);
    st_stream(A.anchor + off, xn);
    st_stream(A.x + off, xn);
    if (POLICY == 0) {
      const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
      st_stream(A.h + off, zero);
      if (NBUF == 2) st_stream(A.v + off, zero);
    }
  }
}

}  // namespace slowmo
