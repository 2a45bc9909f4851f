// K1 for the stochastic-gradient-push base optimizers (Algorithm 2; Table C.1, SGP rows):
// the local step of every worker followed by the push-sum mixing of that step, in one pass.
//
// Graph: time-varying directed exponential graph, one peer per step: worker i keeps half of
// (x_{k+1/2}, w) and pushes half to worker (i + hops) mod m, hops = 2^q. With one out-peer and
// one in-peer per worker the mixing matrix is doubly stochastic, so the push-sum weights w
// stay exactly 1 from their initial value 1 and the de-biased z = x / w is x bit for bit: the
// kernel carries no w and evaluates the gradient at x.
//
// One thread owns a 4-column group of ALL m rows: it walks the rows once doing the local step
// (same arithmetic as local_step_kernel), keeps each row's x_{k+1/2} in its private column of
// a shared-memory tile (no thread reads another thread's column, so no barrier), then walks
// the rows again writing x_i = 1/2 x_{k+1/2,i} + 1/2 x_{k+1/2,i-hops}. HBM traffic is the
// same 20 (28 for Adam) bytes per update as the communication-free step.
#pragma once
#include "kernels.cuh"

#ifndef SLOWMO_SGP_ROWS
#define SLOWMO_SGP_ROWS 4       // rows loaded together (Nesterov; Adam uses half)
#endif

namespace slowmo {
constexpr int kSgpRows = SLOWMO_SGP_ROWS;

constexpr uint32_t kSgpMaxWorkers = 64;

inline uint32_t sgp_block_threads(uint32_t m) { return m <= 48 ? 128u : 64u; }  // m * threads * 16 B <= 96 KB

template <int BASE, int GRAD, int ROWS>
__global__ void __launch_bounds__(128)
sgp_step_kernel(const LocalArgs L, uint32_t hops) {
  extern __shared__ float4 x_half[];  // [m][blockDim.x]
  const uint32_t bd = blockDim.x, tid = threadIdx.x;
  const uint32_t vi = blockIdx.x * bd + tid;
  if (vi >= L.nvec) return;
  const uint64_t col = 4ull * vi;
  const uint32_t m = L.m;

  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  if (GRAD == 0) a = ld_shared_row(L.a + col);

  for (uint32_t i0 = 0; i0 < m; i0 += ROWS) {
    float4 x[ROWS], h[ROWS], v[ROWS], s[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      if (i0 + q < m) {
        const uint64_t off = (uint64_t)(i0 + q) * L.pitch + col;
        x[q] = ld_stream(L.x + off);
        h[q] = ld_stream(L.h + off);
        if (BASE == 1) v[q] = ld_stream(L.v + off);
        s[q] = ld_stream(L.src + off);
      }
    }
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      const uint32_t i = i0 + q;
      if (i >= m) break;
      float4 g;
      if (GRAD == 0) {
        const uint64_t st = L.keys[i] + kGoldenGamma * (2ull * (L.vec0 + vi) + 1);
        float4 z;
        word_to_normal_pair(mix64(st), z.x, z.y);
        word_to_normal_pair(mix64(st + kGoldenGamma), z.z, z.w);
#pragma unroll
        for (int e = 0; e < 4; ++e)
          comp(g, e) = __fmaf_rn(comp(a, e), __fsub_rn(comp(x[q], e), comp(s[q], e)), __fmul_rn(L.sigma, comp(z, e)));
      } else {
        g = s[q];
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) base_step<BASE>(L, comp(g, e), comp(x[q], e), comp(h[q], e), comp(v[q], e));
      const uint64_t off = (uint64_t)i * L.pitch + col;
      st_stream(L.h + off, h[q]);
      if (BASE == 1) st_stream(L.v + off, v[q]);
      x_half[i * bd + tid] = x[q];
    }
  }

  // push-sum mixing: keep half, receive half from the worker `hops` places back
  const uint32_t back = m - hops % m;
  for (uint32_t i = 0; i < m; ++i) {
    const uint32_t from = (i + back) % m;
    const float4 own = x_half[i * bd + tid], got = x_half[from * bd + tid];
    float4 xn;
    xn.x = __fadd_rn(__fmul_rn(0.5f, own.x), __fmul_rn(0.5f, got.x));
    xn.y = __fadd_rn(__fmul_rn(0.5f, own.y), __fmul_rn(0.5f, got.y));
    xn.z = __fadd_rn(__fmul_rn(0.5f, own.z), __fmul_rn(0.5f, got.z));
    xn.w = __fadd_rn(__fmul_rn(0.5f, own.w), __fmul_rn(0.5f, got.w));
    st_stream(L.x + (uint64_t)i * L.pitch + col, xn);
  }
}

inline cudaError_t sgp_configure() {
  const int bytes = 96 * 1024;
  cudaError_t e = cudaSuccess;
#define SLOWMO_SET(B, G, R)                                                                             \
  if (e == cudaSuccess)                                                                                 \
    e = cudaFuncSetAttribute(sgp_step_kernel<B, G, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  SLOWMO_SET(0, 0, kSgpRows) SLOWMO_SET(0, 1, kSgpRows) SLOWMO_SET(1, 0, kSgpRows / 2) SLOWMO_SET(1, 1, kSgpRows / 2)
#undef SLOWMO_SET
  return e;
}

inline void launch_sgp_step(const LocalArgs &L, uint32_t hops, bool adam, bool generated, cudaStream_t stream) {
  const uint32_t bd = sgp_block_threads(L.m);
  const uint32_t blocks = (L.nvec + bd - 1) / bd;
  const size_t smem = (size_t)L.m * bd * sizeof(float4);
  if (adam) {
    if (generated) sgp_step_kernel<1, 0, kSgpRows / 2><<<blocks, bd, smem, stream>>>(L, hops);
    else sgp_step_kernel<1, 1, kSgpRows / 2><<<blocks, bd, smem, stream>>>(L, hops);
  } else {
    if (generated) sgp_step_kernel<0, 0, kSgpRows><<<blocks, bd, smem, stream>>>(L, hops);
    else sgp_step_kernel<0, 1, kSgpRows><<<blocks, bd, smem, stream>>>(L, hops);
  }
}

// Hop distance 2^q at global base-optimizer step s: q cycles through 0 .. floor(log2(m-1)).
inline uint32_t sgp_hops(uint32_t m, uint64_t s) {
  if (m < 2) return 0;
  uint32_t nq = 0;
  for (uint32_t r = m - 1; r > 0; r >>= 1) ++nq;
  return 1u << (uint32_t)(s % nq);
}

}  // namespace slowmo
