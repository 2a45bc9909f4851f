// K2 with the last inner step folded in: the base-optimizer step k = tau-1 of every worker
// (Table C.1 direction, Algorithm 1 update) is taken in registers and followed at once by
// the exact average, Eq. (2), Eq. (3), the broadcast and the buffer policy.
//
// Same arithmetic, in the same order, as local_step_kernel followed by
// outer_step_direct_kernel, so results are bit-identical; what disappears is one round trip
// of x (and of h, v when they are reset or averaged) through HBM: per parameter
//   separate: (20m + 4) + (8m + 16) + policy     fused: 20m + 16 + 4  (+8m for Adam's v)
// with policy = 0 / 4m nb / 8m nb bytes for maintain / reset / average.
#pragma once
#include "kernels.cuh"

#ifndef SLOWMO_FUSED_ROWS
#define SLOWMO_FUSED_ROWS 2        // rows in flight per thread (Nesterov; Adam uses half)
#endif
#ifndef SLOWMO_FUSED_MIN_BLOCKS
#define SLOWMO_FUSED_MIN_BLOCKS 4  // __launch_bounds__ minimum resident blocks per SM
#endif

namespace slowmo {

// Running sum over the workers in index order. The sum starts from -0, the one value for which
// s + v == v bit for bit whatever v is (signed zeros included), so the first worker needs no
// special case and the result equals x_0 + x_1 + ... added left to right.
__device__ __forceinline__ float4 ordered_sum_start() { return make_float4(-0.0f, -0.0f, -0.0f, -0.0f); }
__device__ __forceinline__ void add_in_order(float4 &s, const float4 &v) {
  const float2 lo = add2(make_float2(s.x, s.y), make_float2(v.x, v.y));
  const float2 hi = add2(make_float2(s.z, s.w), make_float2(v.z, v.w));
  s = make_float4(lo.x, lo.y, hi.x, hi.y);
}

__device__ __forceinline__ float4 div4(const float4 &s, float d) {
  return make_float4(__fdiv_rn(s.x, d), __fdiv_rn(s.y, d), __fdiv_rn(s.z, d), __fdiv_rn(s.w, d));
}

// One thread = one 4-element column group, all m rows. ROWS rows are loaded together.
// DERIVE: more rows than noise keys fit the kernel arguments; the warp derives them (RowKeys) and
// threads past the end of the row stay in the loop with their loads and stores switched off.
// LAZY: the broadcast and the reset / average of the buffers are left to the next local step
// (which then reads the anchor instead of the m rows): x rows are not written, "reset" writes
// nothing, "average" writes the means to row 0 only.
template <int BASE, int GRAD, int POLICY, int ROWS, bool LAZY, bool DERIVE>
__global__ void __launch_bounds__(kThreads, SLOWMO_FUSED_MIN_BLOCKS)
last_step_outer_kernel(const LocalArgs L, const OuterArgs O) {
  static_assert(32 % ROWS == 0, "key refills happen at multiples of 32 rows");
  const uint32_t vi = blockIdx.x * kThreads + threadIdx.x;
  if (!DERIVE && vi >= O.nvec) return;
  const bool ok = DERIVE ? vi < O.nvec : true;
  const uint64_t col = ok ? 4ull * vi : 0;
  const uint32_t m = O.m;

  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 x0 = a, u0 = a;
  if (ok) {
    x0 = ld_stream(O.anchor + col);
    u0 = ld_stream(O.u + col);
    if (GRAD == 0) a = ld_shared_row(L.a + col);
  }
  const uint64_t counter = noise_counter(L.vec0 + vi);
  RowKeys<DERIVE> keys;

  float4 sx = ordered_sum_start(), sh = sx, sv = sx;  // ordered sums over the workers
  for (uint32_t i0 = 0; i0 < m; i0 += ROWS) {
    if (GRAD == 0 && (i0 & 31u) == 0) keys.refill(L, i0 + (threadIdx.x & 31u));
    float4 x[ROWS], h[ROWS], v[ROWS], s[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      if (ok && i0 + q < m) {
        const uint64_t off = (uint64_t)(i0 + q) * O.pitch + col;
        x[q] = ld_stream(L.x + off);
        h[q] = ld_stream(L.h + off);
        if (BASE == 1) v[q] = ld_stream(L.v + off);
        s[q] = ld_stream(L.src + off);
        if (prefetch_on<BASE, GRAD>(SLOWMO_PREFETCH_FUSED) && i0 + q + ROWS < m) {
          const uint64_t nxt = off + (uint64_t)ROWS * O.pitch;
          prefetch_l2(L.x + nxt);
          prefetch_l2(L.h + nxt);
          if (BASE == 1) prefetch_l2(L.v + nxt);
          prefetch_l2(L.src + nxt);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < ROWS; ++q) {
      const uint32_t i = i0 + q;
      if (i >= m) break;
      uint64_t key = 0;
      if (GRAD == 0) key = keys.at(L, i, i);
      if (!ok) continue;
      float4 g;
      if (GRAD == 0) g = generated_gradient<true>(key, counter, a, x[q], s[q], L.sigma);
      else g = s[q];
      base_step4<BASE, GRAD == 0>(L, g, x[q], h[q], v[q]);
      add_in_order(sx, x[q]);
      if (POLICY == 1) {  // maintain: the stepped buffers go back to their rows
        const uint64_t off = (uint64_t)i * O.pitch + col;
        st_stream(L.h + off, h[q]);
        if (BASE == 1) st_stream(L.v + off, v[q]);
      } else if (POLICY == 2) {  // average
        add_in_order(sh, h[q]);
        if (BASE == 1) add_in_order(sv, v[q]);
      }
    }
  }

  if (!ok) return;
  const float4 xbar = div4(sx, O.m_float);
  float4 un, xn;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    // Eq. (2): u <- beta u + (x_{t,0} - xbar)/gamma ; Eq. (3): x_{t+1,0} <- x_{t,0} - alpha gamma u
    const float ue = __fmaf_rn(O.beta, comp(u0, e), __fmul_rn(__fsub_rn(comp(x0, e), comp(xbar, e)), O.inv_gamma));
    comp(un, e) = ue;
    comp(xn, e) = __fmaf_rn(O.neg_alpha_gamma, ue, comp(x0, e));
  }
  st_stream(O.u + col, un);
  st_stream(O.anchor + col, xn);
  if (!LAZY) store_rows(O.x + col, O.pitch, m, xn);
  if (POLICY == 0) {
    if (!LAZY) {
      const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
      store_rows(O.h + col, O.pitch, m, zero);
      if (BASE == 1) store_rows(O.v + col, O.pitch, m, zero);
    }
  } else if (POLICY == 2) {
    store_rows(O.h + col, O.pitch, LAZY ? 1u : m, div4(sh, O.m_float));
    if (BASE == 1) store_rows(O.v + col, O.pitch, LAZY ? 1u : m, div4(sv, O.m_float));
  }
}

template <int BASE, int GRAD, bool LAZY, bool DERIVE>
inline void launch_last_step_outer_keys(const LocalArgs &L, const OuterArgs &O, int policy, cudaStream_t stream) {
  const uint32_t blocks = (O.nvec + kThreads - 1) / kThreads;
  constexpr int ROWS = BASE == 1 ? SLOWMO_FUSED_ROWS / 2 : SLOWMO_FUSED_ROWS;
  switch (policy) {
    case 0: last_step_outer_kernel<BASE, GRAD, 0, ROWS, LAZY, DERIVE><<<blocks, kThreads, 0, stream>>>(L, O); break;
    case 1: last_step_outer_kernel<BASE, GRAD, 1, ROWS, LAZY, DERIVE><<<blocks, kThreads, 0, stream>>>(L, O); break;
    default: last_step_outer_kernel<BASE, GRAD, 2, ROWS, LAZY, DERIVE><<<blocks, kThreads, 0, stream>>>(L, O); break;
  }
}

template <int BASE, int GRAD, bool LAZY>
inline void launch_last_step_outer_policy(const LocalArgs &L, const OuterArgs &O, int policy, cudaStream_t stream) {
  // the row keys travel in the arguments up to kInlineKeys workers and are derived in the kernel beyond
  if (GRAD == 0 && L.m > kInlineKeys) launch_last_step_outer_keys<BASE, GRAD, LAZY, GRAD == 0>(L, O, policy, stream);
  else launch_last_step_outer_keys<BASE, GRAD, LAZY, false>(L, O, policy, stream);
}

template <bool LAZY>
inline void launch_last_step_outer_lazy(const LocalArgs &L, const OuterArgs &O, bool adam, bool generated, int policy,
                                        cudaStream_t stream) {
  if (adam) {
    if (generated) launch_last_step_outer_policy<1, 0, LAZY>(L, O, policy, stream);
    else launch_last_step_outer_policy<1, 1, LAZY>(L, O, policy, stream);
  } else {
    if (generated) launch_last_step_outer_policy<0, 0, LAZY>(L, O, policy, stream);
    else launch_last_step_outer_policy<0, 1, LAZY>(L, O, policy, stream);
  }
}

inline void launch_last_step_outer(const LocalArgs &L, const OuterArgs &O, bool adam, bool generated, int policy,
                                   bool lazy, cudaStream_t stream) {
  if (lazy) launch_last_step_outer_lazy<true>(L, O, adam, generated, policy, stream);
  else launch_last_step_outer_lazy<false>(L, O, adam, generated, policy, stream);
}

}  // namespace slowmo
