// K1 for the stochastic-gradient-push base optimizers (Algorithm 2; Table C.1, SGP rows):
// the local step of every worker followed by the push-sum mixing of that step, in one pass.
//
// Graph: time-varying directed exponential graph, one peer per step: worker i keeps half of
// (x_{k+1/2}, w) and pushes half to worker (i + hops) mod m, hops = 2^q. With one out-peer and
// one in-peer per worker the mixing matrix is doubly stochastic, so the push-sum weights w
// stay exactly 1 from their initial value 1 and the de-biased z = x / w is x bit for bit: the
// kernel carries no w and evaluates the gradient at x.
//
// One thread owns a 4-column group of ALL m rows (column-owner layout). The mixing
// x_i = 1/2 x_{k+1/2,i} + 1/2 x_{k+1/2,i-hops} couples row i with row i-hops only, so the
// thread visits the rows along the cycles of i -> i+hops (gcd(m, hops) cycles of length
// m / gcd): the half-step value of the previous row of the walk is still in registers when
// the current row needs it, and the first row of a cycle is closed when the walk returns to
// it. No shared memory, no second pass; HBM traffic is the same 20 (28 for Adam) bytes per
// update as the communication-free step.
#pragma once
#include "kernels.cuh"

#ifndef SLOWMO_SGP_ROWS
#define SLOWMO_SGP_ROWS 2       // rows loaded together (Nesterov; Adam uses half)
#endif

namespace slowmo {
constexpr int kSgpRows = SLOWMO_SGP_ROWS;

__device__ __forceinline__ float4 half_sum(const float4 &p, const float4 &q) {
  return make_float4(__fadd_rn(__fmul_rn(0.5f, p.x), __fmul_rn(0.5f, q.x)), __fadd_rn(__fmul_rn(0.5f, p.y), __fmul_rn(0.5f, q.y)),
                     __fadd_rn(__fmul_rn(0.5f, p.z), __fmul_rn(0.5f, q.z)), __fadd_rn(__fmul_rn(0.5f, p.w), __fmul_rn(0.5f, q.w)));
}

// `cycles` = gcd(m, hops), `len` = m / cycles (host-computed); hops < m, or hops = 0 with m = 1.
// DERIVE: more workers than noise keys fit the kernel arguments; the warp derives the keys along
// the walk (RowKeys), 32 positions of a cycle at a time, and no thread leaves the loop early.
template <int BASE, int GRAD, int ROWS, bool DERIVE>
__global__ void __launch_bounds__(kThreads, 3)
sgp_step_kernel(const LocalArgs L, uint32_t hops, uint32_t cycles, uint32_t len) {
  static_assert(32 % ROWS == 0, "key refills happen at multiples of 32 positions");
  const uint32_t vi = blockIdx.x * kThreads + threadIdx.x;
  if (!DERIVE && vi >= L.nvec) return;
  const bool ok = DERIVE ? vi < L.nvec : true;
  const uint64_t col = ok ? 4ull * vi : 0;
  const uint32_t m = L.m;

  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  if (GRAD == 0 && ok) a = ld_shared_row(L.a + col);
  const uint64_t counter = noise_counter(L.vec0 + vi);
  RowKeys<DERIVE> keys;

  for (uint32_t c = 0; c < cycles; ++c) {
    // walk the cycle c, c+hops, c+2 hops, ... ; `prev` is x_{k+1/2} of the row visited before
    float4 first = a, prev = a;
    uint32_t row = c;
    for (uint32_t n0 = 0; n0 < len; n0 += ROWS) {
      // position n0 + l of the walk is row (row + l hops) mod m
      if (GRAD == 0 && (n0 & 31u) == 0)
        keys.refill(L, (uint32_t)(((uint64_t)row + (uint64_t)(threadIdx.x & 31u) * hops) % m));
      float4 x[ROWS], h[ROWS], v[ROWS], s[ROWS];
      uint32_t rows[ROWS];
      uint32_t r = row;
#pragma unroll
      for (int q = 0; q < ROWS; ++q) {
        rows[q] = r;
        if (ok && n0 + q < len) {
          const uint64_t off = (uint64_t)r * L.pitch + col;
          x[q] = ld_stream(L.x + off);
          h[q] = ld_stream(L.h + off);
          if (BASE == 1) v[q] = ld_stream(L.v + off);
          s[q] = ld_stream(L.src + off);
        }
        r += hops;
        if (r >= m) r -= m;
      }
      row = r;
#pragma unroll
      for (int q = 0; q < ROWS; ++q) {
        if (n0 + q >= len) break;
        const uint32_t i = rows[q];
        uint64_t key = 0;
        if (GRAD == 0) key = keys.at(L, n0 + q, i);
        if (!ok) continue;
        float4 g;
        // packed arithmetic (bit-identical, fewer instructions): with the walk's bookkeeping on top of the
        // generator this kernel is co-bound by instruction issue; measured 2.61 -> 2.49 ms per launch at
        // m = 32 (Nesterov) and 7.32 -> 7.22 ms at m = 8, P = 2.1e8 (Adam)
        if (GRAD == 0) g = generated_gradient<true>(key, counter, a, x[q], s[q], L.sigma);
        else g = s[q];
        base_step4<BASE, GRAD == 0>(L, g, x[q], h[q], v[q]);
        const uint64_t off = (uint64_t)i * L.pitch + col;
        st_stream(L.h + off, h[q]);
        if (BASE == 1) st_stream(L.v + off, v[q]);
        if (n0 + q == 0) {
          first = x[q];  // its in-neighbour is the last row of the walk
        } else {
          st_stream(L.x + off, half_sum(x[q], prev));  // keep half, receive half from the row hops back
        }
        prev = x[q];
      }
    }
    if (ok) st_stream(L.x + (uint64_t)c * L.pitch + col, half_sum(first, prev));
  }
}

inline uint32_t sgp_gcd(uint32_t p, uint32_t q) {
  while (q) {
    const uint32_t t = p % q;
    p = q;
    q = t;
  }
  return p;
}

inline void launch_sgp_step(const LocalArgs &L, uint32_t hops, bool adam, bool generated, cudaStream_t stream) {
  const uint32_t blocks = (L.nvec + kThreads - 1) / kThreads;
  hops = L.m > 1 ? hops % L.m : 0;
  const uint32_t cycles = hops ? sgp_gcd(L.m, hops) : L.m;  // hops = 0: every row is its own cycle (x unchanged)
  const uint32_t len = L.m / cycles;
  const bool derive = generated && L.m > kInlineKeys;  // keys no longer fit the kernel arguments
  if (adam) {
    if (derive) sgp_step_kernel<1, 0, kSgpRows / 2, true><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
    else if (generated) sgp_step_kernel<1, 0, kSgpRows / 2, false><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
    else sgp_step_kernel<1, 1, kSgpRows / 2, false><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
  } else {
    if (derive) sgp_step_kernel<0, 0, kSgpRows, true><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
    else if (generated) sgp_step_kernel<0, 0, kSgpRows, false><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
    else sgp_step_kernel<0, 1, kSgpRows, false><<<blocks, kThreads, 0, stream>>>(L, hops, cycles, len);
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
