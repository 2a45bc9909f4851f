// Worker-sharded outer step for several GPUs: GPU r holds the replica rows of its own m_local
// workers (global workers r*m_local .. r*m_local + m_local - 1) and a full copy of the anchor and
// of u, as every worker does in the paper. The exact average of Algorithm 1 -- an AllReduce in
// the paper -- is done by ONE kernel per GPU over peer-mapped memory:
//   reduce-scatter  GPU g owns a contiguous slice of the columns; for those columns it loads
//                   the rows of ALL GPUs (peer loads) and adds them in global worker order;
//   update          Eq. (2), Eq. (3) on the slice;
//   all-gather      it stores the new anchor slice (and u, and the buffer policy's rows) into
//                   the rows and copies of ALL GPUs (peer stores).
// The sum runs in the same worker order as on one GPU, so the result is bit-identical to the
// single-GPU outer step. Only plain loads and stores touch peer memory (no bulk copies, no
// multicast). The kernels of different GPUs do not wait on one another: the caller orders them
// after every GPU's local steps and before anyone's next local step (a stream-ordered
// collective on each GPU's stream, or a host barrier).
#pragma once
#include "kernels.cuh"

namespace slowmo {

constexpr uint32_t kMaxShardGpus = 16;

struct ShardArgs {
  float *x[kMaxShardGpus], *h[kMaxShardGpus], *v[kMaxShardGpus];  // rows [m_local, pitch] of every GPU
  float *anchor[kMaxShardGpus], *u[kMaxShardGpus];                // every GPU's [pitch] copy
  uint64_t pitch;
  uint32_t world, rank, m_local;
  uint32_t vec_begin, vec_end;  // this GPU's slice of the 4-column groups
  float beta, inv_gamma, neg_alpha_gamma, m_float;
};

// Ordered mean over all world*m_local rows of one column group; the m_local rows of a GPU are
// loaded together.
__device__ __forceinline__ float4 sharded_row_mean(float *const *rows, const ShardArgs &A, uint64_t col) {
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  for (uint32_t r = 0; r < A.world; ++r) {
    const float *base = rows[r] + col;
    for (uint32_t i0 = 0; i0 < A.m_local; i0 += 4) {
      float4 t[4];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (i0 + q < A.m_local) t[q] = ld_stream(base + (uint64_t)(i0 + q) * A.pitch);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (i0 + q >= A.m_local) break;
        if (r == 0 && i0 + q == 0) {
          s = t[q];
        } else {
          s.x = __fadd_rn(s.x, t[q].x);
          s.y = __fadd_rn(s.y, t[q].y);
          s.z = __fadd_rn(s.z, t[q].z);
          s.w = __fadd_rn(s.w, t[q].w);
        }
      }
    }
  }
  return make_float4(__fdiv_rn(s.x, A.m_float), __fdiv_rn(s.y, A.m_float), __fdiv_rn(s.z, A.m_float),
                     __fdiv_rn(s.w, A.m_float));
}

__device__ __forceinline__ void sharded_store_rows(float *const *rows, const ShardArgs &A, uint64_t col, float4 val) {
  for (uint32_t r = 0; r < A.world; ++r) store_rows(rows[r] + col, A.pitch, A.m_local, val);
}

// NBUF buffers (1: h; 2: h, v); POLICY 0 reset, 1 maintain, 2 average.
template <int NBUF, int POLICY>
__global__ void __launch_bounds__(kThreads)
outer_step_sharded_kernel(const ShardArgs A) {
  const uint32_t vi = A.vec_begin + blockIdx.x * kThreads + threadIdx.x;
  if (vi >= A.vec_end) return;
  const uint64_t col = 4ull * vi;

  const float4 x0 = ld_stream(A.anchor[A.rank] + col);
  const float4 u0 = ld_stream(A.u[A.rank] + col);
  const float4 xbar = sharded_row_mean(A.x, A, col);
  float4 un, xn;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    // Eq. (2) and Eq. (3)
    const float ue = __fmaf_rn(A.beta, comp(u0, e), __fmul_rn(__fsub_rn(comp(x0, e), comp(xbar, e)), A.inv_gamma));
    comp(un, e) = ue;
    comp(xn, e) = __fmaf_rn(A.neg_alpha_gamma, ue, comp(x0, e));
  }
  for (uint32_t r = 0; r < A.world; ++r) {
    st_stream(A.u[r] + col, un);
    st_stream(A.anchor[r] + col, xn);
  }
  sharded_store_rows(A.x, A, col, xn);
  if (POLICY == 0) {
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    sharded_store_rows(A.h, A, col, zero);
    if (NBUF == 2) sharded_store_rows(A.v, A, col, zero);
  } else if (POLICY == 2) {
    sharded_store_rows(A.h, A, col, sharded_row_mean(A.h, A, col));
    if (NBUF == 2) sharded_store_rows(A.v, A, col, sharded_row_mean(A.v, A, col));
  }
}

// Column slice of GPU `rank`: contiguous, a whole number of 256-group blocks except the last.
inline void shard_slice(uint32_t nvec, uint32_t world, uint32_t rank, uint32_t *begin, uint32_t *end) {
  uint64_t chunk = ((uint64_t)nvec + world - 1) / world;
  chunk = (chunk + kThreads - 1) / kThreads * kThreads;
  const uint64_t b = chunk * rank, e = b + chunk;
  *begin = (uint32_t)(b < nvec ? b : nvec);
  *end = (uint32_t)(e < nvec ? e : nvec);
}

inline void launch_outer_sharded(const ShardArgs &A, int nbuf, int policy, cudaStream_t stream) {
  if (A.vec_end <= A.vec_begin) return;
  const uint32_t blocks = (A.vec_end - A.vec_begin + kThreads - 1) / kThreads;
#define SLOWMO_GO(NB, PO) outer_step_sharded_kernel<NB, PO><<<blocks, kThreads, 0, stream>>>(A)
  if (nbuf == 1) {
    if (policy == 0) SLOWMO_GO(1, 0); else if (policy == 1) SLOWMO_GO(1, 1); else SLOWMO_GO(1, 2);
  } else {
    if (policy == 0) SLOWMO_GO(2, 0); else if (policy == 1) SLOWMO_GO(2, 1); else SLOWMO_GO(2, 2);
  }
#undef SLOWMO_GO
}

}  // namespace slowmo
