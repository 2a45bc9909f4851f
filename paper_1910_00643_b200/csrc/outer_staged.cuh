// K2, staged variant: the fused outer step of Algorithm 1 (exact average, Eq. 2, Eq. 3,
// broadcast, buffer policy) with the replica rows moved by the bulk-copy engine (TMA).
//
// A persistent CTA (one per SM) owns column tiles of kTileCols = 4096 columns, i.e. 16 KB per row
// segment: a bare bulk-copy pipeline measured 6.1 TB/s with 4 KB copies and 6.56 TB/s with 16 KB
// ones (a plain vector copy: 6.8 TB/s), so the segments are made large and each consumer
// thread handles kSub column groups of a tile. For each tile a producer thread
// streams the m row segments (and, with the first of them, the anchor and u tiles) into a
// ring of shared-memory stages with
// cp.async.bulk (global -> shared, completion on an mbarrier); eight consumer warps add the
// rows in worker order, apply Eq. (2)/(3), put the new anchor tile in shared memory once and
// a store thread sends it to all m replica rows (and the anchor) with m+1 bulk stores
// (shared -> global); consumers and store thread hand tiles over through mbarriers, so no
// CTA-wide barrier sits in the loop. The buffer policy reuses the same machinery: "reset" bulk-stores a
// zero tile, "average" streams the h (and v) rows through the ring like x.
//
// No cluster multicast is used anywhere; every copy is CTA-local and starts on a 16-byte
// boundary (tile starts are multiples of kTileCols, pitch is a multiple of 4, tile widths
// are multiples of 4 elements).
//
// Every mbarrier wait is bounded. A wait that runs out records SLOWMO_ETIMEOUT data in the
// status block, raises a CTA-wide abort flag and the CTA finishes its loops without further
// copies or global writes, then waits (bounded) for the copies it still has in flight.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.cuh"

namespace slowmo {

#ifndef SLOWMO_STAGED_TILE_COLS
#define SLOWMO_STAGED_TILE_COLS 4096   // 16 KB per row segment: bulk copies of 4 KB top out near 6.1 TB/s
#endif
constexpr int kTileCols = SLOWMO_STAGED_TILE_COLS; // columns per tile
#ifndef SLOWMO_STAGED_ROWS
#define SLOWMO_STAGED_ROWS 2
#endif
#ifndef SLOWMO_STAGED_STAGES
#define SLOWMO_STAGED_STAGES 2
#endif
#ifndef SLOWMO_STAGED_CTAS
#define SLOWMO_STAGED_CTAS 1
#endif
constexpr int kStageRows = SLOWMO_STAGED_ROWS;     // row segments per pipeline stage
constexpr int kStages = SLOWMO_STAGED_STAGES;      // ring depth
#ifndef SLOWMO_STAGED_BULK_STORES
#define SLOWMO_STAGED_BULK_STORES 1  // 1: rows written by bulk copies from shared memory; 0: by vector stores
#endif
#ifndef SLOWMO_STAGED_OUT_BUFS
#define SLOWMO_STAGED_OUT_BUFS 3
#endif
constexpr int kOutBufs = SLOWMO_STAGED_OUT_BUFS;                        // output tiles in flight per CTA
constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kSub = kTileCols / (kConsumerThreads * 4);  // column groups per consumer thread and tile
static_assert(kSub >= 1 && kSub * kConsumerThreads * 4 == kTileCols, "tile must be a multiple of 1024 columns");
constexpr int kStagedThreads = kConsumerThreads + 64;  // + one load-producer warp + one store warp
constexpr uint32_t kWaitTries = 1u << 20;          // bound of every mbarrier wait
constexpr int kStagedCtasPerSm = SLOWMO_STAGED_CTAS;

constexpr int kAnchorSlot = kStageRows;            // extra slots of a stage: anchor and u tiles,
constexpr int kUSlot = kStageRows + 1;             // filled with the first row chunk of each tile

struct StagedSmem {
  float stage[kStages][kStageRows + 2][kTileCols];
  float out[kOutBufs][kTileCols];
  float zeros[kTileCols];
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long out_full[kOutBufs];   // consumers -> store thread: tile written
  unsigned long long out_empty[kOutBufs];  // store thread -> consumers: bulk stores have read the tile
  volatile int abort;
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns immediately once the CTA is aborting; on exhaustion records where.
__device__ __forceinline__ void mbar_wait(void *bar, uint32_t parity, volatile int *abort, int *status, int where) {
  if (*abort) return;
  for (uint32_t i = 0; i < kWaitTries; ++i)
    if (mbar_try_wait(bar, parity)) return;
  *abort = 1;
  if (atomicExch(status, 1) == 0) status[1] = where;
}
// global -> shared bulk copy, completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, uint32_t bytes, void *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst_smem)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}
// shared -> global bulk copy, tracked by the thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *dst, const void *src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_addr(src_smem)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// NBUF: base-optimizer buffers (1: h; 2: h, v). POLICY: 0 reset, 1 maintain, 2 average.
template <int NBUF, int POLICY>
__global__ void __launch_bounds__(kStagedThreads, kStagedCtasPerSm)
outer_step_staged_kernel(const OuterArgs A, int *status) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  StagedSmem &S = *reinterpret_cast<StagedSmem *>(smem_raw);

  const uint32_t tid = threadIdx.x;
  const uint32_t warp = tid >> 5;
  const uint64_t total_cols = 4ull * A.nvec;  // beyond 2^32 for the largest vectors: column offsets are 64-bit
  const uint32_t ntiles = (uint32_t)((total_cols + kTileCols - 1) / kTileCols);
  const uint32_t nchunks = (A.m + kStageRows - 1) / kStageRows;
  constexpr int kPasses = POLICY == 2 ? 1 + NBUF : 1;  // x, then h (and v) when averaging

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&S.full[s], 1);
      mbar_init(&S.empty[s], kConsumerWarps);
    }
    for (int b = 0; b < kOutBufs; ++b) {
      mbar_init(&S.out_full[b], kConsumerWarps);
      mbar_init(&S.out_empty[b], 1);
    }
    S.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (uint32_t i = tid; i < kTileCols; i += kStagedThreads) S.zeros[i] = 0.0f;
  fence_async_proxy();  // zeros are read by bulk stores
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ---------------- producer warp: feeds the ring, one lane per row segment ----------------
    const uint32_t lane = tid & 31u;
    uint32_t job = 0, issued = 0;  // issued: jobs whose copies were started
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      const uint64_t col0 = (uint64_t)tile * kTileCols;
      const uint32_t ncols = (uint32_t)min((uint64_t)kTileCols, total_cols - col0);
      for (int pass = 0; pass < kPasses; ++pass) {
        const float *src = pass == 0 ? A.x : (pass == 1 ? A.h : A.v);
        for (uint32_t c = 0; c < nchunks; ++c, ++job) {
          const uint32_t st = job % kStages, round = job / kStages;
          if (lane == 0) mbar_wait(&S.empty[st], (round & 1u) ^ 1u, &S.abort, status, 1);
          __syncwarp();
          if (S.abort) continue;
          issued = job + 1;
          const uint32_t r0 = c * kStageRows;
          const uint32_t rows = min((uint32_t)kStageRows, A.m - r0);
          const bool first = pass == 0 && c == 0;  // this chunk also brings the anchor and u tiles
          if (lane == 0) mbar_expect_tx(&S.full[st], (rows + (first ? 2u : 0u)) * ncols * 4u);
          if (lane < rows)
            bulk_load(&S.stage[st][lane][0], src + (uint64_t)(r0 + lane) * A.pitch + col0, ncols * 4u, &S.full[st]);
          if (first && lane == kAnchorSlot) bulk_load(&S.stage[st][kAnchorSlot][0], A.anchor + col0, ncols * 4u, &S.full[st]);
          if (first && lane == kUSlot) bulk_load(&S.stage[st][kUSlot][0], A.u + col0, ncols * 4u, &S.full[st]);
        }
      }
    }
    // copies still in flight must land before the shared memory is given back
    if (S.abort && lane == 0) {
      for (uint32_t j = issued > (uint32_t)kStages ? issued - kStages : 0; j < issued; ++j)
        for (uint32_t i = 0; i < kWaitTries; ++i)
          if (mbar_try_wait(&S.full[j % kStages], (j / kStages) & 1u)) break;
    }
  } else if (warp < kConsumerWarps) {
    // ---------------- consumers ----------------
    // thread tid owns the column groups tid + k*kConsumerThreads (k < kSub) of the tile
    uint32_t job = 0, outs = 0;
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      const uint64_t col0 = (uint64_t)tile * kTileCols;
      const uint32_t ncols = (uint32_t)min((uint64_t)kTileCols, total_cols - col0);
      float4 x0[kSub], u0[kSub];

      for (int pass = 0; pass < kPasses; ++pass) {
        // ordered sum over the workers, chunk by chunk
        float4 s[kSub];
        for (uint32_t c = 0; c < nchunks; ++c, ++job) {
          const uint32_t st = job % kStages, round = job / kStages;
          mbar_wait(&S.full[st], round & 1u, &S.abort, status, 2);
          const uint32_t rows = min((uint32_t)kStageRows, A.m - c * kStageRows);
#pragma unroll
          for (int k = 0; k < kSub; ++k) {
            const uint32_t lc = (tid + k * kConsumerThreads) * 4u;  // column inside the tile
            if (lc >= ncols) continue;
            if (pass == 0 && c == 0) {
              x0[k] = *reinterpret_cast<const float4 *>(&S.stage[st][kAnchorSlot][lc]);
              u0[k] = *reinterpret_cast<const float4 *>(&S.stage[st][kUSlot][lc]);
            }
#pragma unroll
            for (int r = 0; r < kStageRows; ++r) {
              if ((uint32_t)r < rows) {
                const float4 v = *reinterpret_cast<const float4 *>(&S.stage[st][r][lc]);
                if (c == 0 && r == 0) {
                  s[k] = v;
                } else {
                  s[k].x = __fadd_rn(s[k].x, v.x);
                  s[k].y = __fadd_rn(s[k].y, v.y);
                  s[k].z = __fadd_rn(s[k].z, v.z);
                  s[k].w = __fadd_rn(s[k].w, v.w);
                }
              }
            }
          }
          __syncwarp();
          if ((tid & 31) == 0) mbar_arrive(&S.empty[st]);
        }

        // the tile goes to shared memory once; the store warp sends it to every row
        const uint32_t ob = outs % kOutBufs, oround = outs / kOutBufs;
        ++outs;
#if SLOWMO_STAGED_BULK_STORES
        mbar_wait(&S.out_empty[ob], (oround & 1u) ^ 1u, &S.abort, status, 3);
#endif
#pragma unroll
        for (int k = 0; k < kSub; ++k) {
          const uint32_t lc = (tid + k * kConsumerThreads) * 4u;
          if (lc >= ncols) continue;
          const uint64_t col = col0 + lc;
          const float4 mean = make_float4(__fdiv_rn(s[k].x, A.m_float), __fdiv_rn(s[k].y, A.m_float),
                                          __fdiv_rn(s[k].z, A.m_float), __fdiv_rn(s[k].w, A.m_float));
          float4 outv = mean;  // passes 1, 2: averaged buffer
          if (pass == 0) {
            float4 un;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // Eq. (2) and Eq. (3)
              const float ue =
                  __fmaf_rn(A.beta, comp(u0[k], e), __fmul_rn(__fsub_rn(comp(x0[k], e), comp(mean, e)), A.inv_gamma));
              comp(un, e) = ue;
              comp(outv, e) = __fmaf_rn(A.neg_alpha_gamma, ue, comp(x0[k], e));
            }
            if (!S.abort) st_stream(A.u + col, un);
          }
#if SLOWMO_STAGED_BULK_STORES
          *reinterpret_cast<float4 *>(&S.out[ob][lc]) = outv;
#else
          if (!S.abort) {
            float *dst = pass == 0 ? A.x : (pass == 1 ? A.h : A.v);
            store_rows(dst + col, A.pitch, A.m, outv);
            if (pass == 0) {
              st_stream(A.anchor + col, outv);
              if (POLICY == 0) {
                const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
                store_rows(A.h + col, A.pitch, A.m, zero);
                if (NBUF == 2) store_rows(A.v + col, A.pitch, A.m, zero);
              }
            }
          }
#endif
        }
#if SLOWMO_STAGED_BULK_STORES
        fence_async_proxy();
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(&S.out_full[ob]);
#endif
      }
    }
  } else if (SLOWMO_STAGED_BULK_STORES && warp == kConsumerWarps + 1) {
    // ---------------- store warp: output tiles -> all rows, lanes share the rows ----------------
    const uint32_t lane = tid & 31u;
    uint32_t outs = 0;
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      const uint64_t col0 = (uint64_t)tile * kTileCols;
      const uint32_t ncols = (uint32_t)min((uint64_t)kTileCols, total_cols - col0);
      for (int pass = 0; pass < kPasses; ++pass, ++outs) {
        const uint32_t ob = outs % kOutBufs, oround = outs / kOutBufs;
        if (lane == 0) mbar_wait(&S.out_full[ob], oround & 1u, &S.abort, status, 4);
        __syncwarp();
        if (!S.abort) {
          float *dst = pass == 0 ? A.x : (pass == 1 ? A.h : A.v);
          for (uint32_t i = lane; i < A.m; i += 32) {
            bulk_store(dst + (uint64_t)i * A.pitch + col0, &S.out[ob][0], ncols * 4u);
            if (pass == 0 && POLICY == 0) {  // reset: zero tiles to every buffer row
              bulk_store(A.h + (uint64_t)i * A.pitch + col0, &S.zeros[0], ncols * 4u);
              if (NBUF == 2) bulk_store(A.v + (uint64_t)i * A.pitch + col0, &S.zeros[0], ncols * 4u);
            }
          }
          if (pass == 0 && lane == 31) bulk_store(A.anchor + col0, &S.out[ob][0], ncols * 4u);
        }
        bulk_commit();
        // every lane waits for its own groups: all but the newest kOutBufs-1 have been read out
        // of shared memory, so the tile written kOutBufs-1 outputs ago can be overwritten
        bulk_wait_read<kOutBufs - 1>();
        __syncwarp();
        if (lane == 0 && outs + 1 >= (uint32_t)kOutBufs) mbar_arrive(&S.out_empty[(outs + 1) % kOutBufs]);
      }
    }
    bulk_wait_all();
  }
  __syncthreads();
}

// Test hook for the bounded-wait path: one CTA waits on an mbarrier that nothing ever
// completes, with the same try loop as the pipeline (bound given by the caller), records the
// timeout in the status block and returns. The context stays usable.
__global__ void bounded_wait_probe_kernel(int *status, uint32_t tries) {
  __shared__ unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool done = false;
    for (uint32_t i = 0; i < tries && !done; ++i) done = mbar_try_wait(&bar, 0);
    if (!done && atomicExch(status, 1) == 0) status[1] = 99;
  }
}

inline cudaError_t outer_staged_configure() {
  const int bytes = (int)sizeof(StagedSmem);
  cudaError_t e = cudaSuccess;
#define SLOWMO_SET(NB, PO)                                                                                     \
  if (e == cudaSuccess)                                                                                        \
    e = cudaFuncSetAttribute(outer_step_staged_kernel<NB, PO>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  SLOWMO_SET(1, 0) SLOWMO_SET(1, 1) SLOWMO_SET(1, 2) SLOWMO_SET(2, 0) SLOWMO_SET(2, 1) SLOWMO_SET(2, 2)
#undef SLOWMO_SET
  return e;
}

inline void launch_outer_staged(const OuterArgs &A, int nbuf, int policy, int num_sms, int *status,
                                cudaStream_t stream) {
  const uint32_t ntiles = (uint32_t)((4ull * A.nvec + kTileCols - 1) / kTileCols);
  uint32_t grid = (uint32_t)num_sms * kStagedCtasPerSm;
  if (grid > ntiles) grid = ntiles;
  const size_t bytes = sizeof(StagedSmem);
#define SLOWMO_GO(NB, PO) outer_step_staged_kernel<NB, PO><<<grid, kStagedThreads, bytes, stream>>>(A, status)
  if (nbuf == 1) {
    if (policy == 0) SLOWMO_GO(1, 0); else if (policy == 1) SLOWMO_GO(1, 1); else SLOWMO_GO(1, 2);
  } else {
    if (policy == 0) SLOWMO_GO(2, 0); else if (policy == 1) SLOWMO_GO(2, 1); else SLOWMO_GO(2, 2);
  }
#undef SLOWMO_GO
}

}  // namespace slowmo
