// argus_common.cuh — device helpers shared by the kernels of the CUDA library (sm_100a).
#ifndef ARGUS_COMMON_CUH_
#define ARGUS_COMMON_CUH_

#include <cuda_runtime.h>
#include <stdint.h>

#include "argus.h"
#include "argus_testing.h"

typedef unsigned long long u64;
typedef unsigned int u32;

static_assert(sizeof(argus_event_t) == 16, "event layout");
static_assert(sizeof(argus_interval_t) == 48, "interval layout");
static_assert(sizeof(argus_ambiguity_t) == 32, "ambiguity layout");
static_assert(sizeof(argus_agg_t) == 576, "aggregate layout");
static_assert(sizeof(argus_overlap_t) == 32, "overlap layout");
static_assert(sizeof(argus_status_t) == 64, "status layout");

#define ARGUS_CUDA_TRY(expr)                          \
  do {                                                \
    cudaError_t e__ = (expr);                         \
    if (e__ != cudaSuccess) return ARGUS_ERR_CUDA;    \
  } while (0)

// host-side bookkeeping implemented in argus_api.cu
void argus_count_launch();                                      // one more kernel launched by this library
void argus_prof_mark(int slot, cudaStream_t stream, int end);   // CUDA events around a dominant kernel (if enabled)
void argus_prof_suppress(int delta);                            // +1 / -1: event recording off while > 0 (it creates events)
enum { ARGUS_PROF_PAIR = 0, ARGUS_PROF_AGGREGATE = 1, ARGUS_PROF_OVERLAP = 2, ARGUS_PROF_SLOTS = 4 };

#define ARGUS_CHECK_LAUNCH()                                      \
  do {                                                            \
    if (cudaGetLastError() != cudaSuccess) return ARGUS_ERR_CUDA; \
    argus_count_launch();                                         \
  } while (0)

static inline size_t argus_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// First device-side error wins; the winner also records where it happened.
__device__ __forceinline__ void argus_set_error(argus_status_t* st, u32 code, u32 stream, u64 event) {
  if (atomicCAS(&st->code, 0u, code) == 0u) {
    st->bad_stream = stream;
    st->bad_event = event;
  }
}

// Exclusive prefix sum over the threads of a block (blockDim.x <= 1024, multiple of 32).
// `warp_sums` is shared scratch of >= 33 elements. Returns the exclusive prefix of `v`;
// *total receives the block total. Contains __syncthreads().
template <typename T>
__device__ __forceinline__ T argus_block_exclusive_scan(T v, T* warp_sums, T* total) {
  const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  T incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    T o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= (u32)d) incl += o;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    T w = lane < nwarps ? warp_sums[lane] : T(0);
    T wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      T o = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= (u32)d) wi += o;
    }
    warp_sums[lane] = wi - w;  // exclusive prefix of warp sums
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  const T base = warp_sums[warp];
  *total = warp_sums[32];
  __syncthreads();
  return base + incl - v;
}

#endif  // ARGUS_COMMON_CUH_
