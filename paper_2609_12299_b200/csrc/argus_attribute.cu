// argus_attribute.cu — PC-to-region mapping counts and ambiguity-aware attribution.
//
//   k_map_counts   : exec records of a mapping-run trace arrive as intervals of the extra region id R whose
//                    parent_region is the innermost active region (pairing did the stack work); this pass adds
//                    their execution counts into counts[owner][pc] (integer atomics: order does not matter).
//   k_attr_columns : one thread per PC: column total, alpha, entropy;
//   k_attr_rows    : one block per (row, chunk of PCs): the lifted metric summed in a fixed order;
//   k_attr_finish  : mhat[row] = sum of the chunk partials, in chunk order.
#include "argus_common.cuh"

namespace {

constexpr int kAttrThreads = 256;
constexpr u32 kAttrChunk = 8192;      // PCs one block of the row pass covers
constexpr u32 kMapSlots = 2048;       // shared-memory cache of (owner, pc) cells per block
constexpr u32 kMapEmpty = 0xffffffffu;

// 64-bit add as native 32-bit shared atomics; each carry is propagated exactly once
__device__ __forceinline__ void shared_add64(u64* p64, u64 v) {
  u32* p = reinterpret_cast<u32*>(p64);
  const u32 lo = (u32)v, hi = (u32)(v >> 32);
  if (lo) {
    const u32 old = atomicAdd(p, lo);
    if (old + lo < old) atomicAdd(p + 1, 1u);
  }
  if (hi) atomicAdd(p + 1, hi);
}

// A mapping run touches few of the (R + 1) x P cells and touches them very often, so each block gathers
// its additions in a small direct-mapped table in shared memory (cell index -> sum) and adds the table
// to the global counts at the end; a cell whose slot is taken by another cell goes to the global counts directly.
__global__ void __launch_bounds__(256) k_map_counts(const argus_interval_t* intervals, const u64* interval_offsets,
                                                    u32 num_streams, u32 exec_region, u32 num_pcs, u64* counts,
                                                    argus_status_t* status, int use_cache) {
  __shared__ u32 keys[kMapSlots];
  __shared__ u64 sums[kMapSlots];
  for (u32 i = threadIdx.x; i < kMapSlots; i += blockDim.x) { keys[i] = kMapEmpty; sums[i] = 0; }
  __syncthreads();
  const u64 lo = interval_offsets[0], hi = interval_offsets[num_streams];
  for (u64 i = lo + (u64)blockIdx.x * blockDim.x + threadIdx.x; i < hi; i += (u64)gridDim.x * blockDim.x) {
    const uint4* p = reinterpret_cast<const uint4*>(intervals + i);
    const uint4 q1 = __ldg(p + 1);
    if (q1.z != exec_region) continue;
    const u32 pc = q1.w;
    if (pc >= num_pcs) { argus_set_error(status, ARGUS_ERR_INVALID_ARG, 0, i); continue; }
    const uint4 q0 = __ldg(p), q2 = __ldg(p + 2);
    const u64 k = (u64)q0.z | ((u64)q0.w << 32);
    if (!k) continue;
    const u32 owner = q2.y < exec_region ? q2.y : exec_region;  // no parent, or a malformed nesting of exec records
    const u64 cell = (u64)owner * num_pcs + pc;
    if (use_cache) {
      const u32 key = (u32)cell;
      const u32 slot = (key * 2654435761u) >> 21;  // 11 bits
      const u32 old = atomicCAS(&keys[slot], kMapEmpty, key);
      if (old == kMapEmpty || old == key) { shared_add64(&sums[slot], k); continue; }
    }
    atomicAdd(counts + cell, k);
  }
  __syncthreads();
  for (u32 i = threadIdx.x; i < kMapSlots; i += blockDim.x)
    if (keys[i] != kMapEmpty && sums[i]) atomicAdd(counts + keys[i], sums[i]);
}

// One thread per PC: column total (kept for the row pass), alpha, entropy.
__global__ void __launch_bounds__(kAttrThreads) k_attr_columns(const u64* counts, u32 num_rows, u32 num_pcs,
                                                               double* entropy, double* alpha, u64* totals) {
  const u32 p = blockIdx.x * kAttrThreads + threadIdx.x;
  if (p >= num_pcs) return;
  u64 total = 0;
  for (u32 r = 0; r < num_rows; ++r) total += counts[(size_t)r * num_pcs + p];
  totals[p] = total;
  double h = 0.0;
  for (u32 r = 0; r < num_rows; ++r) {
    const u64 n = counts[(size_t)r * num_pcs + p];
    const double a = (total == 0 || n == 0) ? 0.0 : (double)n / (double)total;
    if (alpha) alpha[(size_t)r * num_pcs + p] = a;
    if (a > 0.0) h -= a * log(a);
  }
  entropy[p] = h;
}

// Block (chunk c, row r): sum over the chunk's PCs of alpha * metric, every thread in index order, then the
// threads by a fixed tree: the same bits every run.
__global__ void __launch_bounds__(kAttrThreads) k_attr_rows(const u64* counts, const u64* totals, u32 num_rows, u32 num_pcs,
                                                            const double* metric, u32 num_chunks, double* partial) {
  __shared__ double sh[kAttrThreads / 32];
  const u32 r = blockIdx.y, c = blockIdx.x;
  const u32 p0 = c * kAttrChunk, p1 = p0 + kAttrChunk < num_pcs ? p0 + kAttrChunk : num_pcs;
  double acc = 0.0;
  for (u32 p = p0 + threadIdx.x; p < p1; p += kAttrThreads) {
    const u64 n = counts[(size_t)r * num_pcs + p], total = totals[p];
    if (n && total) acc += ((double)n / (double)total) * metric[p];
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, d);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kAttrThreads / 32; ++w) s += sh[w];
    partial[(size_t)r * num_chunks + c] = s;
  }
}

__global__ void __launch_bounds__(256) k_attr_finish(const double* partial, u32 num_chunks, u32 num_rows, double* mhat) {
  const u32 r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= num_rows) return;
  double s = 0.0;
  for (u32 c = 0; c < num_chunks; ++c) s += partial[(size_t)r * num_chunks + c];
  mhat[r] = s;
}

struct AttrLayout { size_t totals, partial, total; u32 chunks; };

AttrLayout attr_layout(uint32_t num_rows, uint32_t num_pcs) {
  AttrLayout L;
  L.chunks = (num_pcs + kAttrChunk - 1) / kAttrChunk;
  L.totals = 0;
  L.partial = argus_align_up((size_t)num_pcs * 8, 256);
  L.total = L.partial + argus_align_up((size_t)num_rows * L.chunks * 8 + 8, 256);
  return L;
}

}  // namespace

extern "C" int argus_map_pc_counts(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                                   uint32_t num_streams, uint32_t exec_region, uint32_t num_pcs, uint64_t* counts,
                                   argus_status_t* status, void* cuda_stream) {
  if (!interval_offsets || !counts || !status || num_pcs == 0 || exec_region >= ARGUS_MAX_REGIONS) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)intervals & 15) || ((uintptr_t)counts & 7)) return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  ARGUS_CUDA_TRY(cudaMemsetAsync(counts, 0, ((size_t)exec_region + 1) * num_pcs * sizeof(uint64_t), stream));
  if (num_streams == 0) return ARGUS_OK;
  const int use_cache = ((uint64_t)exec_region + 1) * num_pcs < 0xffffffffull;  // cell indices must fit the 32-bit keys
  k_map_counts<<<148 * 8, 256, 0, stream>>>(intervals, (const u64*)interval_offsets, num_streams, exec_region, num_pcs,
                                            (u64*)counts, status, use_cache);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

extern "C" size_t argus_attribute_workspace_bytes(uint32_t num_rows, uint32_t num_pcs) {
  return attr_layout(num_rows, num_pcs).total;
}

extern "C" int argus_attribute(const uint64_t* counts, uint32_t num_rows, uint32_t num_pcs, const double* metric,
                               double* mhat, double* entropy, double* alpha, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
  if (!counts || !metric || !mhat || !entropy || !workspace || num_rows == 0 || num_pcs == 0) return ARGUS_ERR_INVALID_ARG;
  if (num_rows > 65535) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) || ((uintptr_t)counts & 7) || ((uintptr_t)metric & 7) || ((uintptr_t)mhat & 7) ||
      ((uintptr_t)entropy & 7) || ((uintptr_t)alpha & 7))
    return ARGUS_ERR_INVALID_ARG;
  const AttrLayout L = attr_layout(num_rows, num_pcs);
  if (workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  u64* totals = (u64*)((char*)workspace + L.totals);
  double* partial = (double*)((char*)workspace + L.partial);
  k_attr_columns<<<(num_pcs + kAttrThreads - 1) / kAttrThreads, kAttrThreads, 0, stream>>>((const u64*)counts, num_rows, num_pcs,
                                                                                            entropy, alpha, totals);
  ARGUS_CHECK_LAUNCH();
  k_attr_rows<<<dim3(L.chunks, num_rows), kAttrThreads, 0, stream>>>((const u64*)counts, totals, num_rows, num_pcs, metric,
                                                                     L.chunks, partial);
  ARGUS_CHECK_LAUNCH();
  k_attr_finish<<<(num_rows + 255) / 256, 256, 0, stream>>>(partial, L.chunks, num_rows, mhat);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}
