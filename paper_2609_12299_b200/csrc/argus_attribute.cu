// argus_attribute.cu — PC-to-region mapping counts and ambiguity-aware attribution.
//
//   k_map_counts   : exec records of a mapping-run trace arrive as intervals of the extra region id R whose
//                    parent_region is the innermost active region (pairing did the stack work); this pass adds
//                    their execution counts into counts[owner][pc] (integer atomics: order does not matter).
//   k_attr_columns : one thread per PC: column total, alpha, entropy; the lifted metric is reduced over the
//                    PCs of a block in a fixed order into partial[block][row];
//   k_attr_finish  : mhat[row] = sum of the block partials, in block order.
#include "argus_common.cuh"

namespace {

constexpr int kAttrThreads = 256;

__global__ void __launch_bounds__(256) k_map_counts(const argus_interval_t* intervals, const u64* interval_offsets,
                                                    u32 num_streams, u32 exec_region, u32 num_pcs, u64* counts,
                                                    argus_status_t* status) {
  const u64 lo = interval_offsets[0], hi = interval_offsets[num_streams];
  for (u64 i = lo + (u64)blockIdx.x * blockDim.x + threadIdx.x; i < hi; i += (u64)gridDim.x * blockDim.x) {
    const uint4* p = reinterpret_cast<const uint4*>(intervals + i);
    const uint4 q1 = __ldg(p + 1);
    if (q1.z != exec_region) continue;
    const u32 pc = q1.w;
    if (pc >= num_pcs) { argus_set_error(status, ARGUS_ERR_INVALID_ARG, 0, i); continue; }
    const uint4 q0 = __ldg(p), q2 = __ldg(p + 2);
    const u64 k = (u64)q0.z | ((u64)q0.w << 32);
    const u32 owner = q2.y < exec_region ? q2.y : exec_region;  // no parent, or a malformed nesting of exec records
    if (k) atomicAdd(counts + (size_t)owner * num_pcs + pc, k);
  }
}

__global__ void __launch_bounds__(kAttrThreads) k_attr_columns(const u64* counts, u32 num_rows, u32 num_pcs,
                                                               const double* metric, double* entropy, double* alpha,
                                                               double* partial) {
  __shared__ double sh[kAttrThreads / 32];
  const u32 p = blockIdx.x * kAttrThreads + threadIdx.x;
  const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  u64 total = 0;
  if (p < num_pcs)
    for (u32 r = 0; r < num_rows; ++r) total += counts[(size_t)r * num_pcs + p];
  const double m = p < num_pcs ? metric[p] : 0.0;
  double h = 0.0;
  for (u32 r = 0; r < num_rows; ++r) {
    double contrib = 0.0;
    if (p < num_pcs) {
      const u64 n = counts[(size_t)r * num_pcs + p];
      const double a = (total == 0 || n == 0) ? 0.0 : (double)n / (double)total;
      if (alpha) alpha[(size_t)r * num_pcs + p] = a;
      if (a > 0.0) {
        contrib = a * m;
        h -= a * log(a);
      }
    }
    // fixed-order sum over the block's PCs: lanes by shuffle tree, then the warps in order
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) contrib += __shfl_down_sync(0xffffffffu, contrib, d);
    if (lane == 0) sh[warp] = contrib;
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = 0.0;
      for (int w = 0; w < kAttrThreads / 32; ++w) s += sh[w];
      partial[(size_t)blockIdx.x * num_rows + r] = s;
    }
    __syncthreads();
  }
  if (p < num_pcs) entropy[p] = h;
}

__global__ void __launch_bounds__(256) k_attr_finish(const double* partial, u32 num_blocks, u32 num_rows, double* mhat) {
  const u32 r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= num_rows) return;
  double s = 0.0;
  for (u32 b = 0; b < num_blocks; ++b) s += partial[(size_t)b * num_rows + r];
  mhat[r] = s;
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
  k_map_counts<<<148 * 8, 256, 0, stream>>>(intervals, (const u64*)interval_offsets, num_streams, exec_region, num_pcs,
                                            (u64*)counts, status);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

extern "C" size_t argus_attribute_workspace_bytes(uint32_t num_rows, uint32_t num_pcs) {
  const size_t blocks = ((size_t)num_pcs + kAttrThreads - 1) / kAttrThreads;
  return argus_align_up(blocks * num_rows * sizeof(double) + 256, 256);
}

extern "C" int argus_attribute(const uint64_t* counts, uint32_t num_rows, uint32_t num_pcs, const double* metric,
                               double* mhat, double* entropy, double* alpha, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
  if (!counts || !metric || !mhat || !entropy || !workspace || num_rows == 0 || num_pcs == 0) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) || ((uintptr_t)counts & 7) || ((uintptr_t)metric & 7) || ((uintptr_t)mhat & 7) ||
      ((uintptr_t)entropy & 7) || ((uintptr_t)alpha & 7))
    return ARGUS_ERR_INVALID_ARG;
  if (workspace_bytes < argus_attribute_workspace_bytes(num_rows, num_pcs)) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const u32 blocks = (num_pcs + kAttrThreads - 1) / kAttrThreads;
  k_attr_columns<<<blocks, kAttrThreads, 0, stream>>>((const u64*)counts, num_rows, num_pcs, metric, entropy, alpha,
                                                      (double*)workspace);
  ARGUS_CHECK_LAUNCH();
  k_attr_finish<<<(num_rows + 255) / 256, 256, 0, stream>>>((const double*)workspace, blocks, num_rows, mhat);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}
