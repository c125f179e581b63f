// argus_join.cu — argus_join_samples: probe-run samples joined to reference intervals by exact key
// (stream, region, ctx), with count, sum and the 0/20/40/60/80th percentiles of the joined values.
//
// One block per query: it streams over all samples (reading the 32 bytes of a record that hold the key
// before the 16 that hold the value), gathers the values of matching samples in shared memory, sorts
// them (bitonic network over the next power of two) and picks the ranks. Meant for the selected
// operations of a query, tens to thousands, not for whole-trace joins. When the samples come with the
// interval offsets of the probe runs that produced them (argus_join_samples_grouped), a query reads only
// the samples of its own stream in every run.
#include "argus_common.cuh"

namespace {

constexpr int kJoinThreads = 256;

__global__ void __launch_bounds__(kJoinThreads) k_join(const argus_interval_t* reference, u64 num_reference,
                                                       const u64* ref_index, u32 num_queries,
                                                       const argus_interval_t* samples, u64 num_samples,
                                                       const u64* sample_offsets, u32 num_runs, u32 num_streams,
                                                       argus_join_t* out, argus_status_t* status) {
  __shared__ u64 vals[ARGUS_JOIN_MAX_SAMPLES];
  __shared__ u64 warp_sum[kJoinThreads / 32];
  __shared__ u32 cnt;
  const u32 tid = threadIdx.x;
  for (u32 q = blockIdx.x; q < num_queries; q += gridDim.x) {
    if (tid == 0) cnt = 0;
    __syncthreads();
    const u64 idx = ref_index[q];
    if (idx >= num_reference) {  // uniform in the block
      if (tid == 0) {
        argus_set_error(status, ARGUS_ERR_INVALID_ARG, 0, q);
        argus_join_t z = {};
        out[q] = z;
      }
      continue;
    }
    const uint4* r = reinterpret_cast<const uint4*>(reference + idx);
    const uint4 r1 = __ldg(r + 1);
    const u32 key_region = r1.z, key_ctx = r1.w, key_stream = __ldg(reinterpret_cast<const u32*>(r + 2));
    u64 sum = 0;
    // the ranges of `samples` to look at: everything, or the query's stream in every probe run
    const u32 ranges = sample_offsets ? (key_stream < num_streams ? num_runs : 0u) : 1u;
    for (u32 run = 0; run < ranges; ++run) {
      u64 lo = 0, hi = num_samples;
      if (sample_offsets) {
        lo = sample_offsets[(u64)run * (num_streams + 1) + key_stream];
        hi = sample_offsets[(u64)run * (num_streams + 1) + key_stream + 1];
        if (hi < lo || hi > num_samples) {  // uniform in the block
          if (tid == 0) argus_set_error(status, ARGUS_ERR_BAD_OFFSETS, key_stream, run);
          continue;
        }
      }
      for (u64 i = lo + tid; i < hi; i += kJoinThreads) {
        const uint4* p = reinterpret_cast<const uint4*>(samples + i);
        const uint4 q1 = __ldg(p + 1);
        if (q1.z != key_region || q1.w != key_ctx) continue;
        if (__ldg(reinterpret_cast<const u32*>(p + 2)) != key_stream) continue;
        const uint4 q0 = __ldg(p);
        const u64 v = (u64)q0.z | ((u64)q0.w << 32);
        sum += v;
        const u32 slot = atomicAdd(&cnt, 1u);
        if (slot < ARGUS_JOIN_MAX_SAMPLES) vals[slot] = v;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, d);
    if ((tid & 31) == 0) warp_sum[tid >> 5] = sum;
    __syncthreads();
    const u32 total = cnt;
    const u32 n = total < ARGUS_JOIN_MAX_SAMPLES ? total : ARGUS_JOIN_MAX_SAMPLES;
    u32 m = 1;
    while (m < n) m <<= 1;
    for (u32 i = n + tid; i < m; i += kJoinThreads) vals[i] = ~0ull;  // padding sorts to the end
    __syncthreads();
    for (u32 k = 2; k <= m; k <<= 1) {
      for (u32 j = k >> 1; j > 0; j >>= 1) {
        for (u32 i = tid; i < m; i += kJoinThreads) {
          const u32 l = i ^ j;
          if (l > i) {
            const u64 a = vals[i], b = vals[l];
            const bool up = (i & k) == 0;
            if ((a > b) == up) { vals[i] = b; vals[l] = a; }
          }
        }
        __syncthreads();
      }
    }
    if (tid == 0) {
      argus_join_t o = {};
      o.count = total;
      for (int w = 0; w < kJoinThreads / 32; ++w) o.sum += warp_sum[w];
      if (n) {
        for (u32 j = 0; j < 5; ++j) o.pct[j] = vals[(u64)j * n / 5];
        o.max = vals[n - 1];
      }
      out[q] = o;
      if (total > ARGUS_JOIN_MAX_SAMPLES) argus_set_error(status, ARGUS_ERR_CAPACITY, key_stream, idx);
    }
    __syncthreads();
  }
}

}  // namespace

static int join_impl(const argus_interval_t* reference, uint64_t num_reference, const uint64_t* ref_index,
                     uint32_t num_queries, const argus_interval_t* samples, uint64_t num_samples,
                     const uint64_t* sample_offsets, uint32_t num_runs, uint32_t num_streams, argus_join_t* out,
                     argus_status_t* status, void* cuda_stream) {
  if (!status) return ARGUS_ERR_INVALID_ARG;
  if (num_queries && (!reference || !ref_index || !out)) return ARGUS_ERR_INVALID_ARG;
  if (num_samples && !samples) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)reference & 15) || ((uintptr_t)samples & 15) || ((uintptr_t)ref_index & 7) || ((uintptr_t)out & 7) ||
      ((uintptr_t)sample_offsets & 7))
    return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  if (num_queries == 0) return ARGUS_OK;
  k_join<<<num_queries < 148u * 8u ? num_queries : 148u * 8u, kJoinThreads, 0, stream>>>(
      reference, num_reference, (const u64*)ref_index, num_queries, samples, num_samples, (const u64*)sample_offsets, num_runs,
      num_streams, out, status);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

extern "C" int argus_join_samples(const argus_interval_t* reference, uint64_t num_reference, const uint64_t* ref_index,
                                  uint32_t num_queries, const argus_interval_t* samples, uint64_t num_samples,
                                  argus_join_t* out, argus_status_t* status, void* cuda_stream) {
  return join_impl(reference, num_reference, ref_index, num_queries, samples, num_samples, nullptr, 0, 0, out, status,
                   cuda_stream);
}

extern "C" int argus_join_samples_grouped(const argus_interval_t* reference, uint64_t num_reference, const uint64_t* ref_index,
                                          uint32_t num_queries, const argus_interval_t* samples, uint64_t num_samples,
                                          const uint64_t* sample_offsets, uint32_t num_runs, uint32_t num_streams,
                                          argus_join_t* out, argus_status_t* status, void* cuda_stream) {
  if (!sample_offsets && num_runs) return ARGUS_ERR_INVALID_ARG;
  if (!sample_offsets || num_runs == 0) {  // no probe run: every query comes out empty
    return join_impl(reference, num_reference, ref_index, num_queries, samples, 0, nullptr, 0, 0, out, status, cuda_stream);
  }
  return join_impl(reference, num_reference, ref_index, num_queries, samples, num_samples, sample_offsets, num_runs, num_streams,
                   out, status, cuda_stream);
}
