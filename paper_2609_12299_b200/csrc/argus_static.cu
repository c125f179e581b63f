// argus_static.cu — argus_pair_intervals_static: pairing without any caller-provided workspace.
//
// For callers that must not allocate device memory (tool callbacks, processes whose pool belongs
// to someone else, paths where an allocation could synchronise or fail): the pairing pipeline's
// scratch sits in a fixed array in this library's device image. Nothing here calls cudaMalloc,
// cudaFree or an allocating library routine.
#include "argus_internal.cuh"

#include <atomic>


namespace {

// Enough for the pairing pipeline at the documented maxima (control block, per-stream counters, work queue
// and hand-over records, one bit per event plus its prefix tables, 8-byte ambiguity notes): 0.92 MB.
constexpr size_t kStaticScratchBytes = 960 * 1024;
static __device__ __align__(256) unsigned char g_pair_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_scratch_ptr[kMaxDevices];  // device address of g_pair_scratch, looked up once per device
                                                // (two threads that race here both find the same address)

// The documented maxima fit the array together (the run-time check below is then never the one that refuses them).
static_assert((size_t)ARGUS_STATIC_MAX_EVENTS / 8 * 2 + (size_t)ARGUS_STATIC_MAX_AMBIG * 8 +
                  (size_t)ARGUS_STATIC_MAX_STREAMS * 12 + 64 * 1024 <= kStaticScratchBytes,
              "bitmap + word prefixes + ambiguity notes + per-stream counters and order + queue, records and control block");

}  // namespace

extern "C" int argus_pair_intervals_static(const argus_event_t* events, uint64_t num_events,
                                           const uint64_t* stream_offsets, uint32_t num_streams, uint32_t num_regions,
                                           argus_interval_t* intervals, uint64_t interval_capacity,
                                           uint64_t* interval_offsets, argus_ambiguity_t* ambig, uint64_t ambig_capacity,
                                           uint64_t* ambig_offsets, argus_status_t* status, void* cuda_stream) {
  if (num_events > ARGUS_STATIC_MAX_EVENTS || num_streams > ARGUS_STATIC_MAX_STREAMS ||
      ambig_capacity > ARGUS_STATIC_MAX_AMBIG)
    return ARGUS_ERR_STATIC_LIMIT;
  if (argus_pair_workspace_bytes(num_events, num_streams, ambig_capacity) > kStaticScratchBytes)
    return ARGUS_ERR_STATIC_LIMIT;
  int dev = 0;
  ARGUS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ARGUS_ERR_INVALID_ARG;
  void* scratch = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // The array's name is only a host-side handle; kernels need its address on the current device.
    ARGUS_CUDA_TRY(cudaGetSymbolAddress(&scratch, g_pair_scratch));
    if (!scratch) return ARGUS_ERR_CUDA;
    g_scratch_ptr[dev].store(scratch, std::memory_order_release);
  }
  // The pipeline clears its control block, counters and bitmap itself at the start of every call.
  // Kernel-time profiling would create CUDA events (an allocation), so it stays off in here (for this thread only).
  argus_prof_suppress(+1);
  const int rc = argus_internal_pair(events, num_events, stream_offsets, num_streams, num_regions, intervals,
                                     interval_capacity, interval_offsets, ambig, ambig_capacity, ambig_offsets, status,
                                     scratch, kStaticScratchBytes, cuda_stream, 0, true);
  argus_prof_suppress(-1);
  return rc;
}
