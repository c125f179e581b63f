// argus_static.cu — argus_pair_intervals_static: pairing without any caller-provided workspace.
//
// For callers that must not allocate device memory (tool callbacks, processes whose pool belongs
// to someone else, paths where an allocation could synchronise or fail): the pairing pipeline's
// scratch sits in a fixed array in this library's device image. Nothing here calls cudaMalloc,
// cudaFree or an allocating library routine.
#include "argus_internal.cuh"


namespace {

// Enough for the pairing pipeline at the documented maxima (control block, per-stream counters, work queue
// and hand-over records, one bit per event plus its prefix tables, 8-byte ambiguity notes): 0.92 MB.
constexpr size_t kStaticScratchBytes = 960 * 1024;
static __device__ __align__(256) unsigned char g_pair_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];  // device address of g_pair_scratch, looked up once per device

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
  if (!g_scratch_ptr[dev]) {
    // The array's name is only a host-side handle; kernels need its address on the current device.
    void* p = nullptr;
    ARGUS_CUDA_TRY(cudaGetSymbolAddress(&p, g_pair_scratch));
    if (!p) return ARGUS_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  // The pipeline clears its control block, counters and bitmap itself at the start of every call.
  // Kernel-time profiling would create CUDA events (an allocation), so it stays off in here.
  argus_prof_suppress(+1);
  const int rc = argus_internal_pair(events, num_events, stream_offsets, num_streams, num_regions, intervals,
                                     interval_capacity, interval_offsets, ambig, ambig_capacity, ambig_offsets, status,
                                     g_scratch_ptr[dev], kStaticScratchBytes, cuda_stream, 0, true);
  argus_prof_suppress(-1);
  return rc;
}
