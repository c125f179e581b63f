// argus_api.cu — status fetch, error strings, version.
#include "argus_common.cuh"

extern "C" int argus_status_fetch(const argus_status_t* dev_status, argus_status_t* host_copy, void* cuda_stream) {
  if (!dev_status || !host_copy) return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemcpyAsync(host_copy, dev_status, sizeof(argus_status_t), cudaMemcpyDeviceToHost, stream));
  ARGUS_CUDA_TRY(cudaStreamSynchronize(stream));
  return ARGUS_OK;
}

extern "C" const char* argus_strerror(int code) {
  switch (code) {
    case ARGUS_OK: return "ok";
    case ARGUS_ERR_INVALID_ARG: return "invalid argument";
    case ARGUS_ERR_WORKSPACE: return "workspace too small";
    case ARGUS_ERR_CUDA: return "CUDA runtime error";
    case ARGUS_ERR_CAPACITY: return "output capacity too small (see *_required in the status block)";
    case ARGUS_ERR_DEPTH: return "more than ARGUS_MAX_DEPTH open frames in a stream";
    case ARGUS_ERR_BAD_REGION: return "region id out of range";
    case ARGUS_ERR_BAD_OFFSETS: return "offsets are not non-decreasing or exceed the buffer";
    case ARGUS_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown error code";
  }
}

extern "C" int argus_version(void) { return 100; }
