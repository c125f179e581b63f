// argus_api.cu — status fetch, error strings, version.
#include "argus_common.cuh"

#include <atomic>
#include <mutex>
#include <vector>

namespace {
std::atomic<unsigned long long> g_launches{0};
std::atomic<int> g_prof_on{0};
thread_local int g_prof_suppress = 0;  // per host thread: a call that must not create events does not silence others
std::mutex g_prof_mu;
struct ProfPair { cudaEvent_t a, b; };
std::vector<ProfPair> g_prof[ARGUS_PROF_SLOTS];
}  // namespace

void argus_count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

void argus_prof_mark(int slot, cudaStream_t stream, int end) {
  if (!g_prof_on.load(std::memory_order_relaxed) || g_prof_suppress > 0 || slot < 0 ||
      slot >= ARGUS_PROF_SLOTS)
    return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  if (!end) {
    ProfPair p;
    if (cudaEventCreate(&p.a) != cudaSuccess) return;
    if (cudaEventCreate(&p.b) != cudaSuccess) { cudaEventDestroy(p.a); return; }
    cudaEventRecord(p.a, stream);
    g_prof[slot].push_back(p);
  } else if (!g_prof[slot].empty()) {
    cudaEventRecord(g_prof[slot].back().b, stream);
  }
}

void argus_prof_suppress(int delta) { g_prof_suppress += delta; }

extern "C" unsigned long long argus_launch_count(void) { return g_launches.load(); }

extern "C" void argus_profile_enable(int on) { g_prof_on.store(on ? 1 : 0); }

extern "C" int argus_profile_read(double* ms_total, unsigned long long* launches) {
  if (!ms_total || !launches) return ARGUS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  for (int s = 0; s < ARGUS_PROF_SLOTS; ++s) {
    double ms = 0;
    unsigned long long n = 0;
    for (ProfPair& p : g_prof[s]) {
      float t = 0;
      if (cudaEventSynchronize(p.b) == cudaSuccess && cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) { ms += t; ++n; }
      cudaEventDestroy(p.a);
      cudaEventDestroy(p.b);
    }
    g_prof[s].clear();
    ms_total[s] = ms;
    launches[s] = n;
  }
  return ARGUS_OK;
}

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
    case ARGUS_ERR_STATIC_LIMIT: return "input exceeds the built-in scratch of the allocation-free entry point (see ARGUS_STATIC_MAX_*)";
    default: return "unknown error code";
  }
}

extern "C" int argus_version(void) { return 100; }
