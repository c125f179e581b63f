// tracegen_cuda.cu — device build of the synthetic trace generator (one thread per stream).
// Compiled with -fmad=false so that every floating-point step rounds exactly as on the host.
#include <cuda_runtime.h>

#include "tracegen.h"

namespace {

__global__ void k_lengths(tg_params p, uint32_t S, uint64_t* lens) {
  const uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= S) return;
  const uint64_t full = tg_run_stream(p, s, nullptr, 0);
  lens[s] = tg_truncated_len(p, s, full);
}

__global__ void k_fill(tg_params p, const uint64_t* offs, uint32_t s_lo, uint32_t s_hi, tg_event* out) {
  const uint32_t s = s_lo + blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= s_hi) return;
  const uint64_t n = offs[s + 1] - offs[s];
  if (n) tg_run_stream(p, s, out + (offs[s] - offs[s_lo]), n);
}

}  // namespace

extern "C" {

// lens: device [S]. Enqueues on `stream`; returns a cudaError_t value.
int tg_cuda_lengths(const tg_params* p, uint64_t* lens, void* stream) {
  const uint32_t S = p->num_ctas * tg_warps_per_cta(p->kind);
  if (S == 0) return 0;
  k_lengths<<<(S + 31) / 32, 32, 0, (cudaStream_t)stream>>>(*p, S, lens);
  return (int)cudaGetLastError();
}

// offs: device [S+1]; out: device, stream s at out[offs[s] - offs[s_lo]].
int tg_cuda_fill(const tg_params* p, const uint64_t* offs, uint32_t s_lo, uint32_t s_hi, tg_event* out,
                 void* stream) {
  if (s_hi <= s_lo) return 0;
  const uint32_t n = s_hi - s_lo;
  k_fill<<<(n + 31) / 32, 32, 0, (cudaStream_t)stream>>>(*p, offs, s_lo, s_hi, out);
  return (int)cudaGetLastError();
}
}
