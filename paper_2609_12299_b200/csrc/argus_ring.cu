// argus_ring.cu — argus_ring_linearise: fixed-slot ring buffers (one slot per stream, possibly wrapped)
// -> packed CSR events + stream_offsets, the input form of the pairing kernels.
//
//   k_ring_offsets : single-block scan of min(written, slot_capacity) over the streams; capacity check
//   k_ring_copy    : one block per stream copies the surviving records, oldest first (16-byte loads and stores)
#include "argus_internal.cuh"

namespace {

constexpr int kRingScanThreads = 1024;

__global__ void __launch_bounds__(kRingScanThreads) k_ring_offsets(const u64* written, u32 slot_capacity, u32 num_streams,
                                                                   u64 event_capacity, u64* stream_offsets, u64* dropped,
                                                                   argus_status_t* status) {
  __shared__ u64 sh[33];
  u64 carry = 0;
  for (u32 s0 = 0; s0 < num_streams; s0 += kRingScanThreads) {
    const u32 s = s0 + threadIdx.x;
    const u64 w = s < num_streams ? written[s] : 0;
    const u64 kept = w < slot_capacity ? w : slot_capacity;
    u64 total;
    const u64 ex = argus_block_exclusive_scan<u64>(kept, sh, &total);
    if (s < num_streams) {
      stream_offsets[s] = carry + ex;
      if (dropped) dropped[s] = w - kept;
    }
    carry += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    stream_offsets[num_streams] = carry;
    status->intervals_required = carry;
    if (carry > event_capacity) argus_set_error(status, ARGUS_ERR_CAPACITY, 0, carry);
  }
}

__global__ void __launch_bounds__(256) k_ring_copy(const uint4* ring, u32 slot_capacity, const u64* written, u32 num_streams,
                                                   uint4* events, const u64* stream_offsets, const argus_status_t* status) {
  if (status->code != 0) return;  // the packed records do not fit: nothing is copied
  for (u32 s = blockIdx.x; s < num_streams; s += gridDim.x) {
    const u64 w = written[s];
    const u64 kept = w < slot_capacity ? w : slot_capacity;
    const u64 first = (w - kept) % slot_capacity;  // slot position of the oldest surviving record
    const uint4* src = ring + (u64)s * slot_capacity;
    uint4* dst = events + stream_offsets[s];
    for (u64 i = threadIdx.x; i < kept; i += blockDim.x) {
      u64 p = first + i;
      if (p >= slot_capacity) p -= slot_capacity;
      dst[i] = __ldg(src + p);
    }
  }
}

}  // namespace

int argus_internal_ring_offsets(const uint64_t* written, uint32_t slot_capacity, uint32_t num_streams, uint64_t event_capacity,
                                uint64_t* stream_offsets, uint64_t* dropped, argus_status_t* status, void* cuda_stream) {
  k_ring_offsets<<<1, kRingScanThreads, 0, (cudaStream_t)cuda_stream>>>((const u64*)written, slot_capacity, num_streams, event_capacity,
                                                                        (u64*)stream_offsets, (u64*)dropped, status);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

extern "C" int argus_ring_linearise(const argus_event_t* ring, uint32_t slot_capacity, const uint64_t* written,
                                    uint32_t num_streams, argus_event_t* events, uint64_t event_capacity,
                                    uint64_t* stream_offsets, uint64_t* dropped, argus_status_t* status, void* cuda_stream) {
  if (!status || !stream_offsets || slot_capacity == 0) return ARGUS_ERR_INVALID_ARG;
  if (num_streams && (!ring || !written)) return ARGUS_ERR_INVALID_ARG;
  if (event_capacity && !events) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)ring & 15) || ((uintptr_t)events & 15) || ((uintptr_t)written & 7) || ((uintptr_t)stream_offsets & 7) ||
      ((uintptr_t)dropped & 7))
    return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  k_ring_offsets<<<1, kRingScanThreads, 0, stream>>>((const u64*)written, slot_capacity, num_streams, event_capacity,
                                                     (u64*)stream_offsets, (u64*)dropped, status);
  ARGUS_CHECK_LAUNCH();
  if (num_streams) {
    k_ring_copy<<<num_streams < 148u * 16u ? num_streams : 148u * 16u, 256, 0, stream>>>(
        reinterpret_cast<const uint4*>(ring), slot_capacity, (const u64*)written, num_streams,
        reinterpret_cast<uint4*>(events), (const u64*)stream_offsets, status);
    ARGUS_CHECK_LAUNCH();
  }
  return ARGUS_OK;
}
