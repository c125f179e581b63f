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


// ---------------------------------------------------------------------------------------------
// One pass over the samples for all queries at once (argus_join_samples_hashed). The distinct keys of the
// queries go into an open-addressing table (linear probing; at most a quarter full); every sample is read
// once, looked up, and, when its key is asked for, counted, summed and appended to that key's value list;
// one block per query then sorts its key's list and picks the ranks.
// ---------------------------------------------------------------------------------------------
struct JoinSlot { u32 stream, region, ctx, owner; };  // owner: query index + 1 of the query that claimed the slot; 0 = empty

struct JoinHashArgs {
  const argus_interval_t* reference;
  u64 num_reference;
  const u64* ref_index;
  u32 num_queries;
  const argus_interval_t* samples;
  u64 num_samples;
  JoinSlot* table;
  u32 cap_mask;       // table slots - 1 (a power of two)
  u32* key_of_query;  // [Q] index of the query whose slot this query shares (itself when it claimed one); ~0 = bad index
  u64* count;         // [Q] per claiming query: samples with its key
  u64* sum;           // [Q]
  u64* vals;          // [Q][ARGUS_JOIN_MAX_SAMPLES]
  argus_join_t* out;
  argus_status_t* status;
};

__device__ __forceinline__ u32 join_hash(u32 stream, u32 region, u32 ctx) {
  u32 h = stream * 0x9e3779b1u ^ (region + 0x7f4a7c15u) * 0x85ebca6bu ^ ctx * 0xc2b2ae35u;
  h ^= h >> 15; h *= 0x2c1b3c6du; h ^= h >> 12;
  return h;
}

__device__ __forceinline__ void join_key(const argus_interval_t* rec, u32* stream, u32* region, u32* ctx) {
  const uint4* r = reinterpret_cast<const uint4*>(rec);
  const uint4 r1 = __ldg(r + 1);
  *region = r1.z; *ctx = r1.w; *stream = __ldg(reinterpret_cast<const u32*>(r + 2));
}

// Every query claims the slot of its key, or finds the query that already has. A slot's key is the key of the
// query that owns it (read through the reference record), so claiming is one compare-and-swap and nothing waits.
__global__ void __launch_bounds__(256) k_join_claim(JoinHashArgs g) {
  const u32 q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= g.num_queries) return;
  g.count[q] = 0; g.sum[q] = 0;
  const u64 idx = g.ref_index[q];
  if (idx >= g.num_reference) {
    argus_set_error(g.status, ARGUS_ERR_INVALID_ARG, 0, q);
    g.key_of_query[q] = 0xffffffffu;
    return;
  }
  u32 st, rg, cx;
  join_key(g.reference + idx, &st, &rg, &cx);
  u32 slot = join_hash(st, rg, cx) & g.cap_mask;
  for (u32 probes = 0; probes <= g.cap_mask; ++probes, slot = (slot + 1) & g.cap_mask) {
    const u32 old = atomicCAS(&g.table[slot].owner, 0u, q + 1);
    if (old == 0) { g.key_of_query[q] = q; return; }
    u32 st2, rg2, cx2;
    join_key(g.reference + g.ref_index[old - 1], &st2, &rg2, &cx2);  // owners have valid indices
    if (st2 == st && rg2 == rg && cx2 == cx) { g.key_of_query[q] = old - 1; return; }
  }
  g.key_of_query[q] = 0xffffffffu;  // cannot happen: the table has four slots per query
}

__global__ void __launch_bounds__(256) k_join_fill(JoinHashArgs g) {
  const u32 slot = blockIdx.x * blockDim.x + threadIdx.x;
  if (slot > g.cap_mask) return;
  const u32 o = g.table[slot].owner;
  if (!o) return;
  u32 st, rg, cx;
  join_key(g.reference + g.ref_index[o - 1], &st, &rg, &cx);
  g.table[slot].stream = st; g.table[slot].region = rg; g.table[slot].ctx = cx;
}

__global__ void __launch_bounds__(256) k_join_scan(JoinHashArgs g) {
  const uint4* tab = reinterpret_cast<const uint4*>(g.table);
  for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < g.num_samples; i += (u64)gridDim.x * blockDim.x) {
    const uint4* p = reinterpret_cast<const uint4*>(g.samples + i);
    const uint4 q0 = __ldg(p), q1 = __ldg(p + 1);
    const u32 st = __ldg(reinterpret_cast<const u32*>(p + 2));
    u32 slot = join_hash(st, q1.z, q1.w) & g.cap_mask;
    for (u32 probes = 0; probes <= g.cap_mask; ++probes, slot = (slot + 1) & g.cap_mask) {
      const uint4 t = __ldg(tab + slot);  // stream, region, ctx, owner
      if (t.w == 0) break;                // an empty slot ends the probe sequence: nobody asks for this key
      if (t.x == st && t.y == q1.z && t.z == q1.w) {
        const u32 k = t.w - 1;
        const u64 v = (u64)q0.z | ((u64)q0.w << 32);
        const u64 at = atomicAdd(&g.count[k], 1ull);
        atomicAdd(&g.sum[k], v);
        if (at < ARGUS_JOIN_MAX_SAMPLES) g.vals[(u64)k * ARGUS_JOIN_MAX_SAMPLES + at] = v;
        break;
      }
    }
  }
}

__global__ void __launch_bounds__(kJoinThreads) k_join_rank(JoinHashArgs g) {
  __shared__ u64 vals[ARGUS_JOIN_MAX_SAMPLES];
  const u32 tid = threadIdx.x;
  for (u32 q = blockIdx.x; q < g.num_queries; q += gridDim.x) {
    const u32 k = g.key_of_query[q];
    if (k == 0xffffffffu) {  // uniform in the block
      if (tid == 0) { argus_join_t z = {}; g.out[q] = z; }
      continue;
    }
    const u64 total = g.count[k];
    const u32 n = total < ARGUS_JOIN_MAX_SAMPLES ? (u32)total : (u32)ARGUS_JOIN_MAX_SAMPLES;
    u32 m = 1;
    while (m < n) m <<= 1;
    for (u32 i = tid; i < m; i += kJoinThreads) vals[i] = i < n ? g.vals[(u64)k * ARGUS_JOIN_MAX_SAMPLES + i] : ~0ull;
    __syncthreads();
    for (u32 kk = 2; kk <= m; kk <<= 1) {
      for (u32 j = kk >> 1; j > 0; j >>= 1) {
        for (u32 i = tid; i < m; i += kJoinThreads) {
          const u32 l = i ^ j;
          if (l > i) {
            const u64 a = vals[i], b = vals[l];
            const bool up = (i & kk) == 0;
            if ((a > b) == up) { vals[i] = b; vals[l] = a; }
          }
        }
        __syncthreads();
      }
    }
    if (tid == 0) {
      argus_join_t o = {};
      o.count = total;
      o.sum = g.sum[k];
      if (n) {
        for (u32 j = 0; j < 5; ++j) o.pct[j] = vals[(u64)j * n / 5];
        o.max = vals[n - 1];
      }
      g.out[q] = o;
      if (total > ARGUS_JOIN_MAX_SAMPLES) {
        u32 st, rg, cx;
        join_key(g.reference + g.ref_index[q], &st, &rg, &cx);
        argus_set_error(g.status, ARGUS_ERR_CAPACITY, st, g.ref_index[q]);
      }
    }
    __syncthreads();
  }
}

struct JoinLayout { size_t table, key_of_query, count, sum, vals, total; u32 cap; };

JoinLayout join_layout(uint32_t num_queries) {
  JoinLayout L;
  u32 cap = 1024;
  while (cap < 4ull * num_queries && cap < (1u << 31)) cap <<= 1;
  L.cap = cap;
  size_t o = 0;
  L.table = o; o += argus_align_up((size_t)cap * sizeof(JoinSlot), 256);
  L.key_of_query = o; o += argus_align_up((size_t)num_queries * 4 + 4, 256);
  L.count = o; o += argus_align_up((size_t)num_queries * 8 + 8, 256);
  L.sum = o; o += argus_align_up((size_t)num_queries * 8 + 8, 256);
  L.vals = o; o += argus_align_up((size_t)num_queries * ARGUS_JOIN_MAX_SAMPLES * 8 + 8, 256);
  L.total = o;
  return L;
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

extern "C" size_t argus_join_workspace_bytes(uint32_t num_queries) { return join_layout(num_queries).total; }

extern "C" int argus_join_samples_hashed(const argus_interval_t* reference, uint64_t num_reference, const uint64_t* ref_index,
                                         uint32_t num_queries, const argus_interval_t* samples, uint64_t num_samples,
                                         argus_join_t* out, argus_status_t* status, void* workspace, size_t workspace_bytes,
                                         void* cuda_stream) {
  if (!status) return ARGUS_ERR_INVALID_ARG;
  if (num_queries && (!reference || !ref_index || !out || !workspace)) return ARGUS_ERR_INVALID_ARG;
  if (num_samples && !samples) return ARGUS_ERR_INVALID_ARG;
  if (num_queries > (1u << 28)) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)reference & 15) || ((uintptr_t)samples & 15) || ((uintptr_t)ref_index & 7) || ((uintptr_t)out & 7) ||
      ((uintptr_t)workspace & 255))
    return ARGUS_ERR_INVALID_ARG;
  const JoinLayout L = join_layout(num_queries);
  if (num_queries && workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  if (num_queries == 0) return ARGUS_OK;
  char* ws = (char*)workspace;
  JoinHashArgs g;
  g.reference = reference; g.num_reference = num_reference; g.ref_index = (const u64*)ref_index; g.num_queries = num_queries;
  g.samples = samples; g.num_samples = num_samples; g.table = (JoinSlot*)(ws + L.table); g.cap_mask = L.cap - 1;
  g.key_of_query = (u32*)(ws + L.key_of_query); g.count = (u64*)(ws + L.count); g.sum = (u64*)(ws + L.sum);
  g.vals = (u64*)(ws + L.vals); g.out = out; g.status = status;
  ARGUS_CUDA_TRY(cudaMemsetAsync(ws + L.table, 0, (size_t)L.cap * sizeof(JoinSlot), stream));
  k_join_claim<<<(num_queries + 255) / 256, 256, 0, stream>>>(g);
  ARGUS_CHECK_LAUNCH();
  k_join_fill<<<(L.cap + 255) / 256, 256, 0, stream>>>(g);
  ARGUS_CHECK_LAUNCH();
  if (num_samples) {
    int dev = 0, sms = 0;
    ARGUS_CUDA_TRY(cudaGetDevice(&dev));
    ARGUS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const u64 want = (num_samples + 255) / 256;
    const u64 cap_blocks = (u64)sms * 16;
    k_join_scan<<<(unsigned)(want < cap_blocks ? want : cap_blocks), 256, 0, stream>>>(g);
    ARGUS_CHECK_LAUNCH();
  }
  k_join_rank<<<num_queries < 2368u ? num_queries : 2368u, kJoinThreads, 0, stream>>>(g);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}
