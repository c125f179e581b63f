// argus_aggregate.cu — argus_aggregate: intervals (+ ambiguity records) -> per-(scope, region) tables.
//
//   k_agg_streams : one CTA per stream accumulates that stream's row of the warp-scope table
//                   (a shared-memory private copy when num_regions * 576 B fits, else the global row
//                   itself), integer atomics only, so the result does not depend on thread order.
//   k_agg_cta     : CTA-scope cells = reduction over the warps of each CTA (plain loads, no atomics).
//   k_agg_init / k_agg_scatter : SM-scope and kernel-scope cells by atomic add/min/max of CTA cells.
#include "argus_common.cuh"

namespace {

constexpr int kAggThreads = 256;
constexpr u32 kCell = 72;  // u64 words per argus_agg_t
constexpr size_t kAggSmemLimit = 200 * 1024;

struct AggArgs {
  const argus_interval_t* intervals;
  const u64* interval_offsets;
  const argus_ambiguity_t* ambig;
  const u64* ambig_offsets;
  u32 num_streams, warps_per_cta, num_ctas, num_sms, num_regions;
  const u32* cta_sm;
  u64* warp_tab;  // [S][R][72] (caller's table or workspace)
  u64* cta_tab;   // [C][R][72] (caller's table or workspace)
  u64* sm_tab;    // nullable
  u64* kernel_tab;  // nullable
  argus_status_t* status;
  int use_smem;
};

__device__ __forceinline__ u32 log2_bin(u64 d) { return d ? 63u - (u32)__clzll((long long)d) : 0u; }

__device__ __forceinline__ void agg_add_interval(u64* tab, u32 region, u64 incl, u64 excl, u32 flags) {
  u64* c = tab + (size_t)region * kCell;
  atomicAdd(c + 0, 1ull);
  atomicAdd(c + 1, incl);
  atomicMin(c + 2, incl);
  atomicMax(c + 3, incl);
  atomicAdd(c + 4, excl);
  if (flags) atomicAdd(c + 7, 1ull);
  atomicAdd(c + 8 + log2_bin(incl), 1ull);
}

__global__ void __launch_bounds__(kAggThreads) k_agg_streams(AggArgs a) {
  extern __shared__ __align__(16) u64 sh_tab[];
  const u32 R = a.num_regions;
  const u32 cells = R * kCell;
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    u64* row = a.warp_tab + (size_t)s * cells;
    u64* tab = a.use_smem ? sh_tab : row;
    for (u32 i = threadIdx.x; i < cells; i += blockDim.x) tab[i] = (i % kCell == 2) ? ~0ull : 0ull;
    if (!a.use_smem) __threadfence();
    __syncthreads();
    const u64 lo = a.interval_offsets[s], hi = a.interval_offsets[s + 1];
    if (hi < lo) {
      if (threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
    } else {
      for (u64 i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const uint4* p = reinterpret_cast<const uint4*>(a.intervals + i);
        const uint4 q0 = __ldg(p), q1 = __ldg(p + 1), q2 = __ldg(p + 2);
        const u64 incl = (u64)q0.z | ((u64)q0.w << 32);
        const u64 excl = (u64)q1.x | ((u64)q1.y << 32);
        const u32 region = q1.z;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        agg_add_interval(tab, region, incl, excl, q2.w >> 16);
      }
    }
    if (a.ambig && a.ambig_offsets) {
      const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
      for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
        const u32 region = a.ambig[i].tag >> 1;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        atomicAdd(tab + (size_t)region * kCell + (a.ambig[i].kind == ARGUS_AMBIG_UNMATCHED_END ? 6 : 5), 1ull);
      }
    }
    __syncthreads();
    if (a.use_smem) {
      for (u32 i = threadIdx.x; i < cells; i += blockDim.x) row[i] = sh_tab[i];
      __syncthreads();
    }
  }
}

__device__ __forceinline__ u64 combine(u32 field, u64 x, u64 y) {
  return field == 2 ? (x < y ? x : y) : field == 3 ? (x > y ? x : y) : x + y;
}

// cta_tab[c][r][j] = reduce over w of warp_tab[c*W + w][r][j]
__global__ void __launch_bounds__(256) k_agg_cta(AggArgs a) {
  const u64 per_cta = (u64)a.num_regions * kCell;
  const u64 n = (u64)a.num_ctas * per_cta;
  for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (u64)gridDim.x * blockDim.x) {
    const u64 c = i / per_cta, rem = i % per_cta;
    const u32 field = (u32)(rem % kCell);
    const u64* src = a.warp_tab + c * a.warps_per_cta * per_cta + rem;
    u64 acc = src[0];
    for (u32 w = 1; w < a.warps_per_cta; ++w) acc = combine(field, acc, src[(u64)w * per_cta]);
    a.cta_tab[i] = acc;
  }
}

__global__ void __launch_bounds__(256) k_agg_init(u64* tab, u64 n) {
  for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (u64)gridDim.x * blockDim.x)
    tab[i] = (i % kCell == 2) ? ~0ull : 0ull;
}

// SM-scope and kernel-scope cells from CTA cells (atomic add / min / max on integers).
__global__ void __launch_bounds__(256) k_agg_scatter(AggArgs a) {
  const u64 per_cta = (u64)a.num_regions * kCell;
  const u64 n = (u64)a.num_ctas * per_cta;
  for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (u64)gridDim.x * blockDim.x) {
    const u64 c = i / per_cta, rem = i % per_cta;
    const u32 field = (u32)(rem % kCell);
    const u64 v = a.cta_tab[i];
    if (field == 2 ? v == ~0ull : v == 0ull) continue;  // identity element: nothing to add
    if (a.sm_tab) {
      const u32 m = a.cta_sm[c];
      if (m >= a.num_sms) { argus_set_error(a.status, ARGUS_ERR_INVALID_ARG, (u32)c, m); continue; }
      u64* d = a.sm_tab + (u64)m * per_cta + rem;
      if (field == 2) atomicMin(d, v); else if (field == 3) atomicMax(d, v); else atomicAdd(d, v);
    }
    if (a.kernel_tab) {
      u64* d = a.kernel_tab + rem;
      if (field == 2) atomicMin(d, v); else if (field == 3) atomicMax(d, v); else atomicAdd(d, v);
    }
  }
}

// ambiguity counters into the warp-scope table (used when the intervals were aggregated by the pairing kernel)
__global__ void __launch_bounds__(256) k_agg_ambig(AggArgs a) {
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
    u64* row = a.warp_tab + (size_t)s * a.num_regions * kCell;
    for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
      const u32 region = a.ambig[i].tag >> 1;
      if (region >= a.num_regions) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
      atomicAdd(row + (size_t)region * kCell + (a.ambig[i].kind == ARGUS_AMBIG_UNMATCHED_END ? 6 : 5), 1ull);
    }
  }
}

struct AggLayout { size_t warp, cta, total; };

AggLayout agg_layout(uint32_t num_streams, uint32_t num_regions) {
  AggLayout L;
  const size_t row = (size_t)num_regions * sizeof(argus_agg_t);
  L.warp = 0;
  L.cta = argus_align_up((size_t)num_streams * row, 256);
  L.total = L.cta + argus_align_up((size_t)num_streams * row, 256);  // C <= S
  return L;
}

}  // namespace

// Roll-up of a filled warp-scope table into the CTA, SM and kernel scopes.
static int agg_rollup(AggArgs& a, argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab, cudaStream_t stream) {
  if (cta_tab || sm_tab || kernel_tab) {
    k_agg_cta<<<1184, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  if (sm_tab || kernel_tab) {
    if (sm_tab) { k_agg_init<<<296, 256, 0, stream>>>(a.sm_tab, (u64)a.num_sms * a.num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    if (kernel_tab) { k_agg_init<<<16, 256, 0, stream>>>(a.kernel_tab, (u64)a.num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    k_agg_scatter<<<1184, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  return ARGUS_OK;
}

// Second half of aggregation when the pairing kernel already filled the interval statistics of
// warp_tab: ambiguity counters, then the roll-up. warp_tab and cta_work must be non-null.
int argus_internal_agg_finish(const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                              uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                              argus_agg_t* warp_tab, argus_agg_t* cta_work, bool want_cta, argus_agg_t* sm_tab,
                              argus_agg_t* kernel_tab, argus_status_t* status, void* cuda_stream) {
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (num_streams == 0) return ARGUS_OK;
  AggArgs a;
  a.intervals = nullptr; a.interval_offsets = nullptr; a.ambig = ambig; a.ambig_offsets = (const u64*)ambig_offsets;
  a.num_streams = num_streams; a.warps_per_cta = warps_per_cta; a.num_ctas = num_streams / warps_per_cta;
  a.num_sms = num_sms; a.num_regions = num_regions; a.cta_sm = cta_sm;
  a.warp_tab = (u64*)warp_tab; a.cta_tab = (u64*)cta_work; a.sm_tab = (u64*)sm_tab; a.kernel_tab = (u64*)kernel_tab;
  a.status = status; a.use_smem = 0;
  if (ambig && ambig_offsets) {
    k_agg_ambig<<<num_streams < 1184 ? num_streams : 1184, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  return agg_rollup(a, want_cta || sm_tab || kernel_tab ? cta_work : nullptr, sm_tab, kernel_tab, stream);
}

extern "C" size_t argus_aggregate_workspace_bytes(uint64_t /*num_intervals*/, uint32_t num_streams, uint32_t num_regions) {
  return agg_layout(num_streams, num_regions).total + 256;
}

int argus_internal_aggregate(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                             const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                             uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                             argus_agg_t* warp_tab, argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab,
                             argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream,
                             bool reset_status) {
  if (!interval_offsets || !status || !workspace) return ARGUS_ERR_INVALID_ARG;
  if (warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ARGUS_ERR_INVALID_ARG;
  if (num_regions == 0 || num_regions > ARGUS_MAX_REGIONS) return ARGUS_ERR_INVALID_ARG;
  if (sm_tab && (!cta_sm || num_sms == 0)) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)intervals & 15) || ((uintptr_t)workspace & 255) || ((uintptr_t)warp_tab & 7) || ((uintptr_t)cta_tab & 7) ||
      ((uintptr_t)sm_tab & 7) || ((uintptr_t)kernel_tab & 7))
    return ARGUS_ERR_INVALID_ARG;
  const AggLayout L = agg_layout(num_streams, num_regions);
  if (workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (reset_status) ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  if (num_streams == 0) {
    if (kernel_tab) { k_agg_init<<<64, 256, 0, stream>>>((u64*)kernel_tab, (u64)num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    if (sm_tab) { k_agg_init<<<64, 256, 0, stream>>>((u64*)sm_tab, (u64)num_sms * num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    return ARGUS_OK;
  }
  AggArgs a;
  a.intervals = intervals; a.interval_offsets = (const u64*)interval_offsets; a.ambig = ambig; a.ambig_offsets = (const u64*)ambig_offsets;
  a.num_streams = num_streams; a.warps_per_cta = warps_per_cta; a.num_ctas = num_streams / warps_per_cta;
  a.num_sms = num_sms; a.num_regions = num_regions; a.cta_sm = cta_sm;
  a.warp_tab = warp_tab ? (u64*)warp_tab : (u64*)((char*)workspace + L.warp);
  a.cta_tab = cta_tab ? (u64*)cta_tab : (u64*)((char*)workspace + L.cta);
  a.sm_tab = (u64*)sm_tab; a.kernel_tab = (u64*)kernel_tab; a.status = status;
  const size_t smem = (size_t)num_regions * sizeof(argus_agg_t);
  a.use_smem = smem <= kAggSmemLimit;
  if (a.use_smem && smem > 48 * 1024)
    ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_agg_streams, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  argus_prof_mark(ARGUS_PROF_AGGREGATE, stream, 0);
  k_agg_streams<<<num_streams, kAggThreads, a.use_smem ? smem : 0, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  argus_prof_mark(ARGUS_PROF_AGGREGATE, stream, 1);
  return agg_rollup(a, cta_tab, sm_tab, kernel_tab, stream);
}

extern "C" int argus_aggregate(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                               const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                               uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                               argus_agg_t* warp_tab, argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab,
                               argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return argus_internal_aggregate(intervals, interval_offsets, ambig, ambig_offsets, num_streams, warps_per_cta, cta_sm,
                                  num_sms, num_regions, warp_tab, cta_tab, sm_tab, kernel_tab, status, workspace,
                                  workspace_bytes, cuda_stream, true);
}
