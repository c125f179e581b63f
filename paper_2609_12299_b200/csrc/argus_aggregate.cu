// argus_aggregate.cu — argus_aggregate: intervals (+ ambiguity records) -> per-(scope, region) tables.
//
//   k_agg_streams_digest : argus_synthesize's pass: one CTA per stream reads the 8-byte digests the pairing
//                   kernel wrote beside the interval records (not the records) and gathers the stream's row
//                   in 100-byte shared-memory cells, with per-lane copies of the most frequent regions' cells;
//   k_agg_streams_compact : the same over the 48-byte records, with an optional scope: that stream's row in
//                   a compact shared-memory form (112 B per region: sums, min, max, a 16-bin window, so
//                   several CTAs fit an SM), for up to kAggCompactRegions regions;
//   k_agg_streams : the same with a full 576 B-per-region copy in shared memory when that fits, else on
//                   the global row itself. Integer atomics only: the result does not depend on thread order.
//   k_agg_cta     : CTA-scope cells = reduction over the warps of each CTA (plain loads, no atomics).
//   k_agg_init / k_agg_scatter : SM-scope and kernel-scope cells by atomic add/min/max of CTA cells.
//   k_agg_role    : warp-role cells = reduction over the CTAs of each warp index (plain loads).
//   k_agg_iter    : per-iteration cells (key = ctx - ctx_lo) of the intervals of a scope.
// A scope (iteration window, warp mask, SM mask, region mask) filters what k_agg_streams and
// k_agg_iter take in; without one everything is selected.
#include "argus_internal.cuh"

namespace {

constexpr int kAggThreads = 256;
constexpr u32 kCell = 72;  // u64 words per argus_agg_t
constexpr size_t kAggSmemLimit = 200 * 1024;
constexpr u32 kAggCompactRegions = 400;  // 112 B each: 44.8 KB of shared memory at most
constexpr size_t kIterScratchBytes = 32u << 20;  // workspace for private copies of an iteration table
constexpr u32 kIterMaxCopies = 32;

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
  // scope selection
  int scoped;
  u32 ctx_lo, ctx_hi;
  u64 warp_mask;
  const u32* sm_mask;
  const u32* region_mask;
  u64* role_tab;  // [W][R][72], nullable
  u64* iter_tab;  // [num_iters][R][72], nullable
  u32 num_iters;
  int iter_smem;
  u64* iter_copies;   // global path: private copies of the iteration table, one per group of blocks (null: none)
  u32 num_copies;
  int iter_inline;    // global path taken inside k_agg_streams_compact (one read of the intervals serves both)
  // overlap span selection in the same pass over the intervals (argus_synthesize); ov.ov_spans null = off
  ArgusFuseArgs ov;
  const u64* digest;  // digests of the intervals (k_agg_streams_digest), null = read the records
  u64 interval_limit; // records the interval array holds: a stream whose offsets reach beyond it is reported, not read
};


// The slots of a reserved chunk that the warp leaves unused are tagged, so that the list needs no clearing
// (a warp that holds no chunk has used == the chunk size: nothing to tag).
__device__ __forceinline__ void agg_ov_retire(const ArgusFuseArgs& ov, u64 base, u32 used, u32 lane) {
  for (u32 i = used + lane; i < ov.ov_chunk; i += 32)
    if (base + i < ov.ov_capacity) ov.ov_seg[base + i] = 0xffffffffu;
}

__device__ __forceinline__ bool mask_bit(const u32* mask, u32 i) { return !mask || ((mask[i >> 5] >> (i & 31)) & 1u); }

// Warp-role and SM tests of a scope: one answer per stream. 2 = bad cta_sm entry.
__device__ __forceinline__ int stream_in_scope(const AggArgs& a, u32 s) {
  if (!a.scoped) return 1;
  const u32 w = s % a.warps_per_cta;
  if (a.warp_mask != ~0ull && (w >= 64 || !((a.warp_mask >> w) & 1ull))) return 0;
  if (a.sm_mask) {
    const u32 m = a.cta_sm[s / a.warps_per_cta];
    if (m >= a.num_sms) return 2;
    if (!mask_bit(a.sm_mask, m)) return 0;
  }
  return 1;
}

// Iteration-window and region tests of a scope: one answer per record.
__device__ __forceinline__ bool record_in_scope(const AggArgs& a, u32 ctx, u32 region) {
  return !a.scoped || (ctx >= a.ctx_lo && ctx <= a.ctx_hi && mask_bit(a.region_mask, region));
}

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

// The same for a table in global memory that many blocks share: three atomics per interval instead of six. The
// count is left out (it is the sum of the histogram bins and is filled in afterwards) and min / max are
// only updated while they still move (a stale read only costs a redundant atomic).
__device__ __forceinline__ void agg_add_interval_lean(u64* tab, u32 region, u64 incl, u64 excl, u32 flags) {
  u64* c = tab + (size_t)region * kCell;
  atomicAdd(c + 1, incl);
  if (incl < __ldcg(c + 2)) atomicMin(c + 2, incl);
  if (incl > __ldcg(c + 3)) atomicMax(c + 3, incl);
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
    const int sel = stream_in_scope(a, s);
    if (sel == 2 && threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_INVALID_ARG, s, a.cta_sm[s / a.warps_per_cta]);
    if (hi < lo || hi > a.interval_limit) {
      if (threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
    } else if (sel == 1) {
      for (u64 i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const uint4* p = reinterpret_cast<const uint4*>(a.intervals + i);
        const uint4 q0 = __ldg(p), q1 = __ldg(p + 1), q2 = __ldg(p + 2);
        const u64 incl = (u64)q0.z | ((u64)q0.w << 32);
        const u64 excl = (u64)q1.x | ((u64)q1.y << 32);
        const u32 region = q1.z;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        if (!record_in_scope(a, q1.w, region)) continue;
        agg_add_interval(tab, region, incl, excl, q2.w >> 16);
      }
    }
    if (a.ambig && a.ambig_offsets && sel == 1) {
      const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
      for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
        const u32 region = a.ambig[i].tag >> 1;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        if (!record_in_scope(a, a.ambig[i].ctx, region)) continue;
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

__global__ void __launch_bounds__(kAggThreads) k_agg_streams_compact(AggArgs a) {
  extern __shared__ __align__(16) unsigned char sh_raw[];
  ArgusAggCell* const ctab = reinterpret_cast<ArgusAggCell*>(sh_raw);
  const u32 R = a.num_regions;
  const u32 cells = R * kCell;
  const u32 lane = threadIdx.x & 31;
  // overlap selection: bitmap of the regions that appear in a pair, and the pair list, after the table
  u32* const pairbits = reinterpret_cast<u32*>(ctab + R);
  u32* const pairs_sm = pairbits + (R + 31) / 32;
  const bool has_ov = a.ov.ov_spans != nullptr && a.ov.num_pairs != 0;
  // iteration table too large for shared memory: this block's private copy in global memory (or the table itself)
  u64* const iter_base = !a.iter_inline ? nullptr
                         : a.iter_copies ? a.iter_copies + (u64)(blockIdx.x % a.num_copies) * a.num_iters * cells : a.iter_tab;
  u64 ovc_base = 0;             // warp-uniform: current chunk of the global span list
  u32 ovc_used = a.ov.ov_chunk;  // none held yet
  if (has_ov) {
    for (u32 i = threadIdx.x; i < (R + 31) / 32; i += blockDim.x) pairbits[i] = 0;
    __syncthreads();
    for (u32 i = threadIdx.x; i < 2 * a.ov.num_pairs; i += blockDim.x) {
      const u32 r = a.ov.pairs[i];
      pairs_sm[i] = r;
      if (r < R) atomicOr(&pairbits[r >> 5], 1u << (r & 31));
    }
    __syncthreads();
  }
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    u64* row = a.warp_tab + (size_t)s * cells;
    // the global row takes flag counts' overflow path, bins outside the window and the ambiguity counters directly
    for (u32 i = threadIdx.x; i < cells; i += blockDim.x) row[i] = (i % kCell == 2) ? ~0ull : 0ull;
    argus_fuse_init(ctab, R, threadIdx.x, blockDim.x);
    __threadfence();
    __syncthreads();
    ArgusFuseCtx fx;
    fx.tab = ctab; fx.pairbits = nullptr; fx.row = row; fx.sm_index = 0;
    const u64 lo = a.interval_offsets[s], hi = a.interval_offsets[s + 1];
    const int sel = stream_in_scope(a, s);
    if (sel == 2 && threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_INVALID_ARG, s, a.cta_sm[s / a.warps_per_cta]);
    u32 sm_index = 0;
    if (has_ov) {
      const u32 m = a.cta_sm[s / a.warps_per_cta];
      if (m >= a.num_sms && threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_INVALID_ARG, s, m);
      sm_index = m < a.num_sms ? m : 0;
    }
    if (hi < lo || hi > a.interval_limit) {
      if (threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
    } else if (sel == 1) {
      // every lane of a warp runs the same number of rounds, so that spans can be appended a warp at a time
      for (u64 base = lo + (threadIdx.x & ~31u); base < hi; base += blockDim.x) {
        const u64 i = base + lane;
        bool cand = false;
        u32 region = 0;
        u64 t0 = 0, incl = 0;
        if (i < hi) {
          const uint4* p = reinterpret_cast<const uint4*>(a.intervals + i);
          const uint4 q0 = __ldg(p), q1 = __ldg(p + 1), q2 = __ldg(p + 2);
          region = q1.z;
          if (region >= R) {
            argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i);
          } else if (record_in_scope(a, q1.w, region)) {
            t0 = (u64)q0.x | ((u64)q0.y << 32);
            incl = (u64)q0.z | ((u64)q0.w << 32);
            const u64 excl = (u64)q1.x | ((u64)q1.y << 32);
            argus_fuse_aggregate(fx, region, incl, excl, q2.w >> 16);
            if (a.iter_inline) agg_add_interval_lean(iter_base + (u64)(q1.w - a.ctx_lo) * cells, region, incl, excl, q2.w >> 16);
            cand = has_ov && incl && ((pairbits[region >> 5] >> (region & 31)) & 1u);
          }
        }
        if (has_ov && __ballot_sync(0xffffffffu, cand)) {
          for (u32 k = 0; k < 2 * a.ov.num_pairs; ++k) {
            const bool pick = cand && pairs_sm[k] == region;
            const u32 bal = __ballot_sync(0xffffffffu, pick);
            if (!bal) continue;
            const u32 c = __popc(bal);
            if (ovc_used + c > a.ov.ov_chunk) {
              agg_ov_retire(a.ov, ovc_base, ovc_used, lane);
              u64 nb64 = 0;
              if (lane == 0) nb64 = atomicAdd(a.ov.ov_count, (u64)a.ov.ov_chunk);
              ovc_base = __shfl_sync(0xffffffffu, nb64, 0);
              ovc_used = 0;
            }
            if (pick) {
              const u64 slot = ovc_base + ovc_used + __popc(bal & ((1u << lane) - 1u));
              if (slot < a.ov.ov_capacity) {
                a.ov.ov_spans[slot] = make_ulonglong2(t0, t0 + incl);
                a.ov.ov_seg[slot] = ((k >> 1) * a.num_sms + sm_index) * 2 + (k & 1u);
              }
            }
            ovc_used += c;
          }
        }
      }
    }
    if (a.ambig && a.ambig_offsets && sel == 1) {
      const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
      for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
        const u32 region = a.ambig[i].tag >> 1;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        if (!record_in_scope(a, a.ambig[i].ctx, region)) continue;
        const u32 which = a.ambig[i].kind == ARGUS_AMBIG_UNMATCHED_END ? 6 : 5;
        atomicAdd(row + (size_t)region * kCell + which, 1ull);
        if (a.iter_inline) atomicAdd(iter_base + ((u64)(a.ambig[i].ctx - a.ctx_lo) * R + region) * kCell + which, 1ull);
      }
    }
    __syncthreads();
    argus_fuse_flush(ctab, row, R, threadIdx.x, blockDim.x);
    __syncthreads();
  }
  if (has_ov) agg_ov_retire(a.ov, ovc_base, ovc_used, lane);
}

// ---- the pass over the intervals' 8-byte digests (what argus_synthesize's pairing wrote beside the records) ----
// One CTA per stream, no scope. The stream's row is gathered in shared memory in cells of kDgWords = 25 32-bit
// words (an odd size: the cells of 32 different regions start in 32 different banks). A few regions usually own
// most intervals of a stream, and 32 lanes adding to one address serialise; so after a probe of the stream's
// first intervals the kDigestHot most frequent regions get 32 copies of their cell, one per lane (consecutive
// cells: never a bank conflict), which are folded into the region's cell when the stream ends. The last word of
// a region's cell (meta) holds what a lane needs to know about its region: histogram window base, copy slot,
// whether the region appears in an overlap pair. A digest marked wide (a duration of 2^23 ticks or more) sends
// its lane to the record and to 64-bit atomics on the global row. Overlap candidates take their start time from
// the record. The table is addressed with 32-bit shared-memory addresses and the fields by constant offsets.
constexpr u32 kDigestHot = 4;
constexpr u32 kDgSumInclLo = 0, kDgSumInclHi = 1, kDgSumExclLo = 2, kDgSumExclHi = 3, kDgMin = 4, kDgMax = 5, kDgFlag = 6,
              kDgCountOut = 7, kDgBins = 8, kDgMeta = kDgBins + kAggWindow, kDgWords = kDgMeta + 1;
static_assert(kDgWords % 2 == 1, "an odd cell size keeps the cells of different regions in different banks");
constexpr u32 kDgNone = 0xffu;                 // meta: bits 0-7 window base, 8-15 copy slot (kDgNone = unset), bit 16 in a pair
constexpr u32 kDigestProbe = 512;              // intervals looked at before the hot regions are chosen
constexpr u32 kDigestMinStream = 2048;         // shorter streams are gathered without copies

__host__ __device__ constexpr size_t digest_table_words(u32 R) { return (size_t)kDgWords * (R + kDigestHot * 32); }

template <u32 F> __device__ __forceinline__ u32 dg_add(u32 cell, u32 v) {  // returns the old value
  u32 old;
  asm volatile("atom.shared.add.u32 %0, [%1+%3], %2;" : "=r"(old) : "r"(cell), "r"(v), "n"(F * 4) : "memory");
  return old;
}
template <u32 F> __device__ __forceinline__ void dg_inc(u32 cell, u32 v) {
  asm volatile("red.shared.add.u32 [%0+%2], %1;" :: "r"(cell), "r"(v), "n"(F * 4) : "memory");
}
template <u32 F> __device__ __forceinline__ void dg_min(u32 cell, u32 v) {
  asm volatile("red.shared.min.u32 [%0+%2], %1;" :: "r"(cell), "r"(v), "n"(F * 4) : "memory");
}
template <u32 F> __device__ __forceinline__ void dg_max(u32 cell, u32 v) {
  asm volatile("red.shared.max.u32 [%0+%2], %1;" :: "r"(cell), "r"(v), "n"(F * 4) : "memory");
}

// The histogram bin of an interval whose bin is not inside the region's window as the lane saw it: the window
// may not be chosen yet (then this lane tries to), or the bin really lies outside (then it is counted here).
// Returns the bin's place in the window, or kAggWindow and beyond when it has been dealt with.
__device__ __noinline__ u32 digest_bin_rare(u32* meta_word, u32 bin, u32 cell, u64* row_bins) {
  const u32 m = *reinterpret_cast<volatile u32*>(meta_word);
  u32 hb = m & 0xffu;
  if (hb == kDgNone) {
    const u32 want = bin > 6u ? bin - 6u : 0u;   // bin <= 22: the window never passes bin 63
    const u32 prev = atomicCAS(meta_word, m, (m & ~0xffu) | want);  // only the window base changes while intervals are added
    hb = (prev & 0xffu) == kDgNone ? want : (prev & 0xffu);
  }
  const u32 rel = bin - hb;
  if (rel < kAggWindow) return rel;
  dg_inc<kDgCountOut>(cell, 1u);
  atomicAdd(row_bins + bin, 1ull);
  return 0xffffffffu;
}

// (512 threads, three blocks per SM: the same 48 warps as six blocks of 256, but a stream's set-up, the choice of its hot
// regions and the write-back of its row are shared by twice the threads; measured 2.33 ms against 2.45 ms on trace 3)
constexpr int kDgThreads = 512;
__global__ void __launch_bounds__(kDgThreads, 3) k_agg_streams_digest(AggArgs a) {
  extern __shared__ __align__(16) unsigned char sh_raw[];
  u32* const tab = reinterpret_cast<u32*>(sh_raw);
  const u32 R = a.num_regions;
  const u32 num_cells = R + kDigestHot * 32;
  u32* const pairbits = tab + (size_t)kDgWords * num_cells;
  u32* const pairs_sm = pairbits + (R + 31) / 32;
  __shared__ u32 hot_region[kDigestHot];
  const u32 tab_addr = (u32)__cvta_generic_to_shared(tab);
  const u32 cells = R * kCell;
  const u32 lane = threadIdx.x & 31;
  const bool has_ov = a.ov.ov_spans != nullptr && a.ov.num_pairs != 0;
  u64 ovc_base = 0;
  u32 ovc_used = a.ov.ov_chunk;  // none held yet
  for (u32 i = threadIdx.x; i < (R + 31) / 32; i += blockDim.x) pairbits[i] = 0;
  __syncthreads();
  if (has_ov) {
    for (u32 i = threadIdx.x; i < 2 * a.ov.num_pairs; i += blockDim.x) {
      const u32 r = a.ov.pairs[i];
      pairs_sm[i] = r;
      if (r < R) atomicOr(&pairbits[r >> 5], 1u << (r & 31));
    }
    __syncthreads();
  }
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    u64* row = a.warp_tab + (size_t)s * cells;
    for (u32 i = threadIdx.x; i < cells; i += blockDim.x) row[i] = (i % kCell == 2) ? ~0ull : 0ull;
    for (u32 i = threadIdx.x; i < kDgWords * num_cells; i += blockDim.x) {
      const u32 f = i % kDgWords, c = i / kDgWords;
      u32 v = f == kDgMin ? 0xffffffffu : 0u;
      if (f == kDgMeta && c < R) v = kDgNone | (kDgNone << 8) | (((pairbits[c >> 5] >> (c & 31)) & 1u) << 16);
      tab[i] = v;
    }
    if (threadIdx.x < kDigestHot) hot_region[threadIdx.x] = 0xffffffffu;
    __threadfence();
    __syncthreads();
    const u64 lo = a.interval_offsets[s], hi = a.interval_offsets[s + 1];
    u32 sm_index = 0;
    if (has_ov) {
      const u32 m = a.cta_sm[s / a.warps_per_cta];
      if (m >= a.num_sms && threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_INVALID_ARG, s, m);
      sm_index = m < a.num_sms ? m : 0;
    }
    if (hi < lo || hi > a.interval_limit || ((hi - lo) >> 32)) {
      if (threadIdx.x == 0) argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
    } else {
      const u32 n = (u32)(hi - lo);
      const u64* const dgs = a.digest + lo;
      const argus_interval_t* const ivs = a.intervals + lo;
      // two legs: the probe (every interval into its region's cell), then, hot regions chosen, the rest of the stream
      const u32 probe_end = n >= kDigestMinStream ? kDigestProbe : n;
      for (int leg = 0; leg < 2; ++leg) {
        const u32 leg_lo = leg ? probe_end : 0u, leg_hi = leg ? n : probe_end;
        if (leg && leg_lo < leg_hi) {
          // warp 0 ranks the regions by their counts so far; kDigestHot rounds of a warp-wide maximum
          if (threadIdx.x < 32) {
            for (u32 h = 0; h < kDigestHot; ++h) {
              u32 best = 0;
              for (u32 r = lane; r < R; r += 32) {
                const u32* c = tab + r * kDgWords;
                if (((c[kDgMeta] >> 8) & 0xffu) != kDgNone) continue;
                u32 cnt = c[kDgCountOut];
#pragma unroll
                for (u32 j = 0; j < kAggWindow; ++j) cnt += c[kDgBins + j];
                const u32 key = ((cnt > 0xffffu ? 0xffffu : cnt) << 16) | r;
                best = key > best ? key : best;
              }
              const u32 top = __reduce_max_sync(0xffffffffu, best);
              if ((top >> 16) < kDigestProbe / 64) break;  // not worth a set of copies
              if (lane == 0) { atomicAnd(&tab[(top & 0xffffu) * kDgWords + kDgMeta], ~0xff00u | (h << 8)); hot_region[h] = top & 0xffffu; }
              __syncwarp();
            }
          }
          __syncthreads();
        }
        // every lane of a warp runs the same number of rounds, so that spans can be appended a warp at a time
        u32 b = leg_lo + (threadIdx.x & ~31u);
        // digests are asked for two rounds ahead (one round is shorter than a loaded DRAM access)
        u64 dg_next = b + lane < leg_hi ? __ldg(dgs + b + lane) : 0ull;
        u64 dg_next2 = b + lane + kDgThreads < leg_hi ? __ldg(dgs + b + lane + kDgThreads) : 0ull;
        for (; b < leg_hi; b += kDgThreads) {
          const u32 i = b + lane;
          const u64 dg = dg_next;
          dg_next = dg_next2;
          dg_next2 = i + 2 * kDgThreads < leg_hi ? __ldg(dgs + i + 2 * kDgThreads) : 0ull;
          const u32 dlo = (u32)dg, dhi = (u32)(dg >> 32);
          const bool in = i < leg_hi;
          const u32 region = dlo & 0xffffu;
          const bool ok = in && region < R;
          const u32 rsafe = ok ? region : 0u;
          const u32 incl = (dlo >> 18) | ((dhi & 0x1ffu) << 14), excl = dhi >> 9;
          const u32 meta = tab[rsafe * kDgWords + kDgMeta];
          const u32 slot = (meta >> 8) & 0xffu;
          const u32 cell = tab_addr + (slot != kDgNone ? R + slot * 32 + lane : rsafe) * (kDgWords * 4);
          // the common case without a branch: a lane that does not take part (past the end, wide, bad region)
          // adds nothing; whatever is rare (a carry, a flag, a bin outside the window, ...) is settled in one place
          const bool take = ok && !(dlo & (1u << 17));
          const u32 vi = take ? incl : 0u, ve = take ? excl : 0u;
          const u32 old_i = dg_add<kDgSumInclLo>(cell, vi);
          const u32 old_e = dg_add<kDgSumExclLo>(cell, ve);
          dg_min<kDgMin>(cell, take ? incl : 0xffffffffu);
          dg_max<kDgMax>(cell, vi);
          const u32 bin = 31u - (u32)__clz((int)(incl | 1u));
          const u32 rel = bin - (meta & 0xffu);
          const bool in_win = take && rel < kAggWindow;
          dg_inc<kDgBins>(cell + (in_win ? rel : 0u) * 4, in_win ? 1u : 0u);
          u64 span = vi;
          const bool rare = in && ((dlo & (3u << 16)) || !ok || old_i + vi < old_i || old_e + ve < old_e || !in_win);
          if (rare) {
            if (!ok) {
              argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, lo + i);
            } else if (!take) {
              u64* const row_cell = row + (size_t)region * kCell;
              const uint4* p = reinterpret_cast<const uint4*>(ivs + i);
              const uint4 q0 = __ldg(p), q1 = __ldg(p + 1);
              span = (u64)q0.z | ((u64)q0.w << 32);
              atomicAdd(row_cell + 0, 1ull);
              atomicAdd(row_cell + 1, span);
              atomicMin(row_cell + 2, span);
              atomicMax(row_cell + 3, span);
              atomicAdd(row_cell + 4, (u64)q1.x | ((u64)q1.y << 32));
              if (dlo & (1u << 16)) atomicAdd(row_cell + 7, 1ull);
              atomicAdd(row_cell + 8 + log2_bin(span), 1ull);
            } else {
              if (old_i + vi < old_i) dg_inc<kDgSumInclHi>(cell, 1u);
              if (old_e + ve < old_e) dg_inc<kDgSumExclHi>(cell, 1u);
              if (dlo & (1u << 16)) dg_inc<kDgFlag>(cell, 1u);
              if (!in_win) {
                const u32 r2 = digest_bin_rare(tab + region * kDgWords + kDgMeta, bin, cell, row + (size_t)region * kCell + 8);
                if (r2 < kAggWindow) dg_inc<kDgBins>(cell + r2 * 4, 1u);
              }
            }
          }
          const bool cand = ok && ((meta >> 16) & 1u) && span;
          if (has_ov && __ballot_sync(0xffffffffu, cand)) {
            u64 t0 = 0;
            if (cand) t0 = __ldg(reinterpret_cast<const u64*>(ivs + i));
            for (u32 k = 0; k < 2 * a.ov.num_pairs; ++k) {
              const bool pick = cand && pairs_sm[k] == region;
              const u32 bal = __ballot_sync(0xffffffffu, pick);
              if (!bal) continue;
              const u32 c = __popc(bal);
              if (ovc_used + c > a.ov.ov_chunk) {
                agg_ov_retire(a.ov, ovc_base, ovc_used, lane);
                u64 nb64 = 0;
                if (lane == 0) nb64 = atomicAdd(a.ov.ov_count, (u64)a.ov.ov_chunk);
                ovc_base = __shfl_sync(0xffffffffu, nb64, 0);
                ovc_used = 0;
              }
              if (pick) {
                const u64 slot_o = ovc_base + ovc_used + __popc(bal & ((1u << lane) - 1u));
                if (slot_o < a.ov.ov_capacity) {
                  a.ov.ov_spans[slot_o] = make_ulonglong2(t0, t0 + span);
                  a.ov.ov_seg[slot_o] = ((k >> 1) * a.num_sms + sm_index) * 2 + (k & 1u);
                }
              }
              ovc_used += c;
            }
          }
        }
        __syncthreads();
      }
    }
    if (a.ambig && a.ambig_offsets) {
      const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
      for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
        const u32 region = a.ambig[i].tag >> 1;
        if (region >= R) { argus_set_error(a.status, ARGUS_ERR_BAD_REGION, s, i); continue; }
        atomicAdd(row + (size_t)region * kCell + (a.ambig[i].kind == ARGUS_AMBIG_UNMATCHED_END ? 6 : 5), 1ull);
      }
    }
    __syncthreads();
    // fold the lanes' copies into their region's cell: one thread per (hot region, field)
    if (threadIdx.x < kDigestHot * kDgMeta) {
      const u32 h = threadIdx.x / kDgMeta, f = threadIdx.x % kDgMeta;
      const u32 r = hot_region[h];
      if (r != 0xffffffffu && f != kDgSumInclHi && f != kDgSumExclHi) {
        const u32* src = tab + (R + h * 32) * kDgWords + f;
        u32* dst = tab + r * kDgWords + f;
        if (f == kDgSumInclLo || f == kDgSumExclLo) {
          u64 sum = (u64)dst[0] | ((u64)dst[1] << 32);
          for (u32 l = 0; l < 32; ++l) sum += (u64)src[l * kDgWords] | ((u64)src[l * kDgWords + 1] << 32);
          dst[0] = (u32)sum;
          dst[1] = (u32)(sum >> 32);
        } else {
          u32 acc = dst[0];
          for (u32 l = 0; l < 32; ++l) {
            const u32 v = src[l * kDgWords];
            acc = f == kDgMin ? (v < acc ? v : acc) : f == kDgMax ? (v > acc ? v : acc) : acc + v;
          }
          dst[0] = acc;
        }
      }
    }
    __syncthreads();
    // the regions' cells into the global row, which already holds the wide intervals, the bins outside the
    // windows and the ambiguity counters: everything is combined, nothing overwritten
    constexpr u32 kItems = 6 + kAggWindow;
    for (u32 i = threadIdx.x; i < R * kItems; i += blockDim.x) {
      const u32 r = i % R, f = i / R;
      const u32* c = tab + r * kDgWords;
      u64* cell = row + (size_t)r * kCell;
      switch (f) {
        case 0: {
          u64 cnt = c[kDgCountOut];
#pragma unroll
          for (u32 j = 0; j < kAggWindow; ++j) cnt += c[kDgBins + j];
          if (cnt) atomicAdd(cell + 0, cnt);
          break;
        }
        case 1: { const u64 v = (u64)c[kDgSumInclLo] | ((u64)c[kDgSumInclHi] << 32); if (v) atomicAdd(cell + 1, v); break; }
        case 2: { const u32 v = c[kDgMin]; if (v != 0xffffffffu) atomicMin(cell + 2, (u64)v); break; }
        case 3: { const u32 v = c[kDgMax]; if (v) atomicMax(cell + 3, (u64)v); break; }
        case 4: { const u64 v = (u64)c[kDgSumExclLo] | ((u64)c[kDgSumExclHi] << 32); if (v) atomicAdd(cell + 4, v); break; }
        case 5: { const u32 v = c[kDgFlag]; if (v) atomicAdd(cell + 7, (u64)v); break; }
        default: {
          const u32 j = f - 6;
          const u32 v = c[kDgBins + j];
          if (v) atomicAdd(cell + 8 + (c[kDgMeta] & 0xffu) + j, (u64)v);
        }
      }
    }
    __syncthreads();
  }
  if (has_ov) agg_ov_retire(a.ov, ovc_base, ovc_used, lane);
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

// role_tab[w][r][j] = reduce over c of warp_tab[c*W + w][r][j]
__global__ void __launch_bounds__(256) k_agg_role(AggArgs a) {
  const u64 per_row = (u64)a.num_regions * kCell;
  const u64 n = (u64)a.warps_per_cta * per_row;
  for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (u64)gridDim.x * blockDim.x) {
    const u64 w = i / per_row, rem = i % per_row;
    const u32 field = (u32)(rem % kCell);
    const u64* src = a.warp_tab + w * per_row + rem;
    u64 acc = src[0];
    for (u32 c = 1; c < a.num_ctas; ++c) acc = combine(field, acc, src[(u64)c * a.warps_per_cta * per_row]);
    a.role_tab[i] = acc;
  }
}

// iter_tab[ctx - ctx_lo][r]: selected intervals and ambiguity records keyed by iteration. A block gathers its
// streams in a shared-memory copy of the table when that fits and adds the non-empty cells to the global
// table (initialised by k_agg_init) at the end; otherwise it updates the global table record by record.
__global__ void __launch_bounds__(kAggThreads) k_agg_iter(AggArgs a) {
  extern __shared__ __align__(16) u64 sh_tab[];
  const u32 R = a.num_regions;
  const u64 cells = (u64)a.num_iters * R * kCell;
  // too large for shared memory: blocks add to one of a few private copies in global memory, which spreads the
  // atomics over more addresses; k_agg_iter_reduce combines the copies afterwards
  u64* tab = a.iter_smem ? sh_tab : a.iter_copies ? a.iter_copies + (u64)(blockIdx.x % a.num_copies) * cells : a.iter_tab;
  if (a.iter_smem) {
    for (u64 i = threadIdx.x; i < cells; i += blockDim.x) sh_tab[i] = (i % kCell == 2) ? ~0ull : 0ull;
    __syncthreads();
  }
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    if (stream_in_scope(a, s) != 1) continue;  // a bad cta_sm entry is reported by k_agg_streams
    const u64 lo = a.interval_offsets[s], hi = a.interval_offsets[s + 1];
    for (u64 i = lo + threadIdx.x; i < hi && hi >= lo && hi <= a.interval_limit; i += blockDim.x) {
      const uint4* p = reinterpret_cast<const uint4*>(a.intervals + i);
      const uint4 q1 = __ldg(p + 1);
      const u32 region = q1.z, ctx = q1.w;
      if (region >= R || !record_in_scope(a, ctx, region)) continue;
      const uint4 q0 = __ldg(p), q2 = __ldg(p + 2);
      u64* row = tab + (u64)(ctx - a.ctx_lo) * R * kCell;
      const u64 incl = (u64)q0.z | ((u64)q0.w << 32), excl = (u64)q1.x | ((u64)q1.y << 32);
      if (a.iter_smem) agg_add_interval(row, region, incl, excl, q2.w >> 16);
      else agg_add_interval_lean(row, region, incl, excl, q2.w >> 16);
    }
    if (a.ambig && a.ambig_offsets) {
      const u64 alo = a.ambig_offsets[s], ahi = a.ambig_offsets[s + 1];
      for (u64 i = alo + threadIdx.x; i < ahi && ahi >= alo; i += blockDim.x) {
        const u32 region = a.ambig[i].tag >> 1, ctx = a.ambig[i].ctx;
        if (region >= R || !record_in_scope(a, ctx, region)) continue;
        atomicAdd(tab + ((u64)(ctx - a.ctx_lo) * R + region) * kCell + (a.ambig[i].kind == ARGUS_AMBIG_UNMATCHED_END ? 6 : 5), 1ull);
      }
    }
  }
  if (a.iter_smem) {
    __syncthreads();
    for (u64 i = threadIdx.x; i < cells; i += blockDim.x) {
      const u32 field = (u32)(i % kCell);
      const u64 v = sh_tab[i];
      if (field == 2 ? v == ~0ull : v == 0ull) continue;
      u64* d = a.iter_tab + i;
      if (field == 2) atomicMin(d, v); else if (field == 3) atomicMax(d, v); else atomicAdd(d, v);
    }
  }
}

// iter_tab[i] = combination of cell word i over the private copies (none: iter_tab holds the sums already);
// the interval count of a cell, which the global path leaves out, is the sum of its histogram bins.
__global__ void __launch_bounds__(256) k_agg_iter_reduce(AggArgs a) {
  const u64 cells = (u64)a.num_iters * a.num_regions * kCell;
  if (a.iter_copies) {
    for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < cells; i += (u64)gridDim.x * blockDim.x) {
      const u32 field = (u32)(i % kCell);
      if (field == 0) continue;
      u64 acc = a.iter_copies[i];
      for (u32 c = 1; c < a.num_copies; ++c) acc = combine(field, acc, a.iter_copies[(u64)c * cells + i]);
      a.iter_tab[i] = acc;
    }
  }
  for (u64 cell = (u64)blockIdx.x * blockDim.x + threadIdx.x; cell < cells / kCell; cell += (u64)gridDim.x * blockDim.x) {
    u64 n = 0;
    for (u32 b = 0; b < 64; ++b) {
      u64 v = 0;
      if (a.iter_copies) for (u32 c = 0; c < a.num_copies; ++c) v += a.iter_copies[(u64)c * cells + cell * kCell + 8 + b];
      else v = a.iter_tab[cell * kCell + 8 + b];
      n += v;
    }
    a.iter_tab[cell * kCell] = n;
  }
}

struct AggLayout { size_t warp, cta, iter, total; };

AggLayout agg_layout(uint32_t num_streams, uint32_t num_regions) {
  AggLayout L;
  const size_t row = (size_t)num_regions * sizeof(argus_agg_t);
  L.warp = 0;
  L.cta = argus_align_up((size_t)num_streams * row, 256);
  L.iter = L.cta + argus_align_up((size_t)num_streams * row, 256);  // C <= S
  L.total = L.iter + kIterScratchBytes;
  return L;
}

}  // namespace

extern "C" size_t argus_aggregate_workspace_bytes(uint64_t /*num_intervals*/, uint32_t num_streams, uint32_t num_regions) {
  return agg_layout(num_streams, num_regions).total + 256;
}

int argus_internal_aggregate_scoped(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                                    const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                                    uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                                    const argus_scope_t* scope, argus_agg_t* warp_tab, argus_agg_t* cta_tab,
                                    argus_agg_t* sm_tab, argus_agg_t* kernel_tab, argus_agg_t* role_tab,
                                    argus_agg_t* iter_tab, argus_status_t* status, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream, bool reset_status,
                                    const ArgusFuseArgs* ov_select, const uint64_t* digest, uint64_t interval_limit) {
  if (!interval_offsets || !status || !workspace) return ARGUS_ERR_INVALID_ARG;
  if (ov_select && (num_regions > kAggCompactRegions || ov_select->num_pairs > kFuseMaxPairs)) return ARGUS_ERR_INVALID_ARG;
  if (warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ARGUS_ERR_INVALID_ARG;
  if (num_regions == 0 || num_regions > ARGUS_MAX_REGIONS) return ARGUS_ERR_INVALID_ARG;
  if ((sm_tab || (scope && scope->sm_mask)) && ((!cta_sm && num_streams) || num_sms == 0)) return ARGUS_ERR_INVALID_ARG;
  if (scope && scope->ctx_hi < scope->ctx_lo) return ARGUS_ERR_INVALID_ARG;
  if (iter_tab && (!scope || scope->ctx_hi - scope->ctx_lo >= ARGUS_MAX_ITER_ROWS)) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)intervals & 15) || ((uintptr_t)workspace & 255) || ((uintptr_t)warp_tab & 7) || ((uintptr_t)cta_tab & 7) ||
      ((uintptr_t)sm_tab & 7) || ((uintptr_t)kernel_tab & 7) || ((uintptr_t)role_tab & 7) || ((uintptr_t)iter_tab & 7))
    return ARGUS_ERR_INVALID_ARG;
  const AggLayout L = agg_layout(num_streams, num_regions);
  if (workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (reset_status) ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  const u32 num_iters = iter_tab ? scope->ctx_hi - scope->ctx_lo + 1 : 0;
  if (kernel_tab) { k_agg_init<<<16, 256, 0, stream>>>((u64*)kernel_tab, (u64)num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
  if (sm_tab) { k_agg_init<<<296, 256, 0, stream>>>((u64*)sm_tab, (u64)num_sms * num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
  if (num_streams == 0) {
    if (role_tab) { k_agg_init<<<64, 256, 0, stream>>>((u64*)role_tab, (u64)warps_per_cta * num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    if (iter_tab) { k_agg_init<<<64, 256, 0, stream>>>((u64*)iter_tab, (u64)num_iters * num_regions * kCell); ARGUS_CHECK_LAUNCH(); }
    return ARGUS_OK;
  }
  AggArgs a;
  a.intervals = intervals; a.interval_offsets = (const u64*)interval_offsets; a.ambig = ambig; a.ambig_offsets = (const u64*)ambig_offsets;
  a.num_streams = num_streams; a.warps_per_cta = warps_per_cta; a.num_ctas = num_streams / warps_per_cta;
  a.num_sms = num_sms; a.num_regions = num_regions; a.cta_sm = cta_sm;
  a.warp_tab = warp_tab ? (u64*)warp_tab : (u64*)((char*)workspace + L.warp);
  a.cta_tab = cta_tab ? (u64*)cta_tab : (u64*)((char*)workspace + L.cta);
  a.sm_tab = (u64*)sm_tab; a.kernel_tab = (u64*)kernel_tab; a.status = status;
  a.scoped = scope != nullptr;
  a.ctx_lo = scope ? scope->ctx_lo : 0; a.ctx_hi = scope ? scope->ctx_hi : 0xffffffffu;
  a.warp_mask = scope ? scope->warp_mask : ~0ull;
  a.sm_mask = scope ? scope->sm_mask : nullptr; a.region_mask = scope ? scope->region_mask : nullptr;
  a.role_tab = (u64*)role_tab; a.iter_tab = (u64*)iter_tab; a.num_iters = num_iters;
  if (ov_select) { a.ov = *ov_select; } else { a.ov.ov_spans = nullptr; a.ov.num_pairs = 0; a.ov.ov_chunk = 256; }
  a.digest = !scope && !role_tab && !iter_tab && num_regions <= kAggCompactRegions ? (const u64*)digest : nullptr;
  a.interval_limit = interval_limit;
  const size_t smem = (size_t)num_regions * sizeof(argus_agg_t);
  a.use_smem = smem <= kAggSmemLimit;
  const size_t iter_bytes = (size_t)num_iters * smem;
  a.iter_smem = iter_tab && iter_bytes <= kAggSmemLimit;
  a.iter_copies = nullptr; a.num_copies = 0;
  if (iter_tab && !a.iter_smem && 2 * iter_bytes <= kIterScratchBytes) {
    a.num_copies = (u32)(kIterScratchBytes / iter_bytes < kIterMaxCopies ? kIterScratchBytes / iter_bytes : kIterMaxCopies);
    a.iter_copies = (u64*)((char*)workspace + L.iter);
  }
  const size_t need = a.use_smem ? smem : 0, need_iter = a.iter_smem ? iter_bytes : 0;
  if (need > 48 * 1024)
    ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_agg_streams, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need));
  if (need_iter > 48 * 1024)
    ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_agg_iter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need_iter));
  const u64 iter_cells = (u64)num_iters * num_regions * kCell;
  a.iter_inline = iter_tab && !a.iter_smem && num_regions <= kAggCompactRegions;
  if (iter_tab) {
    if (a.iter_copies) {
      k_agg_init<<<592, 256, 0, stream>>>(a.iter_copies, iter_cells * a.num_copies);
    } else {
      k_agg_init<<<296, 256, 0, stream>>>((u64*)iter_tab, iter_cells);
    }
    ARGUS_CHECK_LAUNCH();
  }
  argus_prof_mark(ARGUS_PROF_AGGREGATE, stream, 0);
  if (num_regions <= kAggCompactRegions) {
    const size_t compact = (size_t)num_regions * sizeof(ArgusAggCell) + ((num_regions + 31) / 32) * 4 + (size_t)a.ov.num_pairs * 8;
    if (compact > 48 * 1024)
      ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_agg_streams_compact, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)compact));
    if (a.digest) {
      const size_t dg = digest_table_words(num_regions) * 4 + ((num_regions + 31) / 32) * 4 + (size_t)a.ov.num_pairs * 8;
      if (dg > 48 * 1024)
        ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_agg_streams_digest, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dg));
      k_agg_streams_digest<<<num_streams, kDgThreads, dg, stream>>>(a);
    } else {
      k_agg_streams_compact<<<num_streams, kAggThreads, compact, stream>>>(a);
    }
  } else {
    k_agg_streams<<<num_streams, kAggThreads, need, stream>>>(a);
  }
  ARGUS_CHECK_LAUNCH();
  argus_prof_mark(ARGUS_PROF_AGGREGATE, stream, 1);
  if (iter_tab) {
    if (!a.iter_inline) {
      const unsigned iter_grid = a.iter_smem ? 296u : 148u * 8u;
      k_agg_iter<<<num_streams < iter_grid ? num_streams : iter_grid, kAggThreads, need_iter, stream>>>(a);
      ARGUS_CHECK_LAUNCH();
    }
    if (!a.iter_smem) {
      k_agg_iter_reduce<<<296, 256, 0, stream>>>(a);
      ARGUS_CHECK_LAUNCH();
    }
  }
  if (role_tab) {
    k_agg_role<<<296, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  if (cta_tab || sm_tab || kernel_tab) {
    k_agg_cta<<<1184, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  if (sm_tab || kernel_tab) {
    k_agg_scatter<<<1184, 256, 0, stream>>>(a);
    ARGUS_CHECK_LAUNCH();
  }
  return ARGUS_OK;
}

int argus_internal_aggregate(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                             const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                             uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                             argus_agg_t* warp_tab, argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab,
                             argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream,
                             bool reset_status, uint64_t interval_limit) {
  return argus_internal_aggregate_scoped(intervals, interval_offsets, ambig, ambig_offsets, num_streams, warps_per_cta, cta_sm,
                                         num_sms, num_regions, nullptr, warp_tab, cta_tab, sm_tab, kernel_tab, nullptr,
                                         nullptr, status, workspace, workspace_bytes, cuda_stream, reset_status, nullptr,
                                         nullptr, interval_limit);
}

bool argus_aggregate_can_select_overlap(uint32_t num_regions, uint32_t num_pairs) {
  return num_regions <= kAggCompactRegions && num_pairs <= kFuseMaxPairs;
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

extern "C" int argus_aggregate_scoped(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                                      const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                                      uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                                      const argus_scope_t* scope, argus_agg_t* warp_tab, argus_agg_t* cta_tab,
                                      argus_agg_t* sm_tab, argus_agg_t* kernel_tab, argus_agg_t* role_tab,
                                      argus_agg_t* iter_tab, argus_status_t* status, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  return argus_internal_aggregate_scoped(intervals, interval_offsets, ambig, ambig_offsets, num_streams, warps_per_cta, cta_sm,
                                         num_sms, num_regions, scope, warp_tab, cta_tab, sm_tab, kernel_tab, role_tab, iter_tab,
                                         status, workspace, workspace_bytes, cuda_stream, true, nullptr);
}
