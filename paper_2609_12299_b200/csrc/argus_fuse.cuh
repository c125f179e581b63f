// argus_fuse.cuh — what the pairing kernels and the aggregation passes share: the compact shared-memory
// form of a stream's row of the warp-scope table, the 8-byte digest of an interval, and the arguments of
// overlap span selection.
//
// Compact row: per region the sums, min, max, counts and a 16-bin window of the 64-bin log2 histogram
// (bins outside the window go straight to the global row); the CTA that aggregates a stream keeps the row
// in shared memory and writes it to the global row when the stream ends. All updates are integer atomics,
// so thread order is irrelevant.
// Overlap selection: spans of intervals whose region appears in a (producer, consumer) pair are appended to
// a global list tagged with their (pair, SM, role) segment; the overlap kernels take it from there.
#ifndef ARGUS_FUSE_CUH_
#define ARGUS_FUSE_CUH_

#include "argus_common.cuh"

constexpr u32 kAggWindow = 16;          // histogram bins kept in shared memory per region
constexpr u32 kAggUnset = 0xffffffffu;  // window base not chosen yet
constexpr u32 kFuseMaxPairs = 128;      // span selection keeps the pair list (8 bytes a pair) in shared memory
constexpr u32 kAggCellWords = 72;       // u64 words of one argus_agg_t

struct ArgusAggCell {  // 112 bytes
  u64 sum_incl, sum_excl, min_incl, max_incl;
  u32 count_out, nflag, hbase, pad;  // count_out: intervals whose bin fell outside the window
  u32 h[kAggWindow];                 // the interval count of the region is count_out + the sum of these
};

struct ArgusFuseArgs {
  u64* warp_tab;          // unused by span selection (kept for layout)
  const u32* cta_sm;      // [C]
  u32 warps_per_cta, num_sms;
  const u32* pairs;       // [K][2]
  u32 num_pairs;
  ulonglong2* ov_spans;   // appended (start, end); null = no fused overlap selection
  u32* ov_seg;            // segment of each appended span: (pair * num_sms + sm) * 2 + role
  u64 ov_capacity;
  u32 ov_chunk;           // list slots a warp reserves at a time: a power of two from 32 to 256
  u64* ov_count;          // spans appended so far (may exceed the capacity)
};

struct ArgusFuseCtx {     // per CTA, for the stream it is aggregating
  ArgusAggCell* tab;      // shared memory [R]; null = aggregation off
  const u32* pairbits;    // shared memory bitmap over regions: region appears in some pair; null = overlap off
  u64* row;               // global row of this stream in the warp-scope table
  u32 sm_index;           // SM of this stream's CTA
};

// Digest of an interval (8 bytes): all that aggregation needs of it. argus_synthesize lets the pairing kernels
// write one per interval record, at the same position, so that the aggregation pass reads 8 bytes per interval
// instead of 48. Bits 0-15 region, 16 any flag set, 17 wide (a duration does not fit: take both from the
// record; the duration bits then mean nothing), 18-40 inclusive, 41-63 exclusive duration.
constexpr u32 kDigestBits = 23;
__device__ __forceinline__ u64 argus_digest_pack(u32 region, u64 incl, u64 excl, u32 flags) {
  const u32 il = (u32)incl, el = (u32)excl;
  const bool wide = (((il | el) >> kDigestBits) | (u32)(incl >> 32) | (u32)(excl >> 32)) != 0;
  const u32 lo = region | (flags ? 1u << 16 : 0u) | (wide ? 1u << 17 : 0u) | (il << 18);
  const u32 hi = ((il >> 14) & 0x1ffu) | (el << 9);
  return (u64)lo | ((u64)hi << 32);
}

__device__ __forceinline__ u32 argus_log2_bin(u64 d) { return d ? 63u - (u32)__clzll((long long)d) : 0u; }

// 64-bit add as native 32-bit atomics; each carry is propagated exactly once
__device__ __forceinline__ void argus_atomic_add64_split(u64* p64, u64 v) {
  u32* p = reinterpret_cast<u32*>(p64);
  const u32 lo = (u32)v, hi = (u32)(v >> 32);
  if (lo) {
    const u32 old = atomicAdd(p, lo);
    if (old + lo < old) atomicAdd(p + 1, 1u);
  }
  if (hi) atomicAdd(p + 1, hi);
}

__device__ __forceinline__ void argus_fuse_init(ArgusAggCell* tab, u32 num_regions, u32 tid, u32 nthreads) {
  u32* w = reinterpret_cast<u32*>(tab);
  constexpr u32 kWords = sizeof(ArgusAggCell) / 4;
  for (u32 i = tid; i < num_regions * kWords; i += nthreads) {
    const u32 f = i % kWords;
    w[i] = (f == 4 || f == 5 || f == 10) ? 0xffffffffu : 0u;  // min_incl = all ones, hbase = unset
  }
}

// sums of one cell (the part a thread may instead keep in registers for hot regions)
__device__ __forceinline__ void argus_fuse_agg_sums(ArgusAggCell& c, u64 sum_incl, u64 sum_excl) {
  argus_atomic_add64_split(&c.sum_incl, sum_incl);
  argus_atomic_add64_split(&c.sum_excl, sum_excl);
}

// min, max, flag count and histogram bin of one interval; the bin also counts the interval
__device__ __forceinline__ void argus_fuse_agg_rest(ArgusAggCell& c, u64* row, u32 region, u64 incl, u32 flags) {
  if (incl < *reinterpret_cast<volatile u64*>(&c.min_incl)) atomicMin(&c.min_incl, incl);
  if (incl > *reinterpret_cast<volatile u64*>(&c.max_incl)) atomicMax(&c.max_incl, incl);
  if (flags) atomicAdd(&c.nflag, 1u);
  const u32 bin = argus_log2_bin(incl);
  u32 hb = *reinterpret_cast<volatile u32*>(&c.hbase);
  if (hb == kAggUnset) {
    const u32 want = bin > 6u ? (bin - 6u > 64u - kAggWindow ? 64u - kAggWindow : bin - 6u) : 0u;
    const u32 old = atomicCAS(&c.hbase, kAggUnset, want);
    hb = old == kAggUnset ? want : old;
  }
  const u32 rel = bin - hb;
  if (rel < kAggWindow) {
    atomicAdd(&c.h[rel], 1u);
  } else {
    atomicAdd(&c.count_out, 1u);
    atomicAdd(row + (size_t)region * kAggCellWords + 8 + bin, 1ull);
  }
}

__device__ __forceinline__ void argus_fuse_aggregate(const ArgusFuseCtx& fx, u32 region, u64 incl, u64 excl, u32 flags) {
  ArgusAggCell& c = fx.tab[region];
  argus_fuse_agg_sums(c, incl, excl);
  argus_fuse_agg_rest(c, fx.row, region, incl, flags);
}

__device__ __forceinline__ void argus_fuse_flush(const ArgusAggCell* tab, u64* row, u32 num_regions, u32 tid, u32 nthreads) {
  constexpr u32 kItems = 8 + kAggWindow;
  for (u32 i = tid; i < num_regions * kItems; i += nthreads) {
    const u32 r = i / kItems, f = i % kItems;
    const ArgusAggCell& c = tab[r];
    u64* cell = row + (size_t)r * kAggCellWords;
    switch (f) {
      case 0: {
        u64 n = c.count_out;
#pragma unroll
        for (u32 j = 0; j < kAggWindow; ++j) n += c.h[j];
        cell[0] = n;
        break;
      }
      case 1: cell[1] = c.sum_incl; break;
      case 2: cell[2] = c.min_incl; break;
      case 3: cell[3] = c.max_incl; break;
      case 4: cell[4] = c.sum_excl; break;
      case 5: case 6: break;  // ambiguity counters are added later from the ambiguity records
      case 7: cell[7] = c.nflag; break;
      default: {
        const u32 j = f - 8;
        if (c.h[j]) atomicAdd(cell + 8 + c.hbase + j, (u64)c.h[j]);
      }
    }
  }
}

#endif  // ARGUS_FUSE_CUH_
