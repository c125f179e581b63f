// argus_overlap.cu — argus_overlap: per-SM overlap time of producer/consumer region pairs.
//
// Segment = (pair k, SM m, role) with role 0 = producer, 1 = consumer.
//   k_ov_select  : one pass over the intervals: selected spans appended to an unordered list with their segment
//                  (argus_synthesize gets the same list from the aggregation pass or the pairing kernel instead)
//   k_ov_list_count_or_scatter : spans counted per segment, then copied into their segment (order irrelevant)
//   k_ov_scan    : segment bases; capacity check
//   k_ov_sort    : one CTA per segment: sort by (start, end) — by buckets of start time with one warp per bucket,
//                  or by a bitonic network on shared-memory tiles when the starts crowd; then turn the sorted spans into the
//                  disjoint pieces of their union, piece i = [max(start_i, E_{i-1}), E_i) with
//                  E_i = max end of spans 0..i, and the running length before each piece
//   k_ov_measure : one CTA per (k, m): |U_P|, |U_C|, and |U_P ∩ U_C| = sum over producer pieces of
//                  F_C(b) - F_C(a), F_C(t) = covered length of U_C before t (threads walk runs of producer pieces
//                  and find each boundary among the C pieces from the one before)
#include "argus_internal.cuh"

namespace {

constexpr int kOvThreads = 1024;
constexpr u32 kMaxPairs = ARGUS_MAX_PAIRS;

struct OvArgs {
  const argus_interval_t* intervals;
  const u64* interval_offsets;
  u64 max_intervals;  // records the interval array holds
  u32 num_streams, warps_per_cta, num_sms, num_pairs;
  const u32* cta_sm;
  const u32* pairs;
  argus_overlap_t* out;
  argus_status_t* status;
  u64* seg_count;   // [nseg]     (zeroed)
  u64* seg_cursor;  // [nseg]     (zeroed)
  u64* seg_base;    // [nseg + 1]
  ulonglong2* spans;  // [capacity] (start, end) -> after k_ov_sort (piece begin, piece end)
  ulonglong2* scratch;  // room k_ov_sort may use (the span list, which is dead by then); null = none
  u64 scratch_capacity;
  u64* cum;           // [capacity] covered length before piece i within its segment
  u64 capacity;
  u32 nseg;
  // scope selection (argus_overlap_scoped): iteration window, warp mask, SM mask, region mask
  int scoped;
  u32 ctx_lo, ctx_hi;
  u64 warp_mask;
  const u32* sm_mask;
  const u32* region_mask;
};

__device__ __forceinline__ bool ov_mask_bit(const u32* mask, u32 i) { return !mask || ((mask[i >> 5] >> (i & 31)) & 1u); }

// One pass over the intervals: spans of intervals whose region appears in a pair are appended to an unordered
// list with their segment. A warp reserves `chunk` list slots at a time (one global atomic per chunk) and
// marks the slots it leaves unused, so the list needs no clearing.
struct OvSelectOut {
  ulonglong2* spans;
  u32* seg;
  u64* count;      // slots reserved so far (zeroed before the kernel)
  u64 capacity;
  u32 chunk;       // power of two, at most 256
};

__device__ __forceinline__ void ov_retire_chunk(const OvSelectOut& o, u64 base, u32 used, u32 lane) {
  for (u32 i = used + lane; i < o.chunk; i += 32)
    if (base + i < o.capacity) o.seg[base + i] = 0xffffffffu;
}

__global__ void __launch_bounds__(256) k_ov_select(OvArgs a, OvSelectOut o) {
  __shared__ u32 sh_pairs[2 * kMaxPairs];
  for (u32 i = threadIdx.x; i < 2 * a.num_pairs; i += blockDim.x) sh_pairs[i] = a.pairs[i];
  __syncthreads();
  const u32 lane = threadIdx.x & 31;
  u64 ovc_base = 0;          // warp-uniform: the chunk this warp is filling
  u32 ovc_used = o.chunk;    // chunk size = none held yet
  bool held = false;
  for (u32 s = blockIdx.x; s < a.num_streams; s += gridDim.x) {
    const u32 m = a.cta_sm[s / a.warps_per_cta];
    const u64 lo = a.interval_offsets[s], hi = a.interval_offsets[s + 1];
    if (m >= a.num_sms || hi < lo || hi > a.max_intervals) {  // offsets beyond the interval array are reported, not read
      if (threadIdx.x == 0) argus_set_error(a.status, m >= a.num_sms ? ARGUS_ERR_INVALID_ARG : ARGUS_ERR_BAD_OFFSETS, s, m);
      continue;
    }
    if (a.scoped) {  // warp-role and SM tests: one answer per stream
      const u32 w = s % a.warps_per_cta;
      if (a.warp_mask != ~0ull && (w >= 64 || !((a.warp_mask >> w) & 1ull))) continue;
      if (!ov_mask_bit(a.sm_mask, m)) continue;
    }
    // every lane of a warp runs the same number of rounds, so that spans can be appended a warp at a time
    for (u64 base = lo + (threadIdx.x & ~31u); base < hi; base += blockDim.x) {
      const u64 i = base + lane;
      bool cand = false;
      u32 region = 0;
      u64 t0 = 0, incl = 0;
      if (i < hi) {
        const uint4* p = reinterpret_cast<const uint4*>(a.intervals + i);
        const uint4 q0 = __ldg(p);
        incl = (u64)q0.z | ((u64)q0.w << 32);
        t0 = (u64)q0.x | ((u64)q0.y << 32);
        region = __ldg(reinterpret_cast<const u32*>(p + 1) + 2);
        cand = incl != 0;
        if (cand && a.scoped) {  // iteration-window and region tests: one answer per interval
          const u32 ctx = __ldg(reinterpret_cast<const u32*>(p + 1) + 3);
          cand = ctx >= a.ctx_lo && ctx <= a.ctx_hi && ov_mask_bit(a.region_mask, region);
        }
      }
      for (u32 k = 0; k < 2 * a.num_pairs; ++k) {
        const bool pick = cand && sh_pairs[k] == region;
        const u32 bal = __ballot_sync(0xffffffffu, pick);
        if (!bal) continue;
        u32 todo = __popc(bal), done = 0;
        while (todo) {  // a ballot may straddle chunks when the chunks are small
          if (ovc_used == o.chunk) {
            u64 nb64 = 0;
            if (lane == 0) nb64 = atomicAdd(reinterpret_cast<unsigned long long*>(o.count), (unsigned long long)o.chunk);
            ovc_base = __shfl_sync(0xffffffffu, nb64, 0);
            ovc_used = 0;
            held = true;
          }
          const u32 room = o.chunk - ovc_used, take = todo < room ? todo : room;
          if (pick) {
            const u32 rank = __popc(bal & ((1u << lane) - 1u));
            if (rank >= done && rank < done + take) {
              const u64 slot = ovc_base + ovc_used + (rank - done);
              if (slot < o.capacity) {
                o.spans[slot] = make_ulonglong2(t0, t0 + incl);
                o.seg[slot] = ((k >> 1) * a.num_sms + m) * 2 + (k & 1u);
              }
            }
          }
          ovc_used += take; done += take; todo -= take;
        }
      }
    }
  }
  if (held) ov_retire_chunk(o, ovc_base, ovc_used, lane);
}

// Same two roles for spans that the pairing kernel already selected: list entries carry their segment;
// entries of reserved but unused slots have segment 0xffffffff.
struct OvList {
  const ulonglong2* spans;
  const u32* seg;
  const u64* count;  // slots reserved (may exceed capacity)
  u64 capacity;
};

constexpr u32 kOvListSegs = 2048;   // segments a block can count in shared memory
constexpr u32 kOvListChunk = 8192;  // list entries a block handles per iteration

__global__ void __launch_bounds__(256) k_ov_list_count_or_scatter(OvArgs a, OvList l, int scatter) {
  __shared__ u32 sh_cnt[kOvListSegs];
  __shared__ u64 sh_base[kOvListSegs];
  if (scatter && a.status->code != 0) return;
  const u64 reserved = *l.count;
  if (reserved > l.capacity && blockIdx.x == 0 && threadIdx.x == 0) {
    argus_set_error(a.status, ARGUS_ERR_CAPACITY, 0, reserved);
    a.status->intervals_required = reserved;
  }
  const u64 n = reserved < l.capacity ? reserved : l.capacity;
  const bool local = a.nseg <= kOvListSegs;
  for (u64 c0 = (u64)blockIdx.x * kOvListChunk; c0 < n; c0 += (u64)gridDim.x * kOvListChunk) {
    const u64 c1 = c0 + kOvListChunk < n ? c0 + kOvListChunk : n;
    if (!local) {  // too many segments for shared counters: global atomics per entry
      for (u64 i = c0 + threadIdx.x; i < c1; i += blockDim.x) {
        const u32 seg = l.seg[i];
        if (seg >= a.nseg) continue;
        if (!scatter) atomicAdd(&a.seg_count[seg], 1ull);
        else {
          const u64 slot = a.seg_base[seg] + atomicAdd(&a.seg_cursor[seg], 1ull);
          if (slot < a.capacity) a.spans[slot] = l.spans[i];
        }
      }
      continue;
    }
    for (u32 g = threadIdx.x; g < a.nseg; g += blockDim.x) sh_cnt[g] = 0;
    __syncthreads();
    for (int pass = 0; pass < (scatter ? 2 : 1); ++pass) {
      for (u64 i = c0 + threadIdx.x; i < c1; i += blockDim.x) {
        const u32 seg = l.seg[i];
        if (seg >= a.nseg) continue;
        const u32 pos = atomicAdd(&sh_cnt[seg], 1u);
        if (pass == 1) {
          const u64 slot = sh_base[seg] + pos;
          if (slot < a.capacity) a.spans[slot] = l.spans[i];
        }
      }
      __syncthreads();
      for (u32 g = threadIdx.x; g < a.nseg; g += blockDim.x) {
        if (pass == 0 && sh_cnt[g]) {
          if (!scatter) atomicAdd(&a.seg_count[g], (u64)sh_cnt[g]);
          else sh_base[g] = a.seg_base[g] + atomicAdd(&a.seg_cursor[g], (u64)sh_cnt[g]);
        }
        sh_cnt[g] = 0;
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(kOvThreads) k_ov_scan(OvArgs a) {
  __shared__ u64 sh[33];
  u64 carry = 0;
  for (u32 g0 = 0; g0 < a.nseg; g0 += kOvThreads) {
    const u32 g = g0 + threadIdx.x;
    const u64 c = g < a.nseg ? a.seg_count[g] : 0;
    u64 total;
    const u64 ex = argus_block_exclusive_scan<u64>(c, sh, &total);
    if (g < a.nseg) a.seg_base[g] = carry + ex;
    carry += total;
  }
  if (threadIdx.x == 0) {
    a.seg_base[a.nseg] = carry;
    if (carry > a.capacity) {
      argus_set_error(a.status, ARGUS_ERR_CAPACITY, 0, carry);
      a.status->intervals_required = carry;
    }
  }
}

__device__ __forceinline__ bool span_less(const ulonglong2& x, const ulonglong2& y) {
  return x.x < y.x || (x.x == y.x && x.y < y.y);
}

__device__ __forceinline__ void cmp_swap(ulonglong2* d, u64 i, u64 l) {
  const ulonglong2 x = d[i], y = d[l];
  if (span_less(y, x)) { d[i] = y; d[l] = x; }
}

constexpr u32 kOvSortTile = 4096;  // spans of a segment sorted in shared memory at a time (64 KB)

// Stages of the network whose partners lie inside one tile, on the tile in shared memory: the flip of block size k
// (if `flip`) and then the distances j_top, j_top / 2, ..., 1. `tbase` is the tile's first index in the segment.
// (every thread takes whole comparators: comparator c of a stage with distance bit h joins i = c with a zero
// inserted at bit h, and its partner)
__device__ __forceinline__ void ov_sort_tile_stages(ulonglong2* t, u64 tbase, u64 n, u32 k, bool flip, u32 j_top) {
  if (flip) {
    const u32 h = k >> 1;
    for (u32 c = threadIdx.x; c < kOvSortTile / 2; c += blockDim.x) {
      const u32 i = ((c & ~(h - 1)) << 1) | (c & (h - 1)), l = i ^ (k - 1);
      if (tbase + l < n) cmp_swap(t, i, l);
    }
    __syncthreads();
  }
  for (u32 j = j_top; j > 0; j >>= 1) {
    for (u32 c = threadIdx.x; c < kOvSortTile / 2; c += blockDim.x) {
      const u32 i = ((c & ~(j - 1)) << 1) | (c & (j - 1)), l = i | j;
      if (tbase + l < n) cmp_swap(t, i, l);
    }
    __syncthreads();
  }
}

// Sort of a large segment in expected linear time: spans are spread over buckets of equal width in start time (about 32
// a bucket for starts spread evenly), copied to `scratch` bucket by bucket, and every bucket is sorted by one warp with a
// small bitonic network in shared memory and written back in place. Returns false, with `d` untouched, when some bucket
// would hold more than kOvBucketMax spans (starts crowded in time): the caller then runs the full network.
// Shared memory (kOvSortSmem bytes at `raw`): bucket offsets, bucket cursors, one slice of kOvBucketMax spans per warp.
constexpr u32 kOvBucketMax = 128;
constexpr u32 kOvBuckets = 4096;
constexpr size_t kOvSortSmem = 2 * (kOvBuckets + 1) * 4 + 32 + (size_t)(kOvThreads / 32) * kOvBucketMax * sizeof(ulonglong2);

__device__ bool ov_bucket_sort(ulonglong2* d, ulonglong2* scratch, u64 n, unsigned char* raw) {
  u32* const off = reinterpret_cast<u32*>(raw);                 // [kOvBuckets + 1]
  u32* const cur = off + kOvBuckets + 1;                        // [kOvBuckets + 1]
  ulonglong2* const slices = reinterpret_cast<ulonglong2*>(raw + ((2 * (kOvBuckets + 1) * 4 + 15) & ~(size_t)15));
  __shared__ u64 red[2][32];
  __shared__ u32 sh_scan[33];
  __shared__ u32 crowded;
  const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (n >> 31) return false;
  // range of the start times
  u64 mn = ~0ull, mx = 0;
  for (u64 i = threadIdx.x; i < n; i += blockDim.x) {
    const u64 s = d[i].x;
    mn = s < mn ? s : mn;
    mx = s > mx ? s : mx;
  }
#pragma unroll
  for (int dd = 16; dd > 0; dd >>= 1) {
    const u64 a = __shfl_xor_sync(0xffffffffu, mn, dd), b = __shfl_xor_sync(0xffffffffu, mx, dd);
    mn = a < mn ? a : mn;
    mx = b > mx ? b : mx;
  }
  if (lane == 0) { red[0][warp] = mn; red[1][warp] = mx; }
  if (threadIdx.x == 0) crowded = 0;
  __syncthreads();
  mn = red[0][0]; mx = red[1][0];
  for (u32 w = 1; w < blockDim.x / 32; ++w) {
    mn = red[0][w] < mn ? red[0][w] : mn;
    mx = red[1][w] > mx ? red[1][w] : mx;
  }
  // buckets: a power of two of them, about 32 spans each; equal width, a power of two of ticks
  u32 nb = 1;
  while (nb < kOvBuckets && (u64)nb * 32 < n) nb <<= 1;
  u32 shift = 0;
  while (((mx - mn) >> shift) >= nb) ++shift;
  for (u32 b = threadIdx.x; b <= nb; b += blockDim.x) { off[b] = 0; cur[b] = 0; }
  __syncthreads();
  for (u64 i = threadIdx.x; i < n; i += blockDim.x) atomicAdd(&off[(u32)((d[i].x - mn) >> shift)], 1u);
  __syncthreads();
  for (u32 b = threadIdx.x; b < nb; b += blockDim.x)
    if (off[b] > kOvBucketMax) crowded = 1;
  __syncthreads();
  if (crowded) return false;  // uniform: every thread read the same word after the barrier
  // exclusive prefix of the counts (nb <= 4 x 1024)
  u32 carry = 0;
  for (u32 b0 = 0; b0 < nb; b0 += blockDim.x) {
    const u32 b = b0 + threadIdx.x;
    const u32 c = b < nb ? off[b] : 0u;
    u32 total;
    const u32 ex = argus_block_exclusive_scan<u32>(c, sh_scan, &total);
    if (b < nb) off[b] = carry + ex;
    carry += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) off[nb] = (u32)n;
  __syncthreads();
  for (u64 i = threadIdx.x; i < n; i += blockDim.x) {
    const ulonglong2 sp = d[i];
    const u32 b = (u32)((sp.x - mn) >> shift);
    scratch[off[b] + atomicAdd(&cur[b], 1u)] = sp;
  }
  __syncthreads();
  // one warp per bucket: small network in the warp's slice, then back in place (buckets are in time order)
  ulonglong2* const sl = slices + (size_t)warp * kOvBucketMax;
  for (u32 b = warp; b < nb; b += blockDim.x / 32) {
    const u32 lo = off[b], c = off[b + 1] - lo;
    if (c == 0) continue;
    u32 m = 1;
    while (m < c) m <<= 1;
    for (u32 t = lane; t < m; t += 32) sl[t] = t < c ? scratch[lo + t] : make_ulonglong2(~0ull, ~0ull);
    __syncwarp();
    for (u32 k = 2; k <= m; k <<= 1) {
      const u32 h = k >> 1;
      for (u32 q = lane; q < m / 2; q += 32) {
        const u32 i = ((q & ~(h - 1)) << 1) | (q & (h - 1));
        cmp_swap(sl, i, i ^ (k - 1));
      }
      __syncwarp();
      for (u32 j = k >> 2; j > 0; j >>= 1) {
        for (u32 q = lane; q < m / 2; q += 32) {
          const u32 i = ((q & ~(j - 1)) << 1) | (q & (j - 1));
          cmp_swap(sl, i, i | j);
        }
        __syncwarp();
      }
    }
    for (u32 t = lane; t < c; t += 32) d[lo + t] = sl[t];
    __syncwarp();
  }
  __syncthreads();
  return true;
}

__global__ void __launch_bounds__(kOvThreads) k_ov_sort(OvArgs a) {
  extern __shared__ __align__(16) unsigned char sort_raw[];
  ulonglong2* const tile = reinterpret_cast<ulonglong2*>(sort_raw);
  __shared__ u64 sh[33];
  __shared__ u64 sh_carry_e, sh_carry_len;
  if (a.status->code != 0) return;
  const u32 seg = blockIdx.x;
  const u64 base = a.seg_base[seg];
  const u64 n = a.seg_base[seg + 1] - base;
  if (n == 0) return;
  ulonglong2* d = a.spans + base;
  if (a.scratch && base + n <= a.scratch_capacity && n > kOvBucketMax && ov_bucket_sort(d, a.scratch + base, n, sort_raw)) {
    // sorted by buckets of start time
  } else {
  u64 p = 1;
  while (p < n) p <<= 1;
  // Bitonic network whose comparators all sort ascending; slots >= n act as +infinity and never move. A stage is a
  // barrier apart from the next, and a segment larger than the L1 pays an L2 round trip per stage in global memory:
  // so every run of stages whose partners lie within kOvSortTile spans is done on tiles in shared memory (one load
  // and one store of the segment per run), and only the stages that reach across tiles work on global memory.
  const u64 ntiles = (n + kOvSortTile - 1) / kOvSortTile;
  for (u64 tI = 0; tI < ntiles; ++tI) {  // all block sizes up to a tile
    const u64 tbase = tI * kOvSortTile;
    const u32 cnt = (u32)(n - tbase < kOvSortTile ? n - tbase : kOvSortTile);
    for (u32 i = threadIdx.x; i < cnt; i += blockDim.x) tile[i] = d[tbase + i];
    __syncthreads();
    for (u32 k = 2; k <= kOvSortTile && k <= p; k <<= 1) ov_sort_tile_stages(tile, tbase, n, k, true, k >> 2);
    for (u32 i = threadIdx.x; i < cnt; i += blockDim.x) d[tbase + i] = tile[i];
    __syncthreads();
  }
  for (u64 k = 2ull * kOvSortTile; k <= p; k <<= 1) {
    const u64 h = k >> 1;
    for (u64 c = threadIdx.x; c < p / 2; c += blockDim.x) {  // the flip and the long distances: across tiles
      const u64 i = ((c & ~(h - 1)) << 1) | (c & (h - 1)), l = i ^ (k - 1);
      if (l < n) cmp_swap(d, i, l);
    }
    __syncthreads();
    u64 j = k >> 2;
    for (; j >= kOvSortTile; j >>= 1) {
      for (u64 c = threadIdx.x; c < p / 2; c += blockDim.x) {
        const u64 i = ((c & ~(j - 1)) << 1) | (c & (j - 1)), l = i | j;
        if (l < n) cmp_swap(d, i, l);
      }
      __syncthreads();
    }
    for (u64 tI = 0; tI < ntiles; ++tI) {  // the distances below a tile
      const u64 tbase = tI * kOvSortTile;
      const u32 cnt = (u32)(n - tbase < kOvSortTile ? n - tbase : kOvSortTile);
      for (u32 i = threadIdx.x; i < cnt; i += blockDim.x) tile[i] = d[tbase + i];
      __syncthreads();
      ov_sort_tile_stages(tile, tbase, n, 0, false, (u32)j);
      for (u32 i = threadIdx.x; i < cnt; i += blockDim.x) d[tbase + i] = tile[i];
      __syncthreads();
    }
  }
  }
  // pieces of the union and running covered length
  if (threadIdx.x == 0) { sh_carry_e = 0; sh_carry_len = 0; }
  __syncthreads();
  const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (u64 i0 = 0; i0 < n; i0 += blockDim.x) {
    const u64 i = i0 + threadIdx.x;
    const bool live = i < n;
    const ulonglong2 sp = live ? d[i] : make_ulonglong2(0, 0);
    // inclusive prefix max of span ends (0 is the identity: ends are > starts >= 0)
    u64 e = live ? sp.y : 0;
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
      const u64 o = __shfl_up_sync(0xffffffffu, e, dd);
      if (lane >= (u32)dd && o > e) e = o;
    }
    if (lane == 31) sh[warp] = e;
    __syncthreads();
    if (warp == 0) {
      u64 w = sh[lane];
#pragma unroll
      for (int dd = 1; dd < 32; dd <<= 1) {
        const u64 o = __shfl_up_sync(0xffffffffu, w, dd);
        if (lane >= (u32)dd && o > w) w = o;
      }
      sh[lane] = w;
    }
    __syncthreads();
    const u64 carry_e = sh_carry_e;
    u64 before = carry_e;  // max end of all earlier spans
    if (warp > 0 && sh[warp - 1] > before) before = sh[warp - 1];
    {
      const u64 own_excl = __shfl_up_sync(0xffffffffu, e, 1);
      if (lane > 0 && own_excl > before) before = own_excl;
    }
    u64 e_incl = e > before ? e : before;
    const u64 pa = sp.x > before ? sp.x : before;
    const u64 pb = e_incl > pa ? e_incl : pa;
    const u64 len = live ? pb - pa : 0;
    __syncthreads();
    u64 total;
    const u64 ex = argus_block_exclusive_scan<u64>(len, sh, &total);
    const u64 carry_len = sh_carry_len;
    if (live) {
      d[i] = make_ulonglong2(pa, pb);
      a.cum[base + i] = carry_len + ex;
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) {
      sh_carry_e = e_incl > carry_e ? e_incl : carry_e;
      sh_carry_len = carry_len + total;
    }
    __syncthreads();
  }
}

constexpr int kOvMeasureThreads = 1024;

// covered length of the consumer pieces before time t, given pos = number of pieces whose begin is < t
__device__ __forceinline__ u64 covered_at(const ulonglong2* pc, const u64* cum, u64 pos, u64 t) {
  if (pos == 0) return 0;
  const ulonglong2 last = pc[pos - 1];
  return cum[pos - 1] + ((t < last.y ? t : last.y) - last.x);
}

// pos = number of consumer pieces whose begin is < t, reached from an earlier boundary's pos (never past it): steps
// of doubling length, then a binary search inside the last step, so a far boundary costs a logarithm of its distance
__device__ __forceinline__ u64 advance_to(const ulonglong2* pc, u64 nc, u64 pos, u64 t) {
  if (pos >= nc || !(pc[pos].x < t)) return pos;
  u64 lo = pos, step = 1;  // pc[lo].x < t
  while (lo + step < nc && pc[lo + step].x < t) { lo += step; step <<= 1; }
  u64 hi = lo + step < nc ? lo + step : nc;  // the first piece with begin >= t lies in (lo, hi]
  ++lo;
  while (lo < hi) {
    const u64 mid = lo + ((hi - lo) >> 1);
    if (pc[mid].x < t) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kOvMeasureThreads) k_ov_measure(OvArgs a) {
  __shared__ u64 sh[kOvMeasureThreads / 32];
  if (a.status->code != 0) return;
  const u32 km = blockIdx.x;  // k * M + m
  const u64 bp = a.seg_base[2 * km], bc = a.seg_base[2 * km + 1], be = a.seg_base[2 * km + 2];
  const u64 np = bc - bp, nc = be - bc;
  const ulonglong2* pp = a.spans + bp;
  const ulonglong2* pc = a.spans + bc;
  const u64* cum_c = a.cum + bc;
  u64 acc = 0;
  if (nc) {
    // Every thread takes a run of consecutive producer pieces. Pieces are disjoint and in time order, so the
    // boundaries a thread asks about never decrease: one binary search places the first, the rest are reached from
    // the one before (usually the next consumer piece or two).
    const u64 per = (np + blockDim.x - 1) / blockDim.x;
    const u64 i0 = (u64)threadIdx.x * per, i1 = i0 + per < np ? i0 + per : np;
    if (i0 < i1) {
      u64 pos;  // number of consumer pieces whose begin is < the boundary at hand
      {
        const u64 t = pp[i0].x;
        u64 lo = 0, hi = nc;
        while (lo < hi) {
          const u64 mid = lo + ((hi - lo) >> 1);
          if (pc[mid].x < t) lo = mid + 1; else hi = mid;
        }
        pos = lo;
      }
      for (u64 i = i0; i < i1; ++i) {
        const ulonglong2 piece = pp[i];
        pos = advance_to(pc, nc, pos, piece.x);
        const u64 before = covered_at(pc, cum_c, pos, piece.x);
        pos = advance_to(pc, nc, pos, piece.y);
        if (piece.y > piece.x) acc += covered_at(pc, cum_c, pos, piece.y) - before;
      }
    }
  }
#pragma unroll
  for (int dd = 16; dd > 0; dd >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, dd);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 both = 0;
    for (u32 w = 0; w < (blockDim.x >> 5); ++w) both += sh[w];
    const u64 p_ns = np ? a.cum[bp + np - 1] + (pp[np - 1].y - pp[np - 1].x) : 0;
    const u64 c_ns = nc ? a.cum[bc + nc - 1] + (pc[nc - 1].y - pc[nc - 1].x) : 0;
    argus_overlap_t o;
    o.overlap_ns = both; o.producer_ns = p_ns; o.consumer_ns = c_ns; o.either_ns = p_ns + c_ns - both;
    a.out[km] = o;
  }
}

struct OvLayout { size_t seg_count, seg_cursor, seg_base, spans, total_fixed; };

OvLayout ov_layout(uint32_t nseg) {
  OvLayout L;
  size_t o = 0;
  L.seg_count = o; o += argus_align_up((size_t)nseg * 8, 256);
  L.seg_cursor = o; o += argus_align_up((size_t)nseg * 8, 256);
  L.seg_base = o; o += argus_align_up(((size_t)nseg + 1) * 8, 256);
  L.spans = o;
  L.total_fixed = o;
  return L;
}

}  // namespace

constexpr size_t kBytesPerSortedSpan = 24;  // (begin, end) + covered length before it
constexpr size_t kBytesPerListedSpan = 20;  // (begin, end) + segment
constexpr unsigned kSelectGrid = 148 * 8;
constexpr unsigned kSelectWarps = kSelectGrid * 8;

extern "C" size_t argus_overlap_workspace_bytes(uint64_t max_intervals, uint32_t /*num_streams*/, uint32_t num_pairs,
                                                uint32_t num_sms) {
  const OvLayout L = ov_layout(num_pairs * num_sms * 2);
  // worst case: every interval selected in both roles of every pair, listed and then sorted; a third more
  // list slots than spans cover the slots that warps reserve and leave unused
  const size_t spans = (size_t)max_intervals * 2 * num_pairs;
  return L.total_fixed + argus_align_up((spans + spans / 3 + 64) * (kBytesPerSortedSpan + kBytesPerListedSpan) + 1024, 256);
}

// Shared tail of both entry paths: from the list of selected spans to the overlap measures.
static int ov_run(OvArgs& a, const OvList* list, cudaStream_t stream) {
  for (int pass = 0; pass < 2; ++pass) {
    k_ov_list_count_or_scatter<<<592, 256, 0, stream>>>(a, *list, pass);
    ARGUS_CHECK_LAUNCH();
    if (pass == 0) {
      k_ov_scan<<<1, kOvThreads, 0, stream>>>(a);
      ARGUS_CHECK_LAUNCH();
    }
  }
  argus_prof_mark(ARGUS_PROF_OVERLAP, stream, 0);
  {
    static bool opted_in[64];  // the shared-memory opt-in belongs to a device
    int dev = 0;
    ARGUS_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ARGUS_ERR_INVALID_ARG;
    if (!opted_in[dev]) {
      ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_ov_sort, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kOvSortSmem));
      opted_in[dev] = true;
    }
  }
  a.scratch = const_cast<ulonglong2*>(list->spans);  // every listed span has been copied into its segment
  a.scratch_capacity = list->capacity;
  k_ov_sort<<<a.nseg, kOvThreads, kOvSortSmem, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  argus_prof_mark(ARGUS_PROF_OVERLAP, stream, 1);
  k_ov_measure<<<a.nseg / 2, kOvMeasureThreads, 0, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

static int ov_setup(OvArgs& a, uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                    const uint32_t* pairs, uint32_t num_pairs, argus_overlap_t* out, argus_status_t* status, void* workspace,
                    size_t workspace_bytes, cudaStream_t stream, size_t own_list_bytes = 0) {
  const u32 nseg = num_pairs * num_sms * 2;
  const OvLayout L = ov_layout(nseg);
  if (workspace_bytes < L.total_fixed + 256 + own_list_bytes) return ARGUS_ERR_WORKSPACE;
  workspace_bytes -= own_list_bytes;  // the caller keeps its list behind the part laid out here
  char* ws = (char*)workspace;
  a.intervals = nullptr; a.interval_offsets = nullptr; a.max_intervals = 0; a.num_streams = num_streams;
  a.warps_per_cta = warps_per_cta; a.num_sms = num_sms; a.num_pairs = num_pairs; a.cta_sm = cta_sm; a.pairs = pairs;
  a.out = out; a.status = status;
  a.seg_count = (u64*)(ws + L.seg_count); a.seg_cursor = (u64*)(ws + L.seg_cursor); a.seg_base = (u64*)(ws + L.seg_base);
  a.capacity = (workspace_bytes - L.total_fixed) / 24;
  a.spans = (ulonglong2*)(ws + L.spans);
  a.scratch = nullptr; a.scratch_capacity = 0;
  a.cum = (u64*)(ws + L.spans + argus_align_up((size_t)a.capacity * 16, 16));
  a.nseg = nseg;
  a.scoped = 0; a.ctx_lo = 0; a.ctx_hi = 0xffffffffu; a.warp_mask = ~0ull; a.sm_mask = nullptr; a.region_mask = nullptr;
  ARGUS_CUDA_TRY(cudaMemsetAsync(ws, 0, L.seg_base, stream));
  ARGUS_CUDA_TRY(cudaMemsetAsync(out, 0, (size_t)num_pairs * num_sms * sizeof(argus_overlap_t), stream));
  return ARGUS_OK;
}

// Overlap from a span list appended by the pairing kernel (see argus_fuse.cuh).
int argus_internal_overlap_from_list(const void* list_spans, const uint32_t* list_seg, const uint64_t* list_count,
                                     uint64_t list_capacity, uint32_t num_sms, uint32_t num_pairs, argus_overlap_t* out,
                                     argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (num_pairs == 0) return ARGUS_OK;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  OvArgs a;
  const int rc = ov_setup(a, 0, 1, nullptr, num_sms, nullptr, num_pairs, out, status, workspace, workspace_bytes, stream);
  if (rc != ARGUS_OK) return rc;
  OvList l;
  l.spans = (const ulonglong2*)list_spans; l.seg = list_seg; l.count = (const u64*)list_count; l.capacity = list_capacity;
  return ov_run(a, &l, stream);
}

static int overlap_scoped(const argus_interval_t* intervals, uint64_t max_intervals, const uint64_t* interval_offsets,
                          uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                          const uint32_t* pairs, uint32_t num_pairs, const argus_scope_t* scope, argus_overlap_t* out,
                          argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream,
                          bool reset_status) {
  if (!interval_offsets || (!cta_sm && num_streams) || !status || !workspace) return ARGUS_ERR_INVALID_ARG;
  if (scope && scope->ctx_hi < scope->ctx_lo) return ARGUS_ERR_INVALID_ARG;
  if (warps_per_cta == 0 || num_streams % warps_per_cta != 0 || num_sms == 0) return ARGUS_ERR_INVALID_ARG;
  if (num_pairs > kMaxPairs || (num_pairs && (!pairs || !out))) return ARGUS_ERR_INVALID_ARG;
  if ((max_intervals && !intervals) || ((uintptr_t)intervals & 15) || ((uintptr_t)workspace & 255) || ((uintptr_t)out & 7))
    return ARGUS_ERR_INVALID_ARG;
  if ((uint64_t)num_pairs * num_sms * 2 > 0x7fffffffull) return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (reset_status) ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  if (num_pairs == 0) return ARGUS_OK;
  OvArgs a;
  // split what the workspace offers beyond the fixed part between the list (20 B a slot) and the sorted spans
  // (24 B each), with a third more list slots than sorted spans
  const OvLayout L0 = ov_layout(num_pairs * num_sms * 2);
  if (workspace_bytes < L0.total_fixed + 2048) return ARGUS_ERR_WORKSPACE;
  const u64 span_cap = (workspace_bytes - L0.total_fixed - 1536) * 3 / (3 * kBytesPerSortedSpan + 4 * kBytesPerListedSpan);
  const u64 list_cap = span_cap + span_cap / 3;
  const size_t list_bytes = argus_align_up(256 + argus_align_up((size_t)list_cap * 4, 256) + (size_t)list_cap * 16, 256);
  const int rc = ov_setup(a, num_streams, warps_per_cta, cta_sm, num_sms, pairs, num_pairs, out, status, workspace,
                          workspace_bytes, stream, list_bytes);
  if (rc != ARGUS_OK) return rc;
  a.intervals = intervals; a.interval_offsets = (const u64*)interval_offsets; a.max_intervals = max_intervals;
  if (scope) {
    a.scoped = 1; a.ctx_lo = scope->ctx_lo; a.ctx_hi = scope->ctx_hi; a.warp_mask = scope->warp_mask;
    a.sm_mask = scope->sm_mask; a.region_mask = scope->region_mask;
  }
  // the list of selected spans sits at the end of the workspace: counter, segments, spans
  char* lbase = (char*)workspace + (workspace_bytes - list_bytes);
  OvSelectOut o;
  o.count = (u64*)lbase;
  o.seg = (u32*)(lbase + 256);
  o.spans = (ulonglong2*)(lbase + 256 + argus_align_up((size_t)list_cap * 4, 256));
  o.capacity = list_cap;
  o.chunk = 256;  // slots left unused are bounded by a quarter of the list: smaller chunks for small lists
  while (o.chunk > 1 && (u64)kSelectWarps * o.chunk * 4 > list_cap) o.chunk >>= 1;
  ARGUS_CUDA_TRY(cudaMemsetAsync(o.count, 0, 256, stream));
  if (num_streams) {
    k_ov_select<<<num_streams < kSelectGrid ? num_streams : kSelectGrid, 256, 0, stream>>>(a, o);
    ARGUS_CHECK_LAUNCH();
  }
  OvList l;
  l.spans = o.spans; l.seg = o.seg; l.count = o.count; l.capacity = list_cap;
  return ov_run(a, &l, stream);
}

int argus_internal_overlap(const argus_interval_t* intervals, uint64_t max_intervals, const uint64_t* interval_offsets,
                           uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                           const uint32_t* pairs, uint32_t num_pairs, argus_overlap_t* out, argus_status_t* status,
                           void* workspace, size_t workspace_bytes, void* cuda_stream, bool reset_status) {
  return overlap_scoped(intervals, max_intervals, interval_offsets, num_streams, warps_per_cta, cta_sm, num_sms, pairs,
                        num_pairs, nullptr, out, status, workspace, workspace_bytes, cuda_stream, reset_status);
}

extern "C" int argus_overlap_scoped(const argus_interval_t* intervals, uint64_t max_intervals,
                                    const uint64_t* interval_offsets, uint32_t num_streams, uint32_t warps_per_cta,
                                    const uint32_t* cta_sm, uint32_t num_sms, const uint32_t* pairs, uint32_t num_pairs,
                                    const argus_scope_t* scope, argus_overlap_t* out, argus_status_t* status,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return overlap_scoped(intervals, max_intervals, interval_offsets, num_streams, warps_per_cta, cta_sm, num_sms, pairs,
                        num_pairs, scope, out, status, workspace, workspace_bytes, cuda_stream, true);
}

extern "C" int argus_overlap(const argus_interval_t* intervals, uint64_t max_intervals, const uint64_t* interval_offsets,
                             uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                             const uint32_t* pairs, uint32_t num_pairs, argus_overlap_t* out, argus_status_t* status,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return argus_internal_overlap(intervals, max_intervals, interval_offsets, num_streams, warps_per_cta, cta_sm, num_sms,
                                pairs, num_pairs, out, status, workspace, workspace_bytes, cuda_stream, true);
}
