// argus_pair_tiled.cu — tiled pairing kernel for sm_100a.
//
// One CTA walks one stream tile by tile (T = NT * E events per tile); tiles arrive in shared
// memory by TMA bulk copies (double buffered, mbarrier completion) and interval records leave with
// coalesced 16-byte stores, one thread per record. The per-stream region stack is carried from tile
// to tile in shared memory, so CTAs never wait on one another.
//
// Inside a tile the stack height before each event comes from a block-wide prefix sum of +1/-1, so
// every marker knows its level (stack position) without walking the stack:
//   - every begin sets its bit in a per-level bitmap over the tile's event positions;
//   - every end (one thread per end marker) finds its begin as the latest set bit of its own level
//     before it, and its parent as the latest set bit one level down before that begin; when there
//     is none in the tile, the frame is in the stack carried from earlier tiles;
//   - every finished interval adds its inclusive time to its parent frame's accumulator (shared
//     atomics), which gives exclusive time without ordering the threads. The accumulators hold what
//     the current window adds, in 32 bits (a frame carried from earlier tiles brings its 64-bit child
//     time along separately); an interval or a sum that does not fit breaks the rules below.
// This is exact when the tile is well nested (every end meets the frame on top with the same region
// id). A tile is consumed in windows: the first position where a rule fails (region mismatch, negative
// height, bad region id, depth overflow, level window exceeded, 2^32 ticks of child time in one
// window) cuts the window there; the prefix is
// redone on its own (nothing of it had been committed), the offending marker goes through the
// sequential stack machine on the carried stack, and a new window starts after it, so the result is
// always the sequential definition's.
#include "argus_internal.cuh"
#include "argus_pair_common.cuh"

#include <atomic>
#include <mutex>
#include <type_traits>

namespace {

__device__ __forceinline__ u32 smem_u32(const void* p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(u64* bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(u64* bar, u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_1d(void* dst, const void* src, u32 bytes, u64* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, u32 parity) {
  u32 ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after ~2^22 polls (seconds); the caller then reports ARGUS_ERR_TIMEOUT.
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity) {
  for (u32 it = 0; it < (1u << 22); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}

constexpr int kLevelWindow = 16;  // begins of a tile may sit at levels [lbase, lbase + 16)
constexpr int kCar = 80;          // slots of a carried-frame block: 64 frames, 1 sink for "no parent", padding
constexpr int kSink = 64;         // index of the sink slot inside a carried-frame block
constexpr int kBadRef = 0x3fff;   // reference that marks a window as not well nested
constexpr int kSeqChunk = 128;    // markers handed to the sequential machine at once when cuts come densely
constexpr u32 kNoRec = 0xffffffffu;

// Takes the next piece of work of pass `p`: a stream nobody has started (position below num_streams) or a
// hand-over from the queue. Returns false when every stream is done (or on a timeout). One thread per CTA.
__device__ __forceinline__ bool tile_pop_work(const ArgusPairArgs& a, int p, u64* stream, u32* rec) {
  const u64 h = atomicAdd(reinterpret_cast<unsigned long long*>(&a.ctl->q_head[p]), 1ull);
  if (h < a.num_streams) { *stream = a.order ? a.order[h] : h; *rec = kNoRec; return true; }
  const u64 slot = h - a.num_streams;
  if (!a.queue || slot >= a.queue_capacity) return false;  // more positions than hand-overs can ever be published
  volatile u32* q = a.queue + slot;
  volatile u32* done = &a.ctl->n_done[p];
  volatile u64* tail = &a.ctl->q_tail[p];
  u64 seen = *tail;
  u32 idle = 0, nap = 64;
  for (;;) {
    const u32 v = *q;
    if (v) {
      *q = 0;  // the second pass uses the same entries
      __threadfence();
      *rec = v - 1;
      *stream = *reinterpret_cast<volatile u32*>(&a.records[v - 1].stream);
      return true;
    }
    if (*done >= a.num_streams) return false;
    const u64 t = *tail;
    if (t != seen) { seen = t; idle = 0; }
    if (++idle > a.poll_limit) {  // ~1 s without any hand-over anywhere
      argus_set_error(a.status, ARGUS_ERR_TIMEOUT, 0, slot);
      return false;
    }
    __nanosleep(nap);
    if (nap < 2048) nap *= 2;
  }
}

// Shared memory of one CTA. Events of the two tile buffers and the frames carried from earlier tiles
// share one index space, so that "the frame an end closes" and "its parent" are plain indices:
//   ev0[0..T) | car0[0..80) | car1[0..80) | ev1[0..T)
// Seen from buffer 0, carried block c holds level L at T + 80 c + L; seen from buffer 1 at 80 c + L - 160.
// A window reads the current block and writes the stack it leaves behind into the other one.
template <int NT, int E>
struct TileSmem {
  static constexpr int T = NT * E;
  static constexpr int NW = NT / 32;
  static constexpr int NWORDS = T / 32;                 // bitmap words per level
  static constexpr int MAXI = T / 2 + ARGUS_MAX_DEPTH;  // intervals a well-nested tile can emit
  static constexpr int NI = (MAXI + NT - 1) / NT;       // intervals per thread in the emission phases
  static constexpr int kDescShift = T <= 1024 ? 10 : 16;
  using desc_t = typename std::conditional<(T <= 1024), unsigned short, u32>::type;
  uint4 evall[2 * T + 2 * kCar];
  u32 accall[T + 4 * kCar];        // child time each frame gathers in the current window (32 bits: an overflow cuts the
                                   // window), same index space shifted by 2 kCar
  desc_t desc[MAXI];               // per end, in end order: event index | level << kDescShift
  union {
    u32 bm[kLevelWindow][NWORDS];    // per level: bit e set = event e of the tile is a begin at that level
    ArgusFrame fstk[ARGUS_MAX_DEPTH];  // stack in the layout the sequential path uses (no bitmap is live while it runs)
  };
  u64 summ[kLevelWindow];          // per level: bit w set = bm[level][w] != 0
  u32 cidx[2][ARGUS_MAX_DEPTH];    // begin index (within the stream) of each carried frame
  u64 cchild[2][ARGUS_MAX_DEPTH];  // child time of each carried frame as the window found it
  u32 warp_tot[32];
  u64 bar[2];
  u64 cur_stream;
  u32 cur_rec;                     // hand-over record of the stream being walked (kNoRec: none)
  u64 n_int;                       // written by the sequential redo path
  int ch;
  int badpos[2];                   // first position of the window where the parallel rules fail (INT_MAX = none); windows alternate
                                   // between the two, so that one can be reset while stragglers still read the other
  int dead, failed;
};

// Latest begin of the tile at level L and position < pos (pos <= T); -1 if there is none. Written without
// branches: the lanes of a warp would otherwise split over "same word", "earlier word" and "not in this tile"
// and run all three paths one after the other.
template <int NT, int E>
__device__ __forceinline__ int tile_latest_begin(const TileSmem<NT, E>& sm, int L, int lbase, int pos) {
  constexpr int NWORDS = TileSmem<NT, E>::NWORDS;
  const int l = L - lbase;
  const bool valid = (unsigned)l < (unsigned)kLevelWindow;
  const int lc = valid ? l : 0;
  const int w = pos >> 5;
  const bool in_tile = w < NWORDS;               // pos == T: every word lies before it
  const int wc = in_tile ? w : NWORDS - 1;
  const u32 below = in_tile ? ((1u << (pos & 31)) - 1u) : 0u;
  const u32 m = sm.bm[lc][wc] & below;           // begins of the level in the same word, before pos
  int w2;                                        // last earlier word with a begin of the level
  bool earlier;
  if (NWORDS <= 32) {                            // one 32-bit word of the summary covers the tile
    const u32 s = reinterpret_cast<const u32*>(&sm.summ[lc])[0] & ((w >= 32) ? ~0u : ((1u << w) - 1u));
    earlier = s != 0;
    w2 = earlier ? 31 - __clz(s) : 0;
  } else {
    const u64 s = sm.summ[lc] & ((w >= 64) ? ~0ull : ((1ull << w) - 1ull));
    earlier = s != 0;
    w2 = earlier ? 63 - __clzll((long long)s) : 0;
  }
  const u32 m2 = sm.bm[lc][w2];
  const int same = wc * 32 + 31 - __clz(m);
  const int prev = w2 * 32 + 31 - __clz(m2);
  const int r = m ? same : ((earlier && m2) ? prev : -1);
  return valid ? r : -1;
}


// One tile of a stream into shared memory: a bulk copy, or two when the stream lives in a ring slot and the
// tile straddles the slot's end. `src` is the stream's first record (packed input) or its slot (ring).
template <bool RING>
__device__ __forceinline__ void tile_fetch(const ArgusPairArgs& a, uint4* dst, const argus_event_t* src, u32 ring_first,
                                           u32 start, u32 count, u64* bar) {
  mbar_expect_tx(bar, count * 16u);
  if (!RING) {
    tma_load_1d(dst, src + start, count * 16u, bar);
  } else {
    u32 p = ring_first + start;  // both below the capacity
    if (p >= a.ring_capacity) p -= a.ring_capacity;
    const u32 room = a.ring_capacity - p;
    const u32 head = count < room ? count : room;
    tma_load_1d(dst, src + p, head * 16u, bar);
    if (count > head) tma_load_1d(dst + head, src, (count - head) * 16u, bar);
  }
}

template <int NT, int E, int MINB, bool RING = false>
__global__ void __launch_bounds__(NT, MINB) k_pair_tiled(ArgusPairArgs a) {
  using SM = TileSmem<NT, E>;
  constexpr int T = SM::T, NW = SM::NW, NWORDS = SM::NWORDS, MAXI = SM::MAXI, NI = SM::NI;
  static_assert(NW <= 32 && NT % 32 == 0 && NT >= ARGUS_MAX_DEPTH && NWORDS <= 64 && T + kCar < kBadRef, "block shape");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  SM& sm = *reinterpret_cast<SM*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (a.redo && !a.ctl->redo) return;
  if (tid == 0) {
    mbar_init(&sm.bar[0], 1);
    mbar_init(&sm.bar[1], 1);
    fence_mbar_init();
    sm.dead = 0;
    sm.badpos[0] = sm.badpos[1] = 0x7fffffff;
  }
  __syncthreads();
  u32 ph0 = 0, ph1 = 0;  // mbarrier phase parities
  int bp = 0;            // which of sm.badpos the next window uses
  const u64 off0 = a.stream_offsets[0];
  u32 tot_ctx = 0, tot_rev = 0, tot_clamp = 0;

  for (;;) {
    if (tid == 0) {
      u64 st = ~0ull;
      u32 rc = kNoRec;
      if (!tile_pop_work(a, a.redo ? 1 : 0, &st, &rc)) st = ~0ull;
      sm.cur_stream = st;
      sm.cur_rec = rc;
    }
    __syncthreads();
    const u64 s64 = sm.cur_stream;
    if (s64 >= a.num_streams) break;
    const u32 s = (u32)s64;
    u32 rec = sm.cur_rec;
    const u64 lo = a.stream_offsets[s], hi = a.stream_offsets[s + 1];
    if (hi < lo || hi > a.num_events || lo < off0 || ((hi - lo) >> 32)) {
      if (tid == 0) {
        argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
        if (!a.redo) a.counts[s] = 0;
        atomicAdd(&a.ctl->n_done[a.redo ? 1 : 0], 1u);
      }
      __syncthreads();
      continue;
    }
    const u32 n = (u32)(hi - lo);
    const u64 gpos0 = lo - off0;
    const u64 out_base = a.redo ? a.interval_offsets[s] : (gpos0 >> 1);
    if (a.redo && rec == kNoRec && out_base == (gpos0 >> 1) && out_base + a.counts[s] <= a.interval_capacity) {
      // second pass: this stream's intervals (and digests) already lie where they belong — the first pass wrote them
      // at the same positions, all of them fitted, and no other stream writes there in either pass
      if (tid == 0) atomicAdd(&a.ctl->n_done[1], 1u);
      __syncthreads();
      continue;
    }
    const argus_event_t* src = RING ? a.events + (u64)s * a.ring_capacity : a.events + lo;
    const u32 ring_first = RING ? argus_ring_first(a, s) : 0u;
    const u32 ntiles = (n + T - 1) / T;
    int ch = 0;          // carried stack height (uniform)
    u64 n_int = 0;       // intervals of this stream so far (uniform)
    bool stream_failed = false;
    // Long streams are walked a chunk at a time. A resumed stream takes its state from the record; a new one
    // reserves a record.
    u32 ti0 = 0;
    constexpr u32 kChunkTiles = (kChunkEvents + T - 1) / T;
    bool chunked = a.queue != nullptr && ntiles > kChunkTiles;
    if (rec != kNoRec) {
      const ArgusStreamRecord* r = a.records + rec;
      ti0 = __ldcg(&r->next_tile);
      ch = __ldcg(&r->ch);
      n_int = __ldcg(&r->n_int);
      if (tid < ch) {  // the carried block 0 is where the first window looks
        sm.evall[T + tid] = __ldcg(&r->frames[tid]);
        sm.cchild[0][tid] = __ldcg(&r->child[tid]);
        sm.cidx[0][tid] = __ldcg(&r->idx[tid]);
      }
    } else if (chunked) {
      __syncthreads();  // everyone has read sm.cur_rec
      if (tid == 0) {
        const u32 r = atomicAdd(&a.ctl->n_records[a.redo ? 1 : 0], 1u);
        sm.cur_rec = r < a.record_capacity ? r : kNoRec;
      }
      __syncthreads();
      rec = sm.cur_rec;
      if (rec == kNoRec) chunked = false;  // cannot happen (one record per long stream); then the stream is walked whole
    }
    const u32 ti_end = chunked && ti0 + kChunkTiles < ntiles ? ti0 + kChunkTiles : ntiles;
    if (tid == 0 && ti0 < ti_end) {  // first tile of this chunk, into the buffer its index selects
      const u32 start = ti0 * (u32)T;
      tile_fetch<RING>(a, (ti0 & 1) ? sm.evall + T + 2 * kCar : sm.evall, src, ring_first, start,
                       (n - start) < (u32)T ? (n - start) : (u32)T, &sm.bar[ti0 & 1]);
    }

    int cpar = 0;        // which carried-frame block holds the current stack
    for (u32 ti = ti0; ti < ti_end; ++ti) {
      const int b = ti & 1;
      const u32 tile_start = ti * (u32)T;
      const int tn = (int)((n - tile_start) < (u32)T ? (n - tile_start) : (u32)T);
      uint4* const ev0 = sm.evall;
      uint4* const ev1 = sm.evall + T + 2 * kCar;
      const uint4* evb = b ? ev1 : ev0;                  // evb[ref] for every reference of this tile
      u32* accb = sm.accall + 2 * kCar;                  // accb[ref], ref in [-2 kCar, T + 2 kCar)
      const int carlo = b ? -2 * kCar : T;               // reference of slot 0 of carried block 0, seen from this buffer
      if (tid == 0 && ti + 1 < ti_end) {  // prefetch the next tile into the other buffer
        const u32 nstart = tile_start + T;
        tile_fetch<RING>(a, b ? ev0 : ev1, src, ring_first, nstart, (n - nstart) < (u32)T ? (n - nstart) : (u32)T, &sm.bar[b ^ 1]);
      }
      {
        const bool ok = mbar_wait_bounded(&sm.bar[b], b ? ph1 : ph0);
        if (b) ph1 ^= 1; else ph0 ^= 1;
        if (!ok) sm.dead = 1;
      }

      // The tile is consumed in windows [w0, wend). A well-nested tile is one window. When the parallel
      // rules fail first at position p, the window is cut there: [w0, p) is redone in parallel (it is well
      // nested), the marker at p goes through the sequential stack machine, and a new window starts after it.
      int w0 = 0, wend = tn, small_streak = 0;
      while (w0 < tn) {
        const int cbase = carlo + cpar * kCar;           // carried level L -> reference cbase + L
        uint4* const car_next = sm.evall + T + (cpar ^ 1) * kCar;

        // ---------------- phase A: heights by prefix sum; begins into per-level bitmaps; ends into `desc` ----------
        u32 tags[E];
        int nb = 0, ne = 0;
#pragma unroll
        for (int k = 0; k < E; ++k) {
          const int e = w0 + tid * E + k;
          const bool valid = e < wend;
          tags[k] = valid ? reinterpret_cast<const u32*>(evb + e)[2] : 0xffffffffu;
          if (!(tags[k] & 1u)) accb[e] = 0;  // child time is gathered at begins only
          if (valid) { if (tags[k] & 1u) ++ne; else ++nb; }
        }
        for (int i = tid; i < kLevelWindow * NWORDS; i += NT) (&sm.bm[0][0])[i] = 0;
        if (tid < kLevelWindow) sm.summ[tid] = 0;
        if (tid < ch) accb[cbase + tid] = 0;  // what this window adds to the carried frames (a cut window starts clean again)
        if (tid == 0) { sm.failed = 0; accb[cbase + kSink] = 0; }
        // block prefix sum of (begins, ends), 16 bits each: one barrier
        const u32 mine_cnt = (u32)nb | ((u32)ne << 16);
        u32 incl_cnt = mine_cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const u32 o = __shfl_up_sync(0xffffffffu, incl_cnt, d);
          if (lane >= d) incl_cnt += o;
        }
        if (lane == 31) sm.warp_tot[warp] = incl_cnt;
        __syncthreads();
        u32 before = 0, tot = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          const u32 t = sm.warp_tot[w];
          if (w < warp) before += t;
          tot += t;
        }
        const u32 ex = before + incl_cnt - mine_cnt;
        const int win_nb = (int)(tot & 0xffffu);
        const int win_ne = (int)(tot >> 16) < MAXI ? (int)(tot >> 16) : MAXI;  // more ends than that means a violation earlier
        const int h0 = ch + (int)(ex & 0xffffu) - (int)(ex >> 16);
        const int lbase = ch > kLevelWindow / 2 ? ch - kLevelWindow / 2 : 0;
        {
          int h = h0, rank = (int)(ex >> 16);
          bool seen = false;  // this thread already reported a violation: later markers only keep `desc` complete
#pragma unroll
          for (int k = 0; k < E; ++k) {  // flat, so that begins and ends of a warp are handled by predication, not by two passes
            const int e = w0 + tid * E + k;
            const bool valid = e < wend;  // (not "tag != all ones": that is a marker too, with a region id out of range)
            const bool is_e = valid && (tags[k] & 1u), is_b = valid && !(tags[k] & 1u);
            const int he = h - 1;            // level of the frame an end closes
            const int l = h - lbase;         // level of the frame a begin opens, inside the window
            // the parallel rules: known region id, height never negative, at most 64 frames, begins inside the level window
            const bool viol = (valid && (tags[k] >> 1) >= a.num_regions) || (is_e && he < 0) ||
                              (is_b && ((unsigned)l >= (unsigned)kLevelWindow || h >= ARGUS_MAX_DEPTH));
            if (is_e && rank < MAXI) sm.desc[rank] = (typename SM::desc_t)((u32)e | ((u32)(he & 0x3f) << SM::kDescShift));
            if (is_b && !viol && !seen) {
              atomicOr(&sm.bm[l][e >> 5], 1u << (e & 31));
              atomicOr(reinterpret_cast<u32*>(&sm.summ[l]) + (e >> 10), 1u << ((e >> 5) & 31));
            }
            rank += is_e ? 1 : 0;
            h += is_b ? 1 : (is_e ? -1 : 0);
            if (viol && !seen) { atomicMin(&sm.badpos[bp], e); seen = true; }
          }
        }
        __syncthreads();

        // ---------------- phase B: one thread per end marker: find begin and parent, feed the parent's child time ---
        u32 refs[NI];
        {
          const int first_bad = sm.badpos[bp];  // violations found so far; ends at or after it need no work
#pragma unroll
          for (int i = 0; i < NI; ++i) {
            // (the last, partly filled round goes to the upper half of the block: the lower half has the block's
            // other duties, and a barrier waits for the slowest warp)
            const int rk = (i == NI - 1 ? (tid + NT / 2) % NT : tid) + i * NT;
            refs[i] = 0;
            if (rk < win_ne) {
              const u32 d = sm.desc[rk];
              const int e = (int)(d & ((1u << SM::kDescShift) - 1u)), L = (int)(d >> SM::kDescShift);
              if (e >= first_bad) continue;
              const uint4 ee = evb[e];  // needed after the lookups; asked for now, so that it arrives meanwhile
              // in the tile, or opened before this window (then so was its parent); selects, not branches
              // (no begin of level L - 1 can lie between the partner and e while the partner's frame is open, so the
              // parent is also the latest begin of level L - 1 before e: the two lookups do not depend on each other)
              const int p_in = tile_latest_begin<NT, E>(sm, L, lbase, e);
              const bool p_car = p_in < 0;
              const int q_in = tile_latest_begin<NT, E>(sm, L - 1, lbase, e);
              const int partner = p_car ? (L < ch ? cbase + L : kBadRef) : p_in;
              const int parent = L == 0 ? cbase + kSink : (q_in >= 0 ? q_in : (L - 1 < ch ? cbase + L - 1 : kBadRef));
              if (partner == kBadRef || parent == kBadRef) { atomicMin(&sm.badpos[bp], e); continue; }
              const uint4 pe = evb[partner];
              if ((pe.z >> 1) != (ee.z >> 1)) { atomicMin(&sm.badpos[bp], e); continue; }
              const u64 ts = (u64)ee.x | ((u64)ee.y << 32), bts = (u64)pe.x | ((u64)pe.y << 32);
              if (ts > bts) {
                // the parent gathers what this window adds to its child time in 32 bits; an interval or a sum of 2^32 ticks
                // cuts the window here, and the sequential machine (64-bit throughout) takes this marker
                const u64 dlt = ts - bts;
                const u32 lo32 = (u32)dlt;
                const u32 old = atomicAdd(&accb[parent], lo32);
                if ((dlt >> 32) || old + lo32 < old) { atomicMin(&sm.badpos[bp], e); continue; }
              }
              refs[i] = ((u32)partner & 0xffffu) | ((u32)parent << 16);
            }
          }
        }
        __syncthreads();
        if (sm.dead) {  // a bulk copy never arrived: report and leave (uniform decision)
          if (tid == 0) {
            argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, tile_start);
            atomicAdd(&a.ctl->n_done[a.redo ? 1 : 0], 1u);  // CTAs that poll for hand-overs must not wait for this stream
          }
          return;
        }
        const int badpos = sm.badpos[bp];
        bp ^= 1;
        if (tid == 0) sm.badpos[bp] = 0x7fffffff;  // nobody reads or reports into it before the next window's barriers

        if (badpos >= wend) {
          // ---------------- phase C: exclusive time, parent region, interval records; carried stack -------------
          const u64 pos0 = out_base + n_int;
#pragma unroll
          for (int i = 0; i < NI; ++i) {
            const int rk = (i == NI - 1 ? (tid + NT / 2) % NT : tid) + i * NT;
            if (rk < win_ne) {
              const u32 d = sm.desc[rk];
              const int partner = (int)(short)(refs[i] & 0xffffu), parent = (int)(short)(refs[i] >> 16);
              const uint4 ee = evb[d & ((1u << SM::kDescShift) - 1u)];
              const uint4 pe = evb[partner];
              const u64 ts = (u64)ee.x | ((u64)ee.y << 32), bts = (u64)pe.x | ((u64)pe.y << 32);
              const bool carried = (u32)partner >= (u32)T;
              const u64 child = (carried ? sm.cchild[cpar][partner - cbase] : 0ull) + accb[partner];
              u32 flags = 0;
              u64 incl = 0, excl = 0;
              if (ee.w != pe.w) { flags |= ARGUS_FLAG_CTX_MISMATCH; ++tot_ctx; }
              if (ts < bts) { flags |= ARGUS_FLAG_TIME_REVERSED; ++tot_rev; } else { incl = ts - bts; }
              if (child > incl) { flags |= ARGUS_FLAG_CHILD_CLAMPED; ++tot_clamp; } else { excl = incl - child; }
              const u32 bidx = carried ? sm.cidx[cpar][partner - cbase] : tile_start + (u32)partner;
              const u32 preg = parent == cbase + kSink ? ARGUS_NONE : (reinterpret_cast<const u32*>(evb + parent)[2] >> 1);
              const u64 pos = pos0 + (u64)rk;
              if (pos < a.interval_capacity) {
                uint4* q = reinterpret_cast<uint4*>(a.intervals + pos);
                q[0] = make_uint4(pe.x, pe.y, (u32)incl, (u32)(incl >> 32));
                q[1] = make_uint4((u32)excl, (u32)(excl >> 32), pe.z >> 1, pe.w);
                q[2] = make_uint4(s, preg, bidx, (d >> SM::kDescShift) | (flags << 16));
                if (a.digest) a.digest[pos] = argus_digest_pack(pe.z >> 1, incl, excl, flags);
              } else if (!a.redo) {
                a.ctl->spec_overflow = 1;
              }
            }
          }
          const int new_ch = ch + win_nb - win_ne;
          if (tid < new_ch) {  // the stack this window leaves behind, in the next window's index space
            const int e = tile_latest_begin<NT, E>(sm, tid, lbase, T);
            const int from = e >= 0 ? e : cbase + tid;
            car_next[tid] = evb[from];
            sm.cchild[cpar ^ 1][tid] = (e >= 0 ? 0ull : sm.cchild[cpar][tid]) + accb[from];
            sm.cidx[cpar ^ 1][tid] = e >= 0 ? tile_start + (u32)e : sm.cidx[cpar][tid];
          }
          small_streak = (wend - w0 < 32) ? small_streak + 1 : 0;
          ch = new_ch;
          n_int += (u64)win_ne;
          cpar ^= 1;
          w0 = wend;
          wend = tn;
          __syncthreads();
        } else if (badpos > w0) {
          wend = badpos;  // [w0, badpos) is well nested: do it again on its own (nothing was committed yet)
        } else {
          // ---------------- the marker(s) at w0 go through the sequential stack machine ----------------
          const int nseq = small_streak >= 2 ? ((tn - w0) < kSeqChunk ? (tn - w0) : kSeqChunk) : 1;
          if (tid < ch) {
            const uint4 f = evb[cbase + tid];
            ArgusFrame& o = sm.fstk[tid];
            o.ts = (u64)f.x | ((u64)f.y << 32); o.child = sm.cchild[cpar][tid]; o.region = f.z >> 1; o.ctx = f.w;
            o.idx = sm.cidx[cpar][tid]; o.pad = 0;
          }
          __syncthreads();
          if (tid == 0) {
            ArgusSeqState st;
            st.h = ch; st.n_int = n_int; st.n_ctx = st.n_rev = st.n_clamp = 0; st.failed = false;
            bool ok = true;
            for (int e = w0; e < w0 + nseq && ok; ++e) {
              const uint4 pe = evb[e];
              ok = argus_seq_step(a, sm.fstk, st, s, gpos0, out_base, tile_start + (u32)e, (u64)pe.x | ((u64)pe.y << 32), pe.z, pe.w);
            }
            tot_ctx += st.n_ctx; tot_rev += st.n_rev; tot_clamp += st.n_clamp;
            sm.ch = st.h;
            sm.n_int = st.n_int;
            sm.failed = ok ? 0 : 1;
            if (!a.redo) atomicAdd((u64*)&a.status->n_sequential_tiles, 1ull);
          }
          __syncthreads();
          ch = sm.ch;
          n_int = sm.n_int;
          if (sm.failed) stream_failed = true;
          if (tid < ch) {
            const ArgusFrame f = sm.fstk[tid];
            car_next[tid] = make_uint4((u32)f.ts, (u32)(f.ts >> 32), f.region << 1, f.ctx);
            sm.cchild[cpar ^ 1][tid] = f.child;
            sm.cidx[cpar ^ 1][tid] = f.idx;
          }
          cpar ^= 1;
          w0 += nseq;
          wend = tn;
          ++small_streak;
          __syncthreads();
          if (stream_failed) break;
        }
      }  // windows
      if (stream_failed) {
        if (ti + 1 < ti_end) {  // drain the prefetched tile before the buffer is reused
          const bool ok = mbar_wait_bounded(&sm.bar[b ^ 1], (b ^ 1) ? ph1 : ph0);
          if (b ^ 1) ph1 ^= 1; else ph0 ^= 1;
          if (!ok) sm.dead = 1;
        }
        break;
      }
    }  // tiles


    __syncthreads();
    if (sm.dead) {
      if (tid == 0) {
        argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, 0);
        atomicAdd(&a.ctl->n_done[a.redo ? 1 : 0], 1u);
      }
      return;
    }
    if (!stream_failed && ti_end < ntiles) {
      // hand the stream on: its state goes into the record, the record into the queue
      ArgusStreamRecord* r = a.records + rec;
      if (tid == 0) { r->stream = s; r->next_tile = ti_end; r->ch = ch; r->n_int = n_int; }
      if (tid < ch) {
        r->frames[tid] = sm.evall[T + cpar * kCar + tid];
        r->child[tid] = sm.cchild[cpar][tid];
        r->idx[tid] = sm.cidx[cpar][tid];
      }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const u64 slot = atomicAdd(reinterpret_cast<unsigned long long*>(&a.ctl->q_tail[a.redo ? 1 : 0]), 1ull);
        if (slot < a.queue_capacity) *reinterpret_cast<volatile u32*>(a.queue + slot) = rec + 1;
      }
    } else {
      if (!a.redo) {
        // frames still open at the end of the stream (they sit in the block the next tile would read)
        if (!stream_failed && tid < ch) argus_note_ambiguity(a, gpos0 + sm.cidx[cpar][tid], ARGUS_AMBIG_BEGIN_EOS, (u32)tid);
        if (tid == 0) a.counts[s] = n_int;
      }
      if (tid == 0) atomicAdd(&a.ctl->n_done[a.redo ? 1 : 0], 1u);
    }
    __syncthreads();
  }  // streams

  if (!a.redo) {
    tot_ctx = __reduce_add_sync(0xffffffffu, tot_ctx);
    tot_rev = __reduce_add_sync(0xffffffffu, tot_rev);
    tot_clamp = __reduce_add_sync(0xffffffffu, tot_clamp);
    if (lane == 0) {
      if (tot_ctx) atomicAdd((u64*)&a.status->n_ctx_mismatch, (u64)tot_ctx);
      if (tot_rev) atomicAdd((u64*)&a.status->n_time_reversed, (u64)tot_rev);
      if (tot_clamp) atomicAdd((u64*)&a.status->n_child_clamped, (u64)tot_clamp);
    }
  }
}

// The shared-memory opt-in and the occupancy of one instantiation belong to one device: looked up once per
// device, under a lock (two host threads may make their first call at the same time).
template <int NT, int E, int MINB, bool RING>
int launch_tiled(const ArgusPairArgs& a, cudaStream_t stream) {
  constexpr int kMaxDevices = 64;
  static int grid_of[kMaxDevices];
  static std::mutex mu;
  constexpr size_t smem = ((sizeof(TileSmem<NT, E>) + 15) & ~(size_t)15) + 128;
  int dev = 0;
  ARGUS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ARGUS_ERR_INVALID_ARG;
  int grid_cache;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (!grid_of[dev]) {
      ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_pair_tiled<NT, E, MINB, RING>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      int sms = 0, per_sm = 0;
      ARGUS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
      ARGUS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pair_tiled<NT, E, MINB, RING>, NT, smem));
      if (per_sm < 1) return ARGUS_ERR_CUDA;
      if (per_sm > MINB) per_sm = MINB;
      grid_of[dev] = sms * per_sm;
    }
    grid_cache = grid_of[dev];
  }
  const u32 grid = a.num_streams < (u32)grid_cache ? a.num_streams : (u32)grid_cache;
  k_pair_tiled<NT, E, MINB, RING><<<grid, NT, smem, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

std::atomic<int> g_variant{0};

}  // namespace

bool argus_pair_tiled_usable(const ArgusPairArgs& a) { return a.num_streams > 0; }

// Tile shape used by the tiled kernel: 0 = the default; 1..3 select the other compiled shapes
// <threads, events per thread, CTAs per SM> (test aid: tiles end at other places; results do not depend on it).
extern "C" void argus_set_tile_variant(int v) { g_variant.store(v); }

int argus_launch_pair_tiled(const ArgusPairArgs& a, cudaStream_t stream) {
  if (a.ring_written) return launch_tiled<128, 5, 7, true>(a, stream);  // ring container: one shape
  switch (g_variant.load(std::memory_order_relaxed)) {
    case 1: return launch_tiled<192, 5, 4, false>(a, stream);
    case 2: return launch_tiled<64, 5, 8, false>(a, stream);
    case 3: return launch_tiled<256, 7, 2, false>(a, stream);
    default: return launch_tiled<128, 5, 7, false>(a, stream);  // seven CTAs of 128 threads per SM
  }
}
