// argus_pair_tiled.cu — tiled pairing kernel for sm_100a.
//
// One CTA walks one stream tile by tile (T = NT * E events per tile); tiles arrive in shared
// memory by TMA bulk copies (double buffered, mbarrier completion) and interval records leave with
// coalesced 16-byte stores, one thread per record. The per-stream region stack is carried from tile
// to tile in shared memory, so CTAs never wait on one another.
//
// Inside a tile every thread owns E consecutive events (E odd: conflict-free 16-byte shared loads)
// and the stack height before each event comes from a block-wide prefix sum of +1/-1. With heights
// known, a frame is identified by its level (stack position):
//   - begin/end pairs that fall inside one thread are matched by that thread with a 4-bit-per-entry
//     register stack;
//   - an end whose begin lies in an earlier thread finds it through per-level bitmasks of the
//     threads that leave a begin open at that level (latest such thread before it); if there is
//     none, the begin is in the stack carried from earlier tiles;
//   - every finished interval adds its inclusive time to its parent frame's accumulator (shared
//     atomics), which gives exclusive time without ordering the threads.
// This is exact when the tile is well nested (every end meets the frame on top with the same region
// id). Any doubt (region mismatch, negative height, bad region id, depth overflow, level window
// exceeded) makes the CTA redo that tile with the sequential stack machine on the carried stack, so
// the result is always the sequential definition's.
#include "argus_pair_common.cuh"

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

#ifdef ARGUS_TILE_TIMING
__device__ unsigned long long g_tile_timing[8];
#define TT_MARK(i) do { if (tid == 0) { const long long c__ = clock64(); tt[i] += (unsigned long long)(c__ - tlast); tlast = c__; } } while (0)
#else
#define TT_MARK(i) do { } while (0)
#endif

constexpr int kLevelWindow = 32;  // levels [lbase, lbase + 32) may hold open begins of a tile
constexpr int kCar = 80;          // slots of a carried-frame block: 64 frames, 1 sink for "no parent", padding
constexpr int kSink = 64;         // index of the sink slot inside a carried-frame block

// Shared memory of one CTA. Events of the two tile buffers and the frames carried from earlier tiles
// share one index space, so that "the frame an end closes" and "its parent" are plain indices:
//   ev0[0..T) | car0[0..80) | car1[0..80) | ev1[0..T)
// A tile in buffer 0 addresses carried level L as T + L (car0); a tile in buffer 1 as L - 80 (car1).
// The tile in buffer b reads car_b and writes the stack it leaves behind into car_{b^1}.
template <int NT, int E>
struct TileSmem {
  static constexpr int T = NT * E;
  static constexpr int NW = NT / 32;
  static constexpr int MAXI = T / 2 + ARGUS_MAX_DEPTH;  // intervals a well-nested tile can emit
  static constexpr int NI = (MAXI + NT - 1) / NT;       // intervals per thread in the emission phases
  uint4 evall[2 * T + 2 * kCar];
  u64 accall[T + 2 * kCar];        // child time per frame, same index space shifted by kCar
  uint2 desc[MAXI];                // per end, in end order: {end idx | partner << 16, parent | depth << 16}
  u32 cidx[2][ARGUS_MAX_DEPTH];    // begin index (within the stream) of each carried frame
  u64 cchild[2][ARGUS_MAX_DEPTH];  // child time of each carried frame as the tile found it (for the redo path)
  ArgusFrame fstk[ARGUS_MAX_DEPTH];  // stack in the layout the sequential redo path uses
  u64 opens[NT];                   // per thread: local indices of begins left open (top = low nibble)
  int hend[NT];                    // per thread: stack height after its last event
  u32 mask[kLevelWindow][NW];      // per level: threads that leave a begin open at that level
  u32 wmask[kLevelWindow];         // per level: warps with a non-zero mask word
  short prev[kLevelWindow][NW + 1];  // per level and warp w: latest open begin in warps < w (tile index or -1); [NW] = all warps
  u32 warp_tot[32];
  u64 bar[2];
  u64 cur_stream;
  u64 n_int;                       // written by the sequential redo path
  int ch;
  int bad, dead, failed;
};

template <int NT, int E, int MINB>
__global__ void __launch_bounds__(NT, MINB) k_pair_tiled(ArgusPairArgs a) {
  using SM = TileSmem<NT, E>;
  constexpr int T = SM::T, NW = SM::NW, MAXI = SM::MAXI, NI = SM::NI;
  constexpr int kBad = 0x3fff;  // reference that marks a tile as not well nested
  static_assert(E % 2 == 1 && E <= 15, "E must be odd and fit 4-bit indices");
  static_assert(NW <= 16 && NT % 32 == 0 && NT >= ARGUS_MAX_DEPTH && T + kCar < kBad, "block shape");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  SM& sm = *reinterpret_cast<SM*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (a.redo && !a.ctl->redo) return;
  if (tid == 0) {
    mbar_init(&sm.bar[0], 1);
    mbar_init(&sm.bar[1], 1);
    fence_mbar_init();
    sm.dead = 0;
  }
  __syncthreads();
  u32 ph0 = 0, ph1 = 0;  // mbarrier phase parities
  const u64 off0 = a.stream_offsets[0];
  u32 tot_ctx = 0, tot_rev = 0, tot_clamp = 0;
#ifdef ARGUS_TILE_TIMING
  unsigned long long tt[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  long long tlast = clock64();
#endif

  for (;;) {
    if (tid == 0) sm.cur_stream = atomicAdd(a.redo ? &a.ctl->ticket2 : &a.ctl->ticket, 1ull);
    __syncthreads();
    const u64 s64 = sm.cur_stream;
    if (s64 >= a.num_streams) break;
    const u32 s = (u32)s64;
    const u64 lo = a.stream_offsets[s], hi = a.stream_offsets[s + 1];
    if (hi < lo || hi > a.num_events || lo < off0 || ((hi - lo) >> 32)) {
      if (tid == 0) {
        argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
        if (!a.redo) a.counts[s] = 0;
      }
      __syncthreads();
      continue;
    }
    const u32 n = (u32)(hi - lo);
    const u64 gpos0 = lo - off0;
    const u64 out_base = a.redo ? a.interval_offsets[s] : (gpos0 >> 1);
    const argus_event_t* src = a.events + lo;
    const u32 ntiles = (n + T - 1) / T;
    int ch = 0;          // carried stack height (uniform)
    u64 n_int = 0;       // intervals of this stream so far (uniform)
    bool stream_failed = false;
    if (tid == 0 && ntiles > 0) {
      const u32 bytes = (n < (u32)T ? n : (u32)T) * 16u;
      mbar_expect_tx(&sm.bar[0], bytes);
      tma_load_1d(sm.evall, src, bytes, &sm.bar[0]);
    }

    for (u32 ti = 0; ti < ntiles; ++ti) {
      const int b = ti & 1;
      const u32 tile_start = ti * (u32)T;
      const int tn = (int)((n - tile_start) < (u32)T ? (n - tile_start) : (u32)T);
      uint4* const ev0 = sm.evall;
      uint4* const ev1 = sm.evall + T + 2 * kCar;
      const uint4* evb = b ? ev1 : ev0;                  // evb[ref] for every reference of this tile
      u64* accb = sm.accall + kCar;                      // accb[ref]
      const int cbase = b ? -kCar : T;                   // carried level L of this tile -> reference cbase + L
      const int nbase = b ? T : -kCar;                   // same for the next tile (other buffer)
      uint4* const car_next = sm.evall + T + (b ? 0 : kCar);
      if (tid == 0 && ti + 1 < ntiles) {  // prefetch the next tile into the other buffer
        const u32 nstart = tile_start + T;
        const u32 bytes = ((n - nstart) < (u32)T ? (n - nstart) : (u32)T) * 16u;
        mbar_expect_tx(&sm.bar[b ^ 1], bytes);
        tma_load_1d(b ? ev0 : ev1, src + nstart, bytes, &sm.bar[b ^ 1]);
      }
      TT_MARK(0);
      {
        const bool ok = mbar_wait_bounded(&sm.bar[b], b ? ph1 : ph0);
        if (b) ph1 ^= 1; else ph0 ^= 1;
        if (!ok) sm.dead = 1;
      }
      TT_MARK(1);

      // ---------------- phase A: local shape, prefix sums, open-level masks ----------------
      u32 tags[E];
      u32 valid = 0;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const int e = tid * E + k;
        tags[k] = reinterpret_cast<const u32*>(evb + e)[2];
        if (e < tn) valid |= 1u << k;
        accb[e] = 0;
      }
      u64 stk = 0;
      int lsp = 0, npend = 0, nb = 0, ne = 0, rel = 0, maxrel = 0;
      bool bad = false;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        if (valid & (1u << k)) {
          if ((tags[k] >> 1) >= a.num_regions) bad = true;
          if (tags[k] & 1u) {
            ++ne; --rel;
            if (lsp > 0) { stk >>= 4; --lsp; } else { ++npend; }
          } else {
            ++nb; ++rel;
            stk = (stk << 4) | (u64)k; ++lsp;
            maxrel = rel > maxrel ? rel : maxrel;
          }
        }
      }
      // zero the per-tile tables before the scan's barrier
      sm.mask[tid / NW][tid % NW] = 0;
      if (tid < kLevelWindow) sm.wmask[tid] = 0;
      if (tid == 0) { sm.bad = 0; sm.failed = 0; accb[cbase + kSink] = 0; }
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
      const int tile_nb = (int)(tot & 0xffffu), tile_ne = (int)(tot >> 16);
      const int h0 = ch + (int)(ex & 0xffffu) - (int)(ex >> 16);
      const int rank0 = (int)(ex >> 16);
      const int hend = h0 + nb - ne;
      const int lbase = ch > 16 ? ch - 16 : 0;
      if (h0 - npend < 0 || h0 + maxrel > ARGUS_MAX_DEPTH || tile_ne > MAXI) bad = true;
      const int olo = lsp > 0 ? hend - lsp - lbase : 1000;  // levels of the begins this thread leaves open
      const int ohi = lsp > 0 ? hend - lbase : -1000;       // (relative to lbase, half-open)
      if (lsp > 0 && (olo < 0 || ohi > kLevelWindow)) bad = true;
      const u64 opens_reg = stk;
      sm.opens[tid] = stk;
      sm.hend[tid] = hend;
      u32 mine = 0;  // lane l: threads of this warp that leave a begin open at level lbase + l
      {
        int wlo = __reduce_min_sync(0xffffffffu, olo), whi = __reduce_max_sync(0xffffffffu, ohi);
        wlo = wlo < 0 ? 0 : wlo;
        whi = whi > kLevelWindow ? kLevelWindow : whi;
        for (int l = wlo; l < whi; ++l) {
          const u32 bal = __ballot_sync(0xffffffffu, l >= olo && l < ohi);
          if (lane == l) mine = bal;
        }
        if (mine) {
          sm.mask[lane][warp] = mine;
          atomicOr(&sm.wmask[lane], 1u << warp);
        }
      }
      if (bad) sm.bad = 1;
      __syncthreads();
      {  // per (level, warp): the latest open begin among the warps before it
        const int l = tid / NW, w = tid % NW;
        const u32 wm = sm.wmask[l];
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const int wq = pass ? NW : w;
          if (pass && w != NW - 1) break;
          const u32 ww = wm & ((1u << wq) - 1u);
          int e = -1;
          if (ww) {
            const int wp = 31 - __clz(ww);
            const u32 m = sm.mask[l][wp];
            if (m) {
              const int tau = wp * 32 + 31 - __clz(m);
              const int sh = 4 * (sm.hend[tau] - 1 - (lbase + l));
              e = tau * E + (int)((sm.opens[tau] >> (sh & 63)) & 15ull);
            }
          }
          sm.prev[l][wq] = (short)e;
        }
      }
      __syncthreads();
      TT_MARK(2);

      // ---------------- phase B1: one descriptor per end marker (who is my begin, who is my parent) -------------
      const int nmax = __reduce_max_sync(0xffffffffu, npend);  // warp-wide: the loop below shuffles, so every lane runs it
      // frames below this thread's floor, outermost needed first: level h0-1-j for j = 0..npend, 15 bits each
      u64 outer_lo = 0, outer_hi = 0;
      {
        for (int j = 0; j <= nmax; ++j) {
          const int L = h0 - 1 - j;
          const int l = L - lbase;
          const bool want = j <= npend && L >= 0 && l >= 0 && l < kLevelWindow;
          // the mask word of my warp for level l sits in lane l's register
          const u32 mword = __shfl_sync(0xffffffffu, mine, want ? l : 0);
          const u32 m = want ? (mword & ((1u << lane) - 1u)) : 0u;
          const int srcl = m ? 31 - __clz(m) : lane;
          const int hend_s = __shfl_sync(0xffffffffu, hend, srcl);
          const u64 opens_s = __shfl_sync(0xffffffffu, opens_reg, srcl);
          int ref;
          if (j > npend) ref = 0;
          else if (L < 0) ref = cbase + kSink;
          else {
            if (m) ref = (warp * 32 + srcl) * E + (int)((opens_s >> ((4 * (hend_s - 1 - L)) & 63)) & 15ull);
            else ref = want ? (int)sm.prev[l][warp] : -1;
            if (ref < 0) ref = L < ch ? cbase + L : kBad;
          }
          const u64 v = (u64)((u32)ref & 0x7fffu);
          if (j < 4) outer_lo |= v << (15 * j); else outer_hi |= v << (15 * ((j - 4) & 3));
          if (j >= 8 && j <= npend) bad = true;  // more than 8 frames closed from outside: leave it to the redo path
        }
      }
      if (!bad) {
        int h = h0, rank = rank0, pi = 0;
        stk = 0; lsp = 0;
        auto outer_at = [&](int j) -> int {
          const u64 w = j < 4 ? outer_lo : outer_hi;
          int r = (int)((w >> (15 * (j & 3))) & 0x7fffull);
          return (r & 0x4000) ? r - 0x8000 : r;  // sign-extend 15 bits (carried references of buffer 1 are negative)
        };
#pragma unroll
        for (int k = 0; k < E; ++k) {
          if (!(valid & (1u << k))) continue;
          if (!(tags[k] & 1u)) {
            stk = (stk << 4) | (u64)k; ++lsp; ++h;
            continue;
          }
          --h;  // level of the frame this end closes
          int partner, parent;
          if (lsp > 0) {
            partner = tid * E + (int)(stk & 15ull);
            stk >>= 4; --lsp;
            parent = lsp > 0 ? tid * E + (int)(stk & 15ull) : outer_at(pi);
          } else {
            partner = outer_at(pi);
            ++pi;
            parent = outer_at(pi);
            if (h < 0) bad = true;
          }
          if (partner == kBad || parent == kBad) bad = true;
          sm.desc[rank++] = make_uint2((u32)(tid * E + k) | ((u32)partner << 16), ((u32)parent & 0xffffu) | ((u32)h << 16));
        }
        if (bad) sm.bad = 1;
      }
      __syncthreads();
      TT_MARK(3);

      // ---------------- phase B2a: one thread per end marker: inclusive time feeds the parent frame -------------
      if (!sm.bad) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int rk = tid + i * NT;
          if (rk < tile_ne) {
            const uint2 d = sm.desc[rk];
            const uint4 ee = evb[d.x & 0xffffu];
            const uint4 pe = evb[(int)(short)(d.x >> 16)];
            if ((pe.z >> 1) != (ee.z >> 1) || (pe.z & 1u)) sm.bad = 1;
            const u64 ts = (u64)ee.x | ((u64)ee.y << 32), bts = (u64)pe.x | ((u64)pe.y << 32);
            if (ts > bts) {  // 64-bit add as two native 32-bit shared atomics; each carry is propagated exactly once
              const u64 dlt = ts - bts;
              u32* p = reinterpret_cast<u32*>(&accb[(int)(short)(d.y & 0xffffu)]);
              const u32 lo32 = (u32)dlt, hi32 = (u32)(dlt >> 32);
              const u32 old = atomicAdd(p, lo32);
              if (hi32) atomicAdd(p + 1, hi32);
              if (old + lo32 < old) atomicAdd(p + 1, 1u);
            }
          }
        }
      }
      __syncthreads();
      TT_MARK(4);
      const bool tile_bad = sm.bad != 0;
      if (sm.dead) {  // a bulk copy never arrived: report and leave (uniform decision)
        if (tid == 0) argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, tile_start);
        return;
      }

      if (!tile_bad) {
        // ---------------- phase B2b: exclusive time, parent region, interval records; carried stack -------------
        const u64 pos0 = out_base + n_int;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int rk = tid + i * NT;
          if (rk < tile_ne) {
            const uint2 d = sm.desc[rk];
            const int partner = (int)(short)(d.x >> 16), parent = (int)(short)(d.y & 0xffffu);
            const uint4 ee = evb[d.x & 0xffffu];
            const uint4 pe = evb[partner];
            const u64 ts = (u64)ee.x | ((u64)ee.y << 32), bts = (u64)pe.x | ((u64)pe.y << 32);
            const u64 child = accb[partner];
            u32 flags = 0;
            u64 incl = 0, excl = 0;
            if (ee.w != pe.w) { flags |= ARGUS_FLAG_CTX_MISMATCH; ++tot_ctx; }
            if (ts < bts) { flags |= ARGUS_FLAG_TIME_REVERSED; ++tot_rev; } else { incl = ts - bts; }
            if (child > incl) { flags |= ARGUS_FLAG_CHILD_CLAMPED; ++tot_clamp; } else { excl = incl - child; }
            const bool carried = (u32)partner >= (u32)T;
            const u32 bidx = carried ? sm.cidx[b][partner - cbase] : tile_start + (u32)partner;
            const u32 preg = parent == cbase + kSink ? ARGUS_NONE : (reinterpret_cast<const u32*>(evb + parent)[2] >> 1);
            const u64 pos = pos0 + (u64)rk;
            if (pos < a.interval_capacity) {
              uint4* q = reinterpret_cast<uint4*>(a.intervals + pos);
              q[0] = make_uint4(pe.x, pe.y, (u32)incl, (u32)(incl >> 32));
              q[1] = make_uint4((u32)excl, (u32)(excl >> 32), pe.z >> 1, pe.w);
              q[2] = make_uint4(s, preg, bidx, (d.y >> 16) | (flags << 16));
            } else if (!a.redo) {
              a.ctl->spec_overflow = 1;
            }
          }
        }
        const int new_ch = ch + tile_nb - tile_ne;
        if (tid < new_ch) {  // the stack this tile leaves behind, in the next tile's index space
          const int l = tid - lbase;
          const int e = (l >= 0 && l < kLevelWindow) ? (int)sm.prev[l][NW] : -1;
          const int from = e >= 0 ? e : cbase + tid;
          car_next[tid] = evb[from];
          accb[nbase + tid] = accb[from];
          sm.cidx[b ^ 1][tid] = e >= 0 ? tile_start + (u32)e : sm.cidx[b][tid];
          sm.cchild[b ^ 1][tid] = accb[from];
        }
        ch = new_ch;
        n_int += (u64)tile_ne;
        __syncthreads();
        TT_MARK(5);
      } else {
        // ---------------- redo this tile with the sequential stack machine ----------------
        if (tid < ch) {
          const uint4 f = evb[cbase + tid];
          ArgusFrame& o = sm.fstk[tid];
          o.ts = (u64)f.x | ((u64)f.y << 32); o.child = sm.cchild[b][tid]; o.region = f.z >> 1; o.ctx = f.w;
          o.idx = sm.cidx[b][tid]; o.pad = 0;
        }
        __syncthreads();
        if (tid == 0) {
          ArgusSeqState st;
          st.h = ch; st.n_int = n_int; st.n_ctx = st.n_rev = st.n_clamp = 0; st.failed = false;
          bool ok = true;
          for (int e = 0; e < tn && ok; ++e) {
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
          accb[nbase + tid] = f.child;
          sm.cidx[b ^ 1][tid] = f.idx;
          sm.cchild[b ^ 1][tid] = f.child;
        }
        __syncthreads();
      }
      if (stream_failed) {
        if (ti + 1 < ntiles) {  // drain the prefetched tile before the buffer is reused
          const bool ok = mbar_wait_bounded(&sm.bar[b ^ 1], (b ^ 1) ? ph1 : ph0);
          if (b ^ 1) ph1 ^= 1; else ph0 ^= 1;
          if (!ok) sm.dead = 1;
        }
        break;
      }
    }  // tiles

    __syncthreads();
    if (sm.dead) {
      if (tid == 0) argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, 0);
      return;
    }
    if (!a.redo) {
      // frames still open at the end of the stream (they sit in the block the next tile would read)
      const int bl = (int)(ntiles & 1u);
      if (!stream_failed && tid < ch) argus_note_ambiguity(a, gpos0 + sm.cidx[bl][tid], ARGUS_AMBIG_BEGIN_EOS, (u32)tid);
      if (tid == 0) a.counts[s] = n_int;
    }
    __syncthreads();
  }  // streams

#ifdef ARGUS_TILE_TIMING
  if (tid == 0 && !a.redo) for (int i = 0; i < 8; ++i) atomicAdd(&g_tile_timing[i], tt[i]);
#endif
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
template <int NT, int E, int MINB>
int launch_tiled(const ArgusPairArgs& a, cudaStream_t stream) {
  static int grid_cache = 0;
  const size_t smem = sizeof(TileSmem<NT, E>) + 128;
  if (!grid_cache) {
    ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_pair_tiled<NT, E, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int dev = 0, sms = 0, per_sm = 0;
    ARGUS_CUDA_TRY(cudaGetDevice(&dev));
    ARGUS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ARGUS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pair_tiled<NT, E, MINB>, NT, smem));
    if (per_sm < 1) return ARGUS_ERR_CUDA;
    grid_cache = sms * per_sm;
  }
  const u32 grid = a.num_streams < (u32)grid_cache ? a.num_streams : (u32)grid_cache;
  k_pair_tiled<NT, E, MINB><<<grid, NT, smem, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

int g_variant = 0;

}  // namespace

bool argus_pair_tiled_usable(const ArgusPairArgs& a) { return a.num_streams > 0; }

#ifdef ARGUS_TILE_TIMING
// Debug build only: cycles thread 0 of every CTA spent per phase (other, wait, A, B1, B2a, B2b), summed; resets them.
extern "C" int argus_debug_tile_timing(unsigned long long* out8) {
  if (cudaMemcpyFromSymbol(out8, g_tile_timing, 64) != cudaSuccess) return ARGUS_ERR_CUDA;
  unsigned long long z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (cudaMemcpyToSymbol(g_tile_timing, z, 64) != cudaSuccess) return ARGUS_ERR_CUDA;
  return ARGUS_OK;
}
#endif

// Tile shape used by the tiled kernel: 0 = default. Other values select alternative shapes (tuning aid).
extern "C" void argus_set_tile_variant(int v) { g_variant = v; }

int argus_launch_pair_tiled(const ArgusPairArgs& a, cudaStream_t stream) {
  switch (g_variant) {
    case 1: return launch_tiled<128, 7, 4>(a, stream);
    case 2: return launch_tiled<128, 9, 4>(a, stream);
    case 3: return launch_tiled<256, 7, 2>(a, stream);
    case 4: return launch_tiled<128, 5, 6>(a, stream);
    case 5: return launch_tiled<128, 11, 3>(a, stream);
    case 6: return launch_tiled<256, 9, 2>(a, stream);
    case 7: return launch_tiled<128, 5, 5>(a, stream);
    case 8: return launch_tiled<64, 9, 8>(a, stream);
    default: return launch_tiled<256, 5, 3>(a, stream);
  }
}
