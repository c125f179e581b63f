// argus_pair_tiled.cu — tiled pairing kernel for sm_100a.
//
// One CTA walks one stream tile by tile (T = NT * E events per tile); tiles arrive in shared
// memory by TMA bulk copies (double buffered, mbarrier completion) and the tile's intervals leave
// through a shared-memory staging buffer and one TMA bulk store. The per-stream region stack is
// carried from tile to tile in shared memory, so CTAs never wait on one another.
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
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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
__device__ __forceinline__ void tma_store_1d(void* dst, const void* src, u32 bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Bounded wait: gives up after ~2^22 polls (seconds); the caller then reports ARGUS_ERR_TIMEOUT.
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity) {
  for (u32 it = 0; it < (1u << 22); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}

constexpr int kLevelWindow = 32;  // levels [lbase, lbase + 32) may hold open begins of a tile

template <int NT, int E>
struct TileSmem {
  static constexpr int T = NT * E;
  static constexpr int NW = NT / 32;
  static constexpr int MAXI = T / 2 + ARGUS_MAX_DEPTH;  // intervals a well-nested tile can emit
  uint4 ev[2][T];                  // two event tiles (TMA destinations)
  uint4 stage[MAXI * 3];           // interval records of the current tile (TMA source)
  u64 fchild[T];                   // per begin: inclusive time of its finished children
  ArgusFrame cstack[2][ARGUS_MAX_DEPTH];  // carried stack, double buffered across the carry update
  u64 cacc[ARGUS_MAX_DEPTH];       // this tile's child time for frames of the carried stack
  u64 opens[NT];                   // per thread: local indices of begins left open (top = low nibble)
  int hend[NT];                    // per thread: stack height after its last event
  u32 fix[E][NT];                  // per thread: staged intervals that still need their child time
  u32 mask[kLevelWindow][NW];      // per level: threads that leave a begin open at that level
  u32 wmask[kLevelWindow];         // per level: warps with a non-zero mask word
  u32 scan_ws[36];
  u64 bar[2];
  u64 cur_stream;
  u64 n_int;                       // written by the sequential redo path
  int ch;
  int bad, dead, failed;
};

template <int NT, int E>
__device__ __forceinline__ int tile_lookup(const TileSmem<NT, E>& sm, int L, int lbase, int warp, int lane) {
  // latest begin left open at level L by a thread before (warp, lane); -1 if none in this tile
  const int l = L - lbase;
  if (l < 0 || l >= kLevelWindow) return -1;
  u32 m = warp < TileSmem<NT, E>::NW ? (sm.mask[l][warp] & ((1u << lane) - 1u)) : 0u;
  int w = warp;
  if (!m) {
    const u32 ww = sm.wmask[l] & ((1u << warp) - 1u);
    if (!ww) return -1;
    w = 31 - __clz(ww);
    m = sm.mask[l][w];
    if (!m) return -1;
  }
  const int tau = w * 32 + 31 - __clz(m);
  const int sh = 4 * (sm.hend[tau] - 1 - L);
  const int j = (int)((sm.opens[tau] >> (sh & 63)) & 15ull);
  return tau * E + j;
}

template <int NT, int E>
__global__ void __launch_bounds__(NT) k_pair_tiled(ArgusPairArgs a) {
  using SM = TileSmem<NT, E>;
  constexpr int T = SM::T, NW = SM::NW, MAXI = SM::MAXI;
  static_assert(E % 2 == 1 && E <= 15, "E must be odd (bank-conflict-free) and fit 4-bit indices");
  static_assert(NW <= 16, "warp masks are 16 bits wide at most");
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
  bool stores_pending = false;  // thread 0: a bulk store group may still be reading `stage`

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
    int cs = 0;          // which carried-stack buffer is current
    bool stream_failed = false;
    if (tid == 0 && ntiles > 0) {
      const u32 bytes = (n < (u32)T ? n : (u32)T) * 16u;
      mbar_expect_tx(&sm.bar[0], bytes);
      tma_load_1d(sm.ev[0], src, bytes, &sm.bar[0]);
    }

    for (u32 ti = 0; ti < ntiles; ++ti) {
      const int b = ti & 1;
      const u32 tile_start = ti * (u32)T;
      const int tn = (int)((n - tile_start) < (u32)T ? (n - tile_start) : (u32)T);
      if (tid == 0 && ti + 1 < ntiles) {  // prefetch the next tile into the other buffer
        const u32 nstart = tile_start + T;
        const u32 bytes = ((n - nstart) < (u32)T ? (n - nstart) : (u32)T) * 16u;
        mbar_expect_tx(&sm.bar[b ^ 1], bytes);
        tma_load_1d(sm.ev[b ^ 1], src + nstart, bytes, &sm.bar[b ^ 1]);
      }
      {
        const bool ok = mbar_wait_bounded(&sm.bar[b], b ? ph1 : ph0);
        if (b) ph1 ^= 1; else ph0 ^= 1;
        if (!ok) sm.dead = 1;
      }

      // ---------------- phase A: local shape, prefix sums, open-level masks ----------------
      const uint4* evb = sm.ev[b];
      uint4 r[E];
      u32 valid = 0;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const int e = tid * E + k;
        if (e < tn) { r[k] = evb[e]; valid |= 1u << k; } else { r[k] = make_uint4(0, 0, 0, 0); }
        sm.fchild[e] = 0;
      }
      u64 stk = 0;
      int lsp = 0, npend = 0, nb = 0, ne = 0, rel = 0, maxrel = 0;
      bool bad = false;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        if (valid & (1u << k)) {
          if ((r[k].z >> 1) >= a.num_regions) bad = true;
          if (r[k].z & 1u) {
            ++ne; --rel;
            if (lsp > 0) { stk >>= 4; --lsp; } else { ++npend; }
          } else {
            ++nb; ++rel;
            stk = (stk << 4) | (u64)k; ++lsp;
            maxrel = rel > maxrel ? rel : maxrel;
          }
        }
      }
      // zero the per-tile tables before the scan's barriers
      sm.mask[tid / NW][tid % NW] = 0;
      if (tid < kLevelWindow) sm.wmask[tid] = 0;
      if (tid < ARGUS_MAX_DEPTH) sm.cacc[tid] = 0;
      if (tid == 0) { sm.bad = 0; sm.failed = 0; if (stores_pending) { tma_wait_read0(); stores_pending = false; } }
      u32 tot;
      const u32 ex = argus_block_exclusive_scan<u32>((u32)nb | ((u32)ne << 16), sm.scan_ws, &tot);
      const int tile_nb = (int)(tot & 0xffffu), tile_ne = (int)(tot >> 16);
      const int h0 = ch + (int)(ex & 0xffffu) - (int)(ex >> 16);
      const int rank0 = (int)(ex >> 16);
      const int hend = h0 + nb - ne;
      const int lbase = ch > 16 ? ch - 16 : 0;
      if (h0 - npend < 0 || h0 + maxrel > ARGUS_MAX_DEPTH || tile_ne > MAXI) bad = true;
      const int olo = lsp > 0 ? hend - lsp - lbase : 1000;  // levels of the begins this thread leaves open
      const int ohi = lsp > 0 ? hend - lbase : -1000;       // (relative to lbase, half-open)
      if (lsp > 0 && (olo < 0 || ohi > kLevelWindow)) bad = true;
      sm.opens[tid] = stk;
      sm.hend[tid] = hend;
      {
        int wlo = __reduce_min_sync(0xffffffffu, olo), whi = __reduce_max_sync(0xffffffffu, ohi);
        wlo = wlo < 0 ? 0 : wlo;
        whi = whi > kLevelWindow ? kLevelWindow : whi;
        u32 mine = 0;
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

      // ---------------- phase B: match, emit to staging, feed parent accumulators ----------------
      u32 t_ctx = 0, t_rev = 0, t_clamp = 0;
      int nfix = 0;
      const ArgusFrame* cst = sm.cstack[cs];
      if (!bad) {
        int h = h0, rank = rank0;
        stk = 0; lsp = 0;
        int outer_e = h > 0 ? tile_lookup<NT, E>(sm, h - 1, lbase, warp, lane) : -1;  // frame at level floor-1
#pragma unroll
        for (int k = 0; k < E; ++k) {
          if (!(valid & (1u << k))) continue;
          const u32 tag = r[k].z;
          if (!(tag & 1u)) {
            stk = (stk << 4) | (u64)k; ++lsp; ++h;
            continue;
          }
          --h;  // level of the frame this end closes
          const u64 ts = (u64)r[k].x | ((u64)r[k].y << 32);
          u64 bts = 0, child = 0;
          u32 bregion = 0xffffffffu, bctx = 0, bidx = 0;
          int parent_e, pref = -1;
          bool cross = false;
          if (lsp > 0) {
            const int ej = tid * E + (int)(stk & 15ull);
            stk >>= 4; --lsp;
            const uint4 pe = evb[ej];
            bts = (u64)pe.x | ((u64)pe.y << 32); bregion = pe.z >> 1; bctx = pe.w; bidx = tile_start + (u32)ej;
            child = sm.fchild[ej];
            parent_e = lsp > 0 ? tid * E + (int)(stk & 15ull) : outer_e;
          } else {
            cross = true;
            pref = outer_e;
            if (pref >= 0) {
              const uint4 pe = evb[pref];
              bts = (u64)pe.x | ((u64)pe.y << 32); bregion = pe.z >> 1; bctx = pe.w; bidx = tile_start + (u32)pref;
            } else if (h >= 0 && h < ch) {
              const ArgusFrame& f = cst[h];
              bts = f.ts; bregion = f.region; bctx = f.ctx; bidx = f.idx;
            }
            outer_e = h > 0 ? tile_lookup<NT, E>(sm, h - 1, lbase, warp, lane) : -1;
            parent_e = outer_e;
          }
          if (bregion != (tag >> 1)) { bad = true; break; }
          u32 flags = 0;
          u64 incl;
          if (r[k].w != bctx) { flags |= ARGUS_FLAG_CTX_MISMATCH; ++t_ctx; }
          if (ts < bts) { incl = 0; flags |= ARGUS_FLAG_TIME_REVERSED; ++t_rev; } else { incl = ts - bts; }
          u64 excl = 0;
          if (!cross) {
            if (child > incl) { flags |= ARGUS_FLAG_CHILD_CLAMPED; ++t_clamp; } else { excl = incl - child; }
          } else {
            sm.fix[nfix++][tid] = (u32)rank | ((u32)(pref + 1) << 16);
          }
          u32 preg = ARGUS_NONE;
          if (parent_e >= 0) {
            preg = evb[parent_e].z >> 1;
            if (incl) atomicAdd(&sm.fchild[parent_e], incl);
          } else if (h > 0) {
            if (h - 1 < ch) { preg = cst[h - 1].region; if (incl) atomicAdd(&sm.cacc[h - 1], incl); } else { bad = true; break; }
          }
          uint4* q = sm.stage + rank * 3;
          q[0] = make_uint4((u32)bts, (u32)(bts >> 32), (u32)incl, (u32)(incl >> 32));
          q[1] = make_uint4((u32)excl, (u32)(excl >> 32), bregion, bctx);
          q[2] = make_uint4(s, preg, bidx, ((u32)h & 0xffffu) | (flags << 16));
          ++rank;
        }
        if (bad) sm.bad = 1;
      }
      __syncthreads();
      const bool tile_bad = sm.bad != 0;
      if (sm.dead) {  // a bulk copy never arrived: report and leave (uniform decision)
        if (tid == 0) { argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, tile_start); tma_wait_all0(); }
        return;
      }

      if (!tile_bad) {
        // ---------------- phase C: finish cross-thread intervals, update the carried stack ----------------
        for (int f = 0; f < nfix; ++f) {
          const u32 fx = sm.fix[f][tid];
          const int slot = (int)(fx & 0xffffu), pref = (int)(fx >> 16) - 1;
          uint4* q = sm.stage + slot * 3;
          const uint4 q0 = q[0];
          uint4 q2 = q[2];
          const u64 incl = (u64)q0.z | ((u64)q0.w << 32);
          const int level = (int)(q2.w & 0xffffu);
          const u64 child = pref >= 0 ? sm.fchild[pref] : cst[level].child + sm.cacc[level];
          u64 excl = 0;
          if (child > incl) { q2.w |= ARGUS_FLAG_CHILD_CLAMPED << 16; ++t_clamp; q[2] = q2; } else { excl = incl - child; }
          uint4 q1 = q[1];
          q1.x = (u32)excl; q1.y = (u32)(excl >> 32);
          q[1] = q1;
        }
        const int new_ch = ch + tile_nb - tile_ne;
        if (tid < ARGUS_MAX_DEPTH && tid < new_ch) {
          const int e = tile_lookup<NT, E>(sm, tid, lbase, NW, 0);
          ArgusFrame f;
          if (e >= 0) {
            const uint4 pe = evb[e];
            f.ts = (u64)pe.x | ((u64)pe.y << 32); f.child = sm.fchild[e]; f.region = pe.z >> 1; f.ctx = pe.w;
            f.idx = tile_start + (u32)e; f.pad = 0;
          } else {
            f = cst[tid];
            f.child += sm.cacc[tid];
          }
          sm.cstack[cs ^ 1][tid] = f;
        }
        tot_ctx += t_ctx; tot_rev += t_rev; tot_clamp += t_clamp;
        fence_proxy_async();
        __syncthreads();
        if (tid == 0 && tile_ne > 0) {
          const u64 pos = out_base + n_int;
          u64 fit = (u64)tile_ne;
          if (pos + fit > a.interval_capacity) {
            fit = pos < a.interval_capacity ? a.interval_capacity - pos : 0;
            if (!a.redo) a.ctl->spec_overflow = 1;
          }
          if (fit) {
            tma_store_1d(a.intervals + pos, sm.stage, (u32)fit * 48u);
            tma_commit();
            stores_pending = true;
          }
        }
        ch = new_ch;
        n_int += (u64)tile_ne;
        cs ^= 1;
      } else {
        // ---------------- redo this tile with the sequential stack machine ----------------
        if (tid == 0) {
          ArgusSeqState st;
          st.h = ch; st.n_int = n_int; st.n_ctx = st.n_rev = st.n_clamp = 0; st.failed = false;
          ArgusFrame* stkp = sm.cstack[cs];
          bool ok = true;
          for (int e = 0; e < tn && ok; ++e) {
            const uint4 pe = evb[e];
            ok = argus_seq_step(a, stkp, st, s, gpos0, out_base, tile_start + (u32)e, (u64)pe.x | ((u64)pe.y << 32), pe.z, pe.w);
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
      if (tid == 0) { argus_set_error(a.status, ARGUS_ERR_TIMEOUT, s, 0); tma_wait_all0(); }
      return;
    }
    if (!a.redo) {
      if (!stream_failed && tid < ch) argus_note_ambiguity(a, gpos0 + sm.cstack[cs][tid].idx, ARGUS_AMBIG_BEGIN_EOS, (u32)tid);
      if (tid == 0) a.counts[s] = n_int;
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
  if (tid == 0) tma_wait_all0();  // shared memory must outlive the last bulk store
}

template <int NT, int E>
int launch_tiled(const ArgusPairArgs& a, cudaStream_t stream) {
  static int grid_cache = 0;
  const size_t smem = sizeof(TileSmem<NT, E>) + 128;
  if (!grid_cache) {
    ARGUS_CUDA_TRY(cudaFuncSetAttribute(k_pair_tiled<NT, E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int dev = 0, sms = 0, per_sm = 0;
    ARGUS_CUDA_TRY(cudaGetDevice(&dev));
    ARGUS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ARGUS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pair_tiled<NT, E>, NT, smem));
    if (per_sm < 1) return ARGUS_ERR_CUDA;
    grid_cache = sms * per_sm;
  }
  const u32 grid = a.num_streams < (u32)grid_cache ? a.num_streams : (u32)grid_cache;
  k_pair_tiled<NT, E><<<grid, NT, smem, stream>>>(a);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

}  // namespace

bool argus_pair_tiled_usable(const ArgusPairArgs& a) { return a.num_streams > 0; }

int argus_launch_pair_tiled(const ArgusPairArgs& a, cudaStream_t stream) { return launch_tiled<256, 5>(a, stream); }
