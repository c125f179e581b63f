// argus_pair.cu — argus_pair_intervals: marker events -> nested intervals + ambiguity records.
//
// Pipeline enqueued on the caller's stream (no host synchronisation):
//   memset(control block, event bitmap)
//   pair pass 1   : intervals written at provisional bases floor((off[s]-off[0])/2), exact for
//                   well-formed traces; per-stream counts; ambiguity notes + bitmap bits
//   offsets       : scan of counts -> interval_offsets; sets `redo` when a base was provisional-wrong
//   pair pass 2   : only does work when `redo` is set (malformed traces): rewrites intervals at the
//                   final bases
//   ambiguity     : popcount prefix over the bitmap -> rank of every note -> ordered records, offsets
#include "argus_internal.cuh"
#include "argus_pair_common.cuh"

#include <string.h>

#include <atomic>

namespace {

constexpr int kScanThreads = 1024;
constexpr u32 kWordsPerBlock = 1024;  // bitmap words per prefix block (32768 events)
std::atomic<u32> g_poll_limit{1u << 19};  // see argus_testing_set_poll_limit

// ---------------------------------------------------------------------------------------------
// Reference-order kernel: one thread walks one stream with its stack in local memory.
// Exact for any input; used for small traces and as the arbiter the tiled kernel falls back to.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_pair_thread_per_stream(ArgusPairArgs a) {
  const u32 s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= a.num_streams) return;
  if (a.redo && !a.ctl->redo) return;
  const u64 off0 = a.stream_offsets[0];
  const u64 lo = a.stream_offsets[s], hi = a.stream_offsets[s + 1];
  if (hi < lo || hi > a.num_events || lo < off0 || (hi - lo) >> 32) {
    argus_set_error(a.status, ARGUS_ERR_BAD_OFFSETS, s, 0);
    if (!a.redo) a.counts[s] = 0;
    return;
  }
  const u64 base = a.redo ? a.interval_offsets[s] : ((lo - off0) >> 1);
  // second pass: intervals that already lie where they belong (same position, all of them fitted) stay
  if (a.redo && base == ((lo - off0) >> 1) && base + a.counts[s] <= a.interval_capacity) return;
  ArgusFrame stk[ARGUS_MAX_DEPTH];
  ArgusSeqState st;
  st.h = 0; st.n_int = 0; st.n_ctx = st.n_rev = st.n_clamp = 0; st.failed = false;
  const u32 n = (u32)(hi - lo);
  const uint4* ev = reinterpret_cast<const uint4*>(a.events + lo);
  bool ok = true;
  for (u32 i = 0; i < n && ok; ++i) {
    const uint4 e = __ldg(ev + i);
    ok = argus_seq_step(a, stk, st, s, lo - off0, base, i, (u64)e.x | ((u64)e.y << 32), e.z, e.w);
  }
  if (ok) argus_seq_finish(a, stk, st, lo - off0);
  argus_flush_flag_counters(a, st);
  if (!a.redo) a.counts[s] = st.n_int;
}

// ---------------------------------------------------------------------------------------------
// order: streams sorted by length class (floor(log2(events))), longest first. A stream is a chain of chunks that
// one CTA at a time walks, so when lengths differ (producer and consumer warps of one kernel) the long chains must
// start first or they end last, alone. Counting sort in one block; the order inside a class does not matter.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kScanThreads) k_pair_order(ArgusPairArgs a, u32* order) {
  __shared__ u32 cnt[64], cur[64];
  __shared__ u32 one_class;
  if (threadIdx.x < 64) { cnt[threadIdx.x] = 0; cur[threadIdx.x] = 0; }
  __syncthreads();
  for (u32 s = threadIdx.x; s < a.num_streams; s += blockDim.x) {
    const u64 lo = a.stream_offsets[s], hi = a.stream_offsets[s + 1];
    const u64 n = hi > lo ? hi - lo : 0;
    atomicAdd(&cnt[n ? 63 - __clzll((long long)n) : 0], 1u);
  }
  __syncthreads();
  if (threadIdx.x == 0) {  // bases, classes in descending order
    u32 base = 0;
    one_class = 0;
    for (int c = 63; c >= 0; --c) {
      const u32 k = cnt[c];
      if (k == a.num_streams) one_class = 1;
      cnt[c] = base;
      base += k;
    }
  }
  __syncthreads();
  if (one_class) {  // streams of one length class start in index order, as without this kernel
    for (u32 s = threadIdx.x; s < a.num_streams; s += blockDim.x) order[s] = s;
    return;
  }
  for (u32 s = threadIdx.x; s < a.num_streams; s += blockDim.x) {
    const u64 lo = a.stream_offsets[s], hi = a.stream_offsets[s + 1];
    const u64 n = hi > lo ? hi - lo : 0;
    const u32 c = n ? 63 - __clzll((long long)n) : 0;
    order[cnt[c] + atomicAdd(&cur[c], 1u)] = s;
  }
}

// ---------------------------------------------------------------------------------------------
// offsets: exclusive scan of per-stream counts; decides whether the second pass is needed.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kScanThreads) k_pair_offsets(ArgusPairArgs a) {
  __shared__ u64 sh[33];
  __shared__ u32 mismatch;
  if (threadIdx.x == 0) mismatch = 0;
  __syncthreads();
  const u64 off0 = a.num_streams ? a.stream_offsets[0] : 0;
  u64 carry = 0;
  for (u32 s0 = 0; s0 < a.num_streams; s0 += kScanThreads) {
    const u32 s = s0 + threadIdx.x;
    const u64 c = s < a.num_streams ? a.counts[s] : 0;
    u64 total;
    const u64 ex = argus_block_exclusive_scan<u64>(c, sh, &total);
    if (s < a.num_streams) {
      const u64 fin = carry + ex;
      // (beyond the capacity only when the call ends with ARGUS_ERR_CAPACITY: offsets then stay inside the array, so
      // that a call chained behind this one without a host check reads nothing it must not)
      a.interval_offsets[s] = fin < a.interval_capacity ? fin : a.interval_capacity;
      const u64 lo = a.stream_offsets[s];
      if (lo >= off0 && fin != ((lo - off0) >> 1) && c != 0) mismatch = 1;
    }
    carry += total;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    a.interval_offsets[a.num_streams] = carry < a.interval_capacity ? carry : a.interval_capacity;
    a.ctl->total_intervals = carry;
    a.status->intervals_required = carry;
    if (carry > a.interval_capacity) {
      argus_set_error(a.status, ARGUS_ERR_CAPACITY, 0, carry);
      a.ctl->redo = 0;
    } else {
      a.ctl->redo = (mismatch || a.ctl->spec_overflow) ? 1u : 0u;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// ambiguity ordering
// ---------------------------------------------------------------------------------------------
struct AmbigArgs {
  ArgusPairArgs p;
  u64 num_words;     // bitmap words covering [0, span) event positions
  u64 span;          // stream_offsets[S] - stream_offsets[0] is <= num_events; bitmap covers num_events
  u32* word_prefix;  // per word: set bits before it within its block
  u64* block_prefix; // per block: set bits before it (after the scan); [num_blocks + 1]
  u64 num_blocks;
  argus_ambiguity_t* ambig;
  u64 ambig_capacity;
  u64* ambig_offsets;
};

// (a fixed grid walks the blocks of words: a trace without ambiguous markers, the usual case, costs one small launch)
__global__ void __launch_bounds__(kWordsPerBlock) k_ambig_word_prefix(AmbigArgs g) {
  __shared__ u32 sh[33];
  if (g.p.ctl->n_notes == 0) return;
  for (u64 blk = blockIdx.x; blk < g.num_blocks; blk += gridDim.x) {
    const u64 w = blk * kWordsPerBlock + threadIdx.x;
    const u32 c = w < g.num_words ? __popc(g.p.bits[w]) : 0u;
    u32 total;
    const u32 ex = argus_block_exclusive_scan<u32>(c, sh, &total);
    if (w < g.num_words) g.word_prefix[w] = ex;
    if (threadIdx.x == 0) g.block_prefix[blk] = total;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kScanThreads) k_ambig_block_scan(AmbigArgs g) {
  __shared__ u64 sh[33];
  u64 carry = 0;
  if (g.p.ctl->n_notes != 0) {
    for (u64 b0 = 0; b0 < g.num_blocks; b0 += kScanThreads) {
      const u64 b = b0 + threadIdx.x;
      const u64 c = b < g.num_blocks ? g.block_prefix[b] : 0;
      u64 total;
      const u64 ex = argus_block_exclusive_scan<u64>(c, sh, &total);
      if (b < g.num_blocks) g.block_prefix[b] = carry + ex;
      carry += total;
    }
  }
  if (threadIdx.x == 0) {
    g.block_prefix[g.num_blocks] = carry;
    g.p.ctl->total_ambig = carry;
    g.p.status->ambig_required = carry;
    if (carry > g.ambig_capacity || g.p.ctl->n_notes > g.p.note_capacity)
      argus_set_error(g.p.status, ARGUS_ERR_CAPACITY, 0, carry);
  }
}

// number of ambiguous markers at global positions < gpos
__device__ __forceinline__ u64 ambig_rank(const AmbigArgs& g, u64 gpos) {
  const u64 w = gpos >> 5;
  if (w >= g.num_words) return g.block_prefix[g.num_blocks];
  return g.block_prefix[w / kWordsPerBlock] + g.word_prefix[w] + __popc(g.p.bits[w] & ((1u << (gpos & 31)) - 1u));
}

__global__ void __launch_bounds__(256) k_ambig_scatter(AmbigArgs g) {
  const u64 n_notes = g.p.ctl->n_notes;
  const u64 n = n_notes < g.p.note_capacity ? n_notes : g.p.note_capacity;
  const u64 off0 = g.p.stream_offsets[0];
  for (u64 j = (u64)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (u64)gridDim.x * blockDim.x) {
    const u64 note = g.p.notes[j];
    const u64 gpos = note & ((1ull << ARGUS_NOTE_POS_BITS) - 1);
    const u64 r = ambig_rank(g, gpos);
    if (r >= g.ambig_capacity) continue;
    const u64 x = off0 + gpos;  // index into events
    // stream = last s with stream_offsets[s] <= x (empty streams skipped by taking the upper bound)
    u32 lo = 0, hi = g.p.num_streams;
    while (hi - lo > 1) {
      const u32 mid = lo + ((hi - lo) >> 1);
      if (g.p.stream_offsets[mid] <= x) lo = mid; else hi = mid;
    }
    u64 at = x;  // where the record lies: packed input, or its slot position in a ring container
    if (g.p.ring_written) {
      u64 pos = argus_ring_first(g.p, lo) + (x - g.p.stream_offsets[lo]);
      if (pos >= g.p.ring_capacity) pos -= g.p.ring_capacity;
      at = (u64)lo * g.p.ring_capacity + pos;
    }
    const argus_event_t e = g.p.events[at];
    argus_ambiguity_t rec;
    rec.ts = e.ts; rec.tag = e.tag; rec.ctx = e.ctx; rec.stream = lo;
    rec.event_idx = (u32)(x - g.p.stream_offsets[lo]);
    rec.kind = (u32)(note >> ARGUS_NOTE_POS_BITS) & 3u;
    rec.depth = (u32)(note >> (ARGUS_NOTE_POS_BITS + 2)) & 0x7fu;
    g.ambig[r] = rec;
  }
}

__global__ void __launch_bounds__(256) k_ambig_offsets(AmbigArgs g) {
  const u64 s = (u64)blockIdx.x * blockDim.x + threadIdx.x;
  if (s > g.p.num_streams) return;
  if (g.p.ctl->n_notes == 0) { g.ambig_offsets[s] = 0; return; }
  const u64 off0 = g.p.stream_offsets[0];
  const u64 o = g.p.stream_offsets[s];
  const u64 r = o >= off0 ? ambig_rank(g, o - off0) : 0;
  g.ambig_offsets[s] = r < g.ambig_capacity ? r : g.ambig_capacity;  // inside the array also after ARGUS_ERR_CAPACITY
}

struct Layout {
  size_t ctl, counts, queue, bits, word_prefix, block_prefix, notes, records, order, total;
  u64 num_words, num_blocks, queue_capacity;
  u32 record_capacity;
};

Layout make_layout(uint64_t num_events, uint32_t num_streams, uint64_t ambig_capacity) {
  Layout L;
  L.num_words = (num_events + 31) / 32;
  L.num_blocks = (L.num_words + kWordsPerBlock - 1) / kWordsPerBlock;
  size_t o = 0;
  L.ctl = o; o += argus_align_up(sizeof(ArgusPairCtl), 256);
  L.counts = o; o += argus_align_up(((size_t)num_streams + 1) * 8, 256);
  // every hand-over follows a chunk of at least kChunkEvents events, and only streams longer than that hand over
  L.queue_capacity = num_events / kChunkEvents + 1;
  L.record_capacity = (u32)(L.queue_capacity < num_streams ? L.queue_capacity : num_streams);
  L.queue = o; o += argus_align_up((size_t)L.queue_capacity * 4, 256);
  L.bits = o; o += argus_align_up((size_t)L.num_words * 4 + 4, 256);
  L.word_prefix = o; o += argus_align_up((size_t)L.num_words * 4 + 4, 256);
  L.block_prefix = o; o += argus_align_up(((size_t)L.num_blocks + 1) * 8, 256);
  L.notes = o; o += argus_align_up((size_t)ambig_capacity * 8 + 8, 256);
  L.records = o; o += argus_align_up((size_t)L.record_capacity * sizeof(ArgusStreamRecord), 256);
  L.order = o; o += argus_align_up((size_t)num_streams * 4 + 4, 256);
  L.total = o;
  return L;
}

}  // namespace

// implemented in argus_pair_tiled.cu
int argus_launch_pair_tiled(const ArgusPairArgs& a, cudaStream_t stream);
bool argus_pair_tiled_usable(const ArgusPairArgs& a);

extern "C" void argus_testing_set_poll_limit(unsigned int polls) { g_poll_limit.store(polls ? polls : 1u << 19); }

extern "C" size_t argus_pair_workspace_bytes(uint64_t num_events, uint32_t num_streams, uint64_t ambig_capacity) {
  return make_layout(num_events, num_streams, ambig_capacity).total;
}

// Whole pairing pipeline. kernel_choice: 0 = automatic, 1 = one thread per stream, 2 = tiled.
int argus_internal_pair(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                        uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                        uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                        uint64_t ambig_capacity, uint64_t* ambig_offsets, argus_status_t* status, void* workspace,
                        size_t workspace_bytes, void* cuda_stream, int kernel_choice, bool reset_status,
                        uint64_t* digest, uint64_t digest_capacity,
                        const uint64_t* ring_written, uint32_t ring_capacity) {
  if (!stream_offsets || !interval_offsets || !ambig_offsets || !status || !workspace) return ARGUS_ERR_INVALID_ARG;
  if ((num_events && !events) || (interval_capacity && !intervals) || (ambig_capacity && !ambig)) return ARGUS_ERR_INVALID_ARG;
  if (num_regions == 0 || num_regions > ARGUS_MAX_REGIONS) return ARGUS_ERR_INVALID_ARG;
  if (num_events >> ARGUS_NOTE_POS_BITS) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)events & 15) || ((uintptr_t)intervals & 15) || ((uintptr_t)ambig & 15) || ((uintptr_t)status & 7) ||
      ((uintptr_t)workspace & 255) || ((uintptr_t)stream_offsets & 7) || ((uintptr_t)interval_offsets & 7) ||
      ((uintptr_t)ambig_offsets & 7))
    return ARGUS_ERR_INVALID_ARG;
  const Layout L = make_layout(num_events, num_streams, ambig_capacity);
  if (workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;

  ArgusPairArgs a;
  a.events = events; a.stream_offsets = (const u64*)stream_offsets; a.num_events = num_events;
  a.num_streams = num_streams; a.num_regions = num_regions;
  a.intervals = intervals; a.interval_capacity = interval_capacity; a.interval_offsets = (u64*)interval_offsets;
  a.counts = (u64*)(ws + L.counts);
  a.notes = (u64*)(ws + L.notes); a.note_capacity = ambig_capacity;
  a.bits = (u32*)(ws + L.bits);
  a.ctl = (ArgusPairCtl*)(ws + L.ctl);
  a.status = status;
  a.redo = 0;
  a.queue = (u32*)(ws + L.queue); a.queue_capacity = L.queue_capacity;
  a.records = (ArgusStreamRecord*)(ws + L.records); a.record_capacity = L.record_capacity;
  a.poll_limit = g_poll_limit.load(std::memory_order_relaxed);
  a.ring_written = (const u64*)ring_written; a.ring_capacity = ring_capacity;
  if (ring_written && (ring_capacity == 0 || kernel_choice == 1)) return ARGUS_ERR_INVALID_ARG;  // only the tiled kernel reads rings
  // a stream's intervals start at half its first event's position at the latest, so positions stay below num_events / 2 + 1
  a.digest = digest_capacity >= (interval_capacity < num_events / 2 + 1 ? interval_capacity : num_events / 2 + 1) ? (u64*)digest : nullptr;

  if (reset_status) ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  // control block, counts and bitmap are contiguous at the start of the workspace
  ARGUS_CUDA_TRY(cudaMemsetAsync(ws, 0, L.word_prefix, stream));

  const bool tiled = (kernel_choice != 1 && argus_pair_tiled_usable(a)) || ring_written != nullptr;
  a.order = nullptr;
  if (tiled && num_streams > 1) {
    k_pair_order<<<1, kScanThreads, 0, stream>>>(a, (u32*)(ws + L.order));
    ARGUS_CHECK_LAUNCH();
    a.order = (const u32*)(ws + L.order);
  }
  for (int pass = 0; pass < 2; ++pass) {
    a.redo = pass;
    if (num_streams) {
      if (pass == 0) argus_prof_mark(ARGUS_PROF_PAIR, stream, 0);
      if (tiled) {
        const int rc = argus_launch_pair_tiled(a, stream);
        if (rc != ARGUS_OK) return rc;
      } else {
        k_pair_thread_per_stream<<<(num_streams + 127) / 128, 128, 0, stream>>>(a);
        ARGUS_CHECK_LAUNCH();
      }
      if (pass == 0) argus_prof_mark(ARGUS_PROF_PAIR, stream, 1);
    }
    if (pass == 0) {
      k_pair_offsets<<<1, kScanThreads, 0, stream>>>(a);
      ARGUS_CHECK_LAUNCH();
    }
  }

  AmbigArgs g;
  g.p = a; g.num_words = L.num_words; g.span = num_events;
  g.word_prefix = (u32*)(ws + L.word_prefix); g.block_prefix = (u64*)(ws + L.block_prefix);
  g.num_blocks = L.num_blocks; g.ambig = ambig; g.ambig_capacity = ambig_capacity; g.ambig_offsets = (u64*)ambig_offsets;
  if (L.num_blocks) {
    k_ambig_word_prefix<<<(unsigned)(L.num_blocks < 2368 ? L.num_blocks : 2368), kWordsPerBlock, 0, stream>>>(g);
    ARGUS_CHECK_LAUNCH();
  }
  k_ambig_block_scan<<<1, kScanThreads, 0, stream>>>(g);
  ARGUS_CHECK_LAUNCH();
  if (num_streams && num_events) {
    k_ambig_scatter<<<296, 256, 0, stream>>>(g);
    ARGUS_CHECK_LAUNCH();
  }
  k_ambig_offsets<<<(num_streams + 1 + 255) / 256, 256, 0, stream>>>(g);
  ARGUS_CHECK_LAUNCH();
  return ARGUS_OK;
}

extern "C" int argus_pair_intervals_ex(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                                       uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                                       uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                                       uint64_t ambig_capacity, uint64_t* ambig_offsets, argus_status_t* status,
                                       void* workspace, size_t workspace_bytes, void* cuda_stream, int kernel_choice) {
  return argus_internal_pair(events, num_events, stream_offsets, num_streams, num_regions, intervals, interval_capacity,
                             interval_offsets, ambig, ambig_capacity, ambig_offsets, status, workspace, workspace_bytes,
                             cuda_stream, kernel_choice, true);
}

extern "C" int argus_pair_intervals(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                                    uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                                    uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                                    uint64_t ambig_capacity, uint64_t* ambig_offsets, argus_status_t* status,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return argus_pair_intervals_ex(events, num_events, stream_offsets, num_streams, num_regions, intervals,
                                 interval_capacity, interval_offsets, ambig, ambig_capacity, ambig_offsets, status,
                                 workspace, workspace_bytes, cuda_stream, 0);
}

extern "C" int argus_pair_intervals_ring(const argus_event_t* ring, uint32_t slot_capacity, const uint64_t* written,
                                         uint32_t num_streams, uint32_t num_regions, uint64_t* stream_offsets,
                                         uint64_t* dropped, argus_interval_t* intervals, uint64_t interval_capacity,
                                         uint64_t* interval_offsets, argus_ambiguity_t* ambig, uint64_t ambig_capacity,
                                         uint64_t* ambig_offsets, argus_status_t* status, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  if (!status || !stream_offsets || slot_capacity == 0) return ARGUS_ERR_INVALID_ARG;
  if (num_streams && (!ring || !written)) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)written & 7) || ((uintptr_t)dropped & 7)) return ARGUS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), stream));
  const uint64_t bound = (uint64_t)num_streams * slot_capacity;  // what the slots can hold: sizes the workspace
  int rc = argus_internal_ring_offsets(written, slot_capacity, num_streams, bound, stream_offsets, dropped, status, cuda_stream);
  if (rc != ARGUS_OK) return rc;
  return argus_internal_pair(ring, bound, stream_offsets, num_streams, num_regions, intervals, interval_capacity, interval_offsets,
                             ambig, ambig_capacity, ambig_offsets, status, workspace, workspace_bytes, cuda_stream, 2, false,
                             nullptr, 0, written, slot_capacity);
}
