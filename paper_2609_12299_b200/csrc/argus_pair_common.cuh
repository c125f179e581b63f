// argus_pair_common.cuh — the sequential per-stream stack machine (exact semantics) and the
// ambiguity side channel used by every pairing kernel.
//
// Ambiguity records cannot be written in final order in one pass: whether a begin ends up
// force-closed or open at end of stream is only known later. The pairing kernels therefore
//   (1) append a packed note {global event position, kind, depth} to an unordered list, and
//   (2) set the event's bit in a bitmap over all events;
// afterwards a rank query on the bitmap (popcount prefix) gives every note its slot in
// (stream, event index) order, and stream_offsets give ambig_offsets.
#ifndef ARGUS_PAIR_COMMON_CUH_
#define ARGUS_PAIR_COMMON_CUH_

#include "argus_common.cuh"
#include "argus_fuse.cuh"

struct ArgusFrame {  // one open region occurrence, 32 bytes
  u64 ts;
  u64 child;  // inclusive time of matched intervals directly below
  u32 region;
  u32 ctx;
  u32 idx;  // index of the begin marker within its stream
  u32 pad;
};

struct ArgusPairCtl {  // control block in the workspace, zeroed at the start of a call
  u64 n_notes;         // ambiguity notes appended (may exceed the list capacity)
  u32 redo;            // 1 = provisional interval bases were wrong; second pass needed
  u32 spec_overflow;   // a provisional position fell outside interval_capacity
  u64 total_intervals;
  u64 total_ambig;
  // work queue of the tiled kernel, one set per pass (0 = first, 1 = redo): positions below num_streams are the
  // streams themselves, later positions are streams handed on after a chunk (see ArgusStreamRecord)
  u64 q_head[2];       // positions taken
  u64 q_tail[2];       // hand-overs published (queue entries written)
  u32 n_records[2];    // hand-over records allocated
  u32 n_done[2];       // streams walked to their end (or given up on)
  u64 reserved[2];
};

// A long stream is walked in chunks of about kChunkEvents events. After a chunk the CTA stores the stream's
// state here and puts the record into the work queue, so that whichever CTA is free next carries on: all
// streams advance at the same pace and the kernel has no long tail, whatever the number of streams per SM.
// Queue positions are taken with one atomic add each. A CTA whose position has no entry yet is idle anyway
// (every unfinished stream is in some CTA's hands): it polls until the entry appears or every stream is
// done, and gives up with ARGUS_ERR_TIMEOUT if no hand-over at all is published for about a second.
constexpr u32 kChunkEvents = 32768;
struct ArgusStreamRecord {
  u32 stream, next_tile;
  int ch;                             // stack height at the hand-over
  u32 pad;
  u64 n_int;                          // intervals emitted so far
  uint4 frames[ARGUS_MAX_DEPTH];      // open begin markers as event records
  u64 child[ARGUS_MAX_DEPTH];         // their child time so far
  u32 idx[ARGUS_MAX_DEPTH];           // their index within the stream
};

struct ArgusPairArgs {
  const argus_event_t* events;
  const u64* stream_offsets;
  u64 num_events;
  u32 num_streams;
  u32 num_regions;
  argus_interval_t* intervals;
  u64 interval_capacity;
  u64* interval_offsets;  // final offsets (output of the offsets kernel)
  u64* counts;            // per-stream interval counts (workspace)
  u64* notes;             // packed ambiguity notes (workspace)
  u64 note_capacity;
  u32* bits;              // one bit per event (workspace)
  ArgusPairCtl* ctl;
  argus_status_t* status;
  int redo;               // 0 = first pass with provisional bases, 1 = second pass with final bases
  u32* queue;             // hand-over queue entries (record index + 1; zeroed), null = streams are never split
  u64 queue_capacity;
  ArgusStreamRecord* records;
  u32 record_capacity;
  const u32* order;       // streams in the order in which the tiled kernel starts them: longest first (null = by index)
  u64* digest;            // one digest per interval record, same positions (null = none); holds every position below
                          // min(interval_capacity, num_events / 2 + 1), which is all a stream can reach
  const u64* ring_written; // non-null: `events` is a ring container, one slot of ring_capacity records per stream, record i of
  u32 ring_capacity;       // a stream at slot position i mod capacity; stream_offsets then describe the packed survivors
  u32 poll_limit;          // polls without any hand-over anywhere after which an idle CTA gives up (about a second)
};

#define ARGUS_NOTE_POS_BITS 48

// Ring container: slot position of the oldest surviving record of stream s.
__device__ __forceinline__ u32 argus_ring_first(const ArgusPairArgs& a, u32 s) {
  const u64 w = a.ring_written[s];
  return w > a.ring_capacity ? (u32)(w % a.ring_capacity) : 0u;
}

__device__ __forceinline__ void argus_note_ambiguity(const ArgusPairArgs& a, u64 gpos, u32 kind, u32 depth) {
  const u64 slot = atomicAdd(&a.ctl->n_notes, 1ull);
  if (slot < a.note_capacity) a.notes[slot] = gpos | ((u64)kind << ARGUS_NOTE_POS_BITS) | ((u64)depth << (ARGUS_NOTE_POS_BITS + 2));
  atomicOr(&a.bits[gpos >> 5], 1u << (gpos & 31));
}

__device__ __forceinline__ void argus_store_interval(argus_interval_t* dst, u64 t_begin, u64 incl, u64 excl, u32 region,
                                                     u32 ctx, u32 stream, u32 parent, u32 begin_idx, u32 depth, u32 flags) {
  uint4* p = reinterpret_cast<uint4*>(dst);
  p[0] = make_uint4((u32)t_begin, (u32)(t_begin >> 32), (u32)incl, (u32)(incl >> 32));
  p[1] = make_uint4((u32)excl, (u32)(excl >> 32), region, ctx);
  p[2] = make_uint4(stream, parent, begin_idx, (depth & 0xffffu) | (flags << 16));
}

// Per-stream running state of the sequential machine.
struct ArgusSeqState {
  int h;            // stack height
  u64 n_int;        // intervals emitted so far in this stream
  u32 n_ctx, n_rev, n_clamp;  // flag counters (flushed by the caller)
  bool failed;
};

// Processes one event exactly as the definition states. `stk` holds ARGUS_MAX_DEPTH frames.
// `out_base` is the position of this stream's first interval. Returns false on a device error.
__device__ __forceinline__ bool argus_seq_step(const ArgusPairArgs& a, ArgusFrame* stk, ArgusSeqState& s, u32 stream,
                                               u64 stream_gpos0, u64 out_base, u32 i, u64 ts, u32 tag, u32 ctx) {
  const u32 region = tag >> 1;
  if (region >= a.num_regions) {
    argus_set_error(a.status, ARGUS_ERR_BAD_REGION, stream, i);
    return false;
  }
  if (!(tag & 1u)) {
    if (s.h == ARGUS_MAX_DEPTH) {
      argus_set_error(a.status, ARGUS_ERR_DEPTH, stream, i);
      return false;
    }
    ArgusFrame& f = stk[s.h++];
    f.ts = ts; f.child = 0; f.region = region; f.ctx = ctx; f.idx = i;
    return true;
  }
  int k = s.h - 1;
  while (k >= 0 && stk[k].region != region) --k;
  if (k < 0) {
    if (!a.redo) argus_note_ambiguity(a, stream_gpos0 + i, ARGUS_AMBIG_UNMATCHED_END, (u32)s.h);
    return true;
  }
  u64 moved = 0;
  while (s.h - 1 > k) {  // force-close mis-nested frames; their child time moves down the stack
    const ArgusFrame& f = stk[--s.h];
    if (!a.redo) argus_note_ambiguity(a, stream_gpos0 + f.idx, ARGUS_AMBIG_BEGIN_MISNESTED, (u32)s.h);
    moved += f.child;
  }
  const ArgusFrame f = stk[--s.h];
  const u64 child = f.child + moved;
  u32 flags = 0;
  u64 incl, excl;
  if (ctx != f.ctx) { flags |= ARGUS_FLAG_CTX_MISMATCH; s.n_ctx++; }
  if (ts < f.ts) { incl = 0; flags |= ARGUS_FLAG_TIME_REVERSED; s.n_rev++; } else { incl = ts - f.ts; }
  if (child > incl) { excl = 0; flags |= ARGUS_FLAG_CHILD_CLAMPED; s.n_clamp++; } else { excl = incl - child; }
  const u64 pos = out_base + s.n_int;
  if (pos < a.interval_capacity) {
    argus_store_interval(a.intervals + pos, f.ts, incl, excl, f.region, f.ctx, stream,
                         s.h > 0 ? stk[s.h - 1].region : ARGUS_NONE, f.idx, (u32)s.h, flags);
    if (a.digest) a.digest[pos] = argus_digest_pack(f.region, incl, excl, flags);
  } else if (!a.redo) {
    a.ctl->spec_overflow = 1;
  }
  s.n_int++;
  if (s.h > 0) stk[s.h - 1].child += incl;
  return true;
}

// End of stream: every open frame becomes a BEGIN_EOS note.
__device__ __forceinline__ void argus_seq_finish(const ArgusPairArgs& a, const ArgusFrame* stk, const ArgusSeqState& s,
                                                 u64 stream_gpos0) {
  if (a.redo) return;
  for (int k = 0; k < s.h; ++k) argus_note_ambiguity(a, stream_gpos0 + stk[k].idx, ARGUS_AMBIG_BEGIN_EOS, (u32)k);
}

__device__ __forceinline__ void argus_flush_flag_counters(const ArgusPairArgs& a, const ArgusSeqState& s) {
  if (a.redo) return;
  if (s.n_ctx) atomicAdd((u64*)&a.status->n_ctx_mismatch, (u64)s.n_ctx);
  if (s.n_rev) atomicAdd((u64*)&a.status->n_time_reversed, (u64)s.n_rev);
  if (s.n_clamp) atomicAdd((u64*)&a.status->n_child_clamped, (u64)s.n_clamp);
}

#endif  // ARGUS_PAIR_COMMON_CUH_
