// argus_synthesize.cu — the whole hot path in one call: pair -> aggregate -> overlap.
//
// Pairing writes, beside every 48-byte interval record, an 8-byte digest (region, both durations, a flag
// bit); then ONE pass over the digests both aggregates the intervals and selects the overlap spans (a pass
// over the records themselves reads six times the bytes). More than 400 regions or 128 pairs, or a call that
// asks for no table: the three plain calls. Results are identical in every mode. argus_synthesize_ring is the
// same pipeline on a ring container.
#include "argus_internal.cuh"

#include <atomic>

namespace {

std::atomic<int> g_synth_mode_knob{-1};  // -1 = automatic

struct SynLayout {
  size_t pair, pair_bytes, agg, agg_bytes, list_count, list_seg, list_spans, ov, ov_bytes, digest, total;
  uint64_t digest_capacity, list_capacity, list_slack;
  uint32_t list_chunk;
};

SynLayout syn_layout(uint64_t num_events, uint32_t num_streams, uint32_t num_regions, uint64_t ambig_capacity,
                     uint32_t num_pairs, uint32_t num_sms, uint64_t max_overlap_spans) {
  SynLayout L;
  size_t o = 0;
  L.pair = o; L.pair_bytes = argus_pair_workspace_bytes(num_events, num_streams, ambig_capacity); o += argus_align_up(L.pair_bytes, 256);
  L.agg = o; L.agg_bytes = argus_aggregate_workspace_bytes(num_events / 2, num_streams, num_regions); o += argus_align_up(L.agg_bytes, 256);
  // The span list: warps reserve slots in chunks and leave some unused, so the list is longer than the spans it
  // may hold, by a quarter or by one smallest chunk for every warp that can append, whichever is more
  // (the aggregation passes run at most one block of 8 warps per stream).
  const uint64_t warps = (uint64_t)num_streams * 8 > 1024 ? (uint64_t)num_streams * 8 : 1024;
  L.list_slack = num_pairs ? (max_overlap_spans / 4 > warps * 32 ? max_overlap_spans / 4 : warps * 32) : 0;
  L.list_chunk = 256;
  while (L.list_chunk > 32 && warps * L.list_chunk > L.list_slack) L.list_chunk >>= 1;
  L.list_capacity = max_overlap_spans + L.list_slack;
  L.list_count = o; o += 256;
  L.list_seg = o; o += argus_align_up((size_t)L.list_capacity * 4 + 4, 256);
  L.list_spans = o; o += argus_align_up((size_t)L.list_capacity * 16 + 16, 256);
  L.ov = o;
  // segment counters and the sorted spans (24 B each); a little more, so that the plain overlap call, which gets the
  // list's room and this as one workspace and splits it itself (50.7 B a span), also holds max_overlap_spans
  L.ov_bytes = argus_align_up((size_t)num_pairs * num_sms * 2 * 8 * 3 + 1024 + (size_t)max_overlap_spans * 27 + 4096, 256);
  o += L.ov_bytes;
  // one digest per interval (a stream's intervals start at half its first event's position at the latest)
  L.digest_capacity = argus_aggregate_can_select_overlap(num_regions, num_pairs) ? num_events / 2 + 1 : 0;
  L.digest = o; o += argus_align_up((size_t)L.digest_capacity * 8, 256);
  L.total = o;
  return L;
}

}  // namespace

// Where argus_synthesize aggregates and selects overlap spans: -1 automatic, 1 in one pass over the intervals'
// digests, 2 the plain calls, 3 in one pass over the interval records (test aid; results are identical).
extern "C" void argus_set_synthesize_mode(int mode) { g_synth_mode_knob.store(mode); }

extern "C" size_t argus_synthesize_workspace_bytes(uint64_t num_events, uint32_t num_streams, uint32_t num_regions,
                                                   uint64_t ambig_capacity, uint32_t num_pairs, uint32_t num_sms,
                                                   uint64_t max_overlap_spans) {
  return syn_layout(num_events, num_streams, num_regions, ambig_capacity, num_pairs, num_sms, max_overlap_spans).total;
}

// ring_written non-null: `events` is a ring container whose packed offsets are already in stream_offsets (device);
// num_events then bounds the surviving records and the status block has been cleared by the caller.
static int synthesize_impl(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                           uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                           uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                           uint64_t ambig_capacity, uint64_t* ambig_offsets, uint32_t warps_per_cta,
                           const uint32_t* cta_sm, uint32_t num_sms, argus_agg_t* warp_tab, argus_agg_t* cta_tab,
                           argus_agg_t* sm_tab, argus_agg_t* kernel_tab, const uint32_t* pairs, uint32_t num_pairs,
                           argus_overlap_t* overlap_out, uint64_t max_overlap_spans, argus_status_t* status,
                           void* workspace, size_t workspace_bytes, void* cuda_stream, const uint64_t* ring_written,
                           uint32_t ring_capacity) {
  if (!status || !workspace || ((uintptr_t)workspace & 255)) return ARGUS_ERR_INVALID_ARG;
  if (warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ARGUS_ERR_INVALID_ARG;
  if (num_regions == 0 || num_regions > ARGUS_MAX_REGIONS) return ARGUS_ERR_INVALID_ARG;
  if ((sm_tab || num_pairs) && ((!cta_sm && num_streams) || num_sms == 0)) return ARGUS_ERR_INVALID_ARG;
  if (num_pairs && (!pairs || !overlap_out)) return ARGUS_ERR_INVALID_ARG;
  const SynLayout L = syn_layout(num_events, num_streams, num_regions, ambig_capacity, num_pairs, num_sms, max_overlap_spans);
  if (workspace_bytes < L.total) return ARGUS_ERR_WORKSPACE;
  const int g_synth_mode = g_synth_mode_knob.load(std::memory_order_relaxed);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  const bool want_agg = warp_tab || cta_tab || sm_tab || kernel_tab;

  ArgusFuseArgs f;
  f.warp_tab = nullptr; f.cta_sm = cta_sm; f.warps_per_cta = warps_per_cta; f.num_sms = num_sms;
  f.pairs = pairs; f.num_pairs = num_pairs; f.ov_spans = nullptr; f.ov_seg = nullptr; f.ov_capacity = 0; f.ov_count = nullptr; f.ov_chunk = L.list_chunk;
  // where aggregation and overlap selection happen: 1 = in one pass over the intervals (their digests, or the
  // records themselves) after pairing, 2 = the plain calls
  const bool can_one_pass = num_streams > 0 && want_agg && argus_aggregate_can_select_overlap(num_regions, num_pairs);
  int mode = can_one_pass ? 1 : 2;
  if (g_synth_mode == 2) mode = 2;  // test aid: a forced mode applies when the inputs allow it
  const bool list = mode != 2 && num_pairs;
  if (list) {
    f.ov_spans = (ulonglong2*)(ws + L.list_spans);
    f.ov_seg = (u32*)(ws + L.list_seg);
    f.ov_capacity = L.list_capacity;
    f.ov_count = (u64*)(ws + L.list_count);
    ARGUS_CUDA_TRY(cudaMemsetAsync(ws + L.list_count, 0, 256, stream));
  }
  const bool use_digest = mode == 1 && L.digest_capacity != 0 && g_synth_mode != 3;
  int rc = argus_internal_pair(events, num_events, stream_offsets, num_streams, num_regions, intervals, interval_capacity,
                               interval_offsets, ambig, ambig_capacity, ambig_offsets, status, ws + L.pair, L.pair_bytes,
                               cuda_stream, ring_written ? 2 : 0, ring_written == nullptr,
                               use_digest ? (uint64_t*)(ws + L.digest) : nullptr, L.digest_capacity, ring_written, ring_capacity);
  if (rc != ARGUS_OK) return rc;

  if (want_agg) {
    rc = argus_internal_aggregate_scoped(intervals, interval_offsets, ambig, ambig_offsets, num_streams, warps_per_cta,
                                         cta_sm, num_sms, num_regions, nullptr, warp_tab, cta_tab, sm_tab, kernel_tab,
                                         nullptr, nullptr, status, ws + L.agg, L.agg_bytes, cuda_stream, false,
                                         mode == 1 && list ? &f : nullptr,
                                         use_digest ? (const uint64_t*)(ws + L.digest) : nullptr, interval_capacity);
    if (rc != ARGUS_OK) return rc;
  }
  if (num_pairs) {
    if (mode != 2) {
      rc = argus_internal_overlap_from_list(f.ov_spans, f.ov_seg, (const uint64_t*)f.ov_count, f.ov_capacity, num_sms, num_pairs, overlap_out,
                                            status, ws + L.ov, L.ov_bytes, cuda_stream);
    } else {
      rc = argus_internal_overlap(intervals, interval_capacity, interval_offsets, num_streams, warps_per_cta, cta_sm, num_sms,
                                  pairs, num_pairs, overlap_out, status, ws + L.list_count, L.ov + L.ov_bytes - L.list_count,
                                  cuda_stream, false);
    }
    if (rc != ARGUS_OK) return rc;
  }
  return ARGUS_OK;
}

extern "C" int argus_synthesize(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                                uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                                uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                                uint64_t ambig_capacity, uint64_t* ambig_offsets, uint32_t warps_per_cta,
                                const uint32_t* cta_sm, uint32_t num_sms, argus_agg_t* warp_tab, argus_agg_t* cta_tab,
                                argus_agg_t* sm_tab, argus_agg_t* kernel_tab, const uint32_t* pairs, uint32_t num_pairs,
                                argus_overlap_t* overlap_out, uint64_t max_overlap_spans, argus_status_t* status,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return synthesize_impl(events, num_events, stream_offsets, num_streams, num_regions, intervals, interval_capacity,
                         interval_offsets, ambig, ambig_capacity, ambig_offsets, warps_per_cta, cta_sm, num_sms, warp_tab, cta_tab,
                         sm_tab, kernel_tab, pairs, num_pairs, overlap_out, max_overlap_spans, status, workspace, workspace_bytes,
                         cuda_stream, nullptr, 0);
}

extern "C" int argus_synthesize_ring(const argus_event_t* ring, uint32_t slot_capacity, const uint64_t* written,
                                     uint32_t num_streams, uint32_t num_regions, uint64_t* stream_offsets, uint64_t* dropped,
                                     argus_interval_t* intervals, uint64_t interval_capacity, uint64_t* interval_offsets,
                                     argus_ambiguity_t* ambig, uint64_t ambig_capacity, uint64_t* ambig_offsets,
                                     uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, argus_agg_t* warp_tab,
                                     argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab, const uint32_t* pairs,
                                     uint32_t num_pairs, argus_overlap_t* overlap_out, uint64_t max_overlap_spans,
                                     argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!status || !stream_offsets || slot_capacity == 0) return ARGUS_ERR_INVALID_ARG;
  if (num_streams && (!ring || !written)) return ARGUS_ERR_INVALID_ARG;
  if (((uintptr_t)written & 7) || ((uintptr_t)dropped & 7) || ((uintptr_t)stream_offsets & 7)) return ARGUS_ERR_INVALID_ARG;
  ARGUS_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(argus_status_t), (cudaStream_t)cuda_stream));
  const uint64_t bound = (uint64_t)num_streams * slot_capacity;  // what the slots can hold: sizes the workspace
  const int rc = argus_internal_ring_offsets(written, slot_capacity, num_streams, bound, stream_offsets, dropped, status, cuda_stream);
  if (rc != ARGUS_OK) return rc;
  // without streams there is nothing to read from a ring: the plain path writes the empty results
  return synthesize_impl(ring, bound, stream_offsets, num_streams, num_regions, intervals, interval_capacity, interval_offsets,
                         ambig, ambig_capacity, ambig_offsets, warps_per_cta, cta_sm, num_sms, warp_tab, cta_tab, sm_tab,
                         kernel_tab, pairs, num_pairs, overlap_out, max_overlap_spans, status, workspace, workspace_bytes,
                         cuda_stream, num_streams ? written : nullptr, slot_capacity);
}
