// argus_internal.cuh — functions one translation unit of the library offers to the others (not part of the C-ABI).
#ifndef ARGUS_INTERNAL_CUH_
#define ARGUS_INTERNAL_CUH_

#include "argus_fuse.cuh"

// argus_pair.cu — the whole pairing pipeline. kernel_choice: 0 = automatic, 1 = one thread per stream, 2 = tiled.
// `digest` (nullable): one 8-byte digest per interval record, at the record's position (see argus_fuse.cuh).
// `ring_written` (nullable): `events` is a ring container (one slot of ring_capacity records per stream, written[s] records
// ever written); stream_offsets describe the packed survivors and num_events bounds them. Tiled kernel only.
int argus_internal_pair(const argus_event_t* events, uint64_t num_events, const uint64_t* stream_offsets,
                        uint32_t num_streams, uint32_t num_regions, argus_interval_t* intervals,
                        uint64_t interval_capacity, uint64_t* interval_offsets, argus_ambiguity_t* ambig,
                        uint64_t ambig_capacity, uint64_t* ambig_offsets, argus_status_t* status, void* workspace,
                        size_t workspace_bytes, void* cuda_stream, int kernel_choice, bool reset_status,
                        uint64_t* digest = nullptr, uint64_t digest_capacity = 0,
                        const uint64_t* ring_written = nullptr, uint32_t ring_capacity = 0);

// argus_aggregate.cu
int argus_internal_aggregate(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                             const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                             uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                             argus_agg_t* warp_tab, argus_agg_t* cta_tab, argus_agg_t* sm_tab, argus_agg_t* kernel_tab,
                             argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream,
                             bool reset_status, uint64_t interval_limit = ~0ull);
// scope, role_tab, iter_tab nullable; ov_select (nullable): also append the overlap spans of the selected intervals;
// digest (nullable; needs no scope, no role or iteration table, at most 400 regions): the intervals' digests, read instead of the records;
// interval_limit: records the interval array holds (a stream whose offsets reach beyond it is reported as ARGUS_ERR_BAD_OFFSETS, not read)
int argus_internal_aggregate_scoped(const argus_interval_t* intervals, const uint64_t* interval_offsets,
                                    const argus_ambiguity_t* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                                    uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms, uint32_t num_regions,
                                    const argus_scope_t* scope, argus_agg_t* warp_tab, argus_agg_t* cta_tab,
                                    argus_agg_t* sm_tab, argus_agg_t* kernel_tab, argus_agg_t* role_tab,
                                    argus_agg_t* iter_tab, argus_status_t* status, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream, bool reset_status,
                                    const ArgusFuseArgs* ov_select, const uint64_t* digest = nullptr,
                                    uint64_t interval_limit = ~0ull);
bool argus_aggregate_can_select_overlap(uint32_t num_regions, uint32_t num_pairs);

// argus_ring.cu — stream_offsets (and dropped) of the records that survive in the slots of a ring container;
// status->code = ARGUS_ERR_CAPACITY if they exceed event_capacity. The status block is not cleared.
int argus_internal_ring_offsets(const uint64_t* written, uint32_t slot_capacity, uint32_t num_streams, uint64_t event_capacity,
                                uint64_t* stream_offsets, uint64_t* dropped, argus_status_t* status, void* cuda_stream);

// argus_overlap.cu
int argus_internal_overlap(const argus_interval_t* intervals, uint64_t max_intervals, const uint64_t* interval_offsets,
                           uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                           const uint32_t* pairs, uint32_t num_pairs, argus_overlap_t* out, argus_status_t* status,
                           void* workspace, size_t workspace_bytes, void* cuda_stream, bool reset_status);
// overlap from a list of selected spans (spans + segment of each; *list_count slots reserved, unused ones tagged 0xffffffff)
int argus_internal_overlap_from_list(const void* list_spans, const uint32_t* list_seg, const uint64_t* list_count,
                                     uint64_t list_capacity, uint32_t num_sms, uint32_t num_pairs, argus_overlap_t* out,
                                     argus_status_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

#endif  // ARGUS_INTERNAL_CUH_
