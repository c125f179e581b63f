/*
 * oracle.h — record layouts and entry points of the CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY. This is a plain, slow, single-threaded restatement of what the
 * hot path computes, used by the tests, the smoke check and the CPU-baseline leg of the
 * benchmark. It shares no code with the CUDA library: the layouts below are retyped here
 * on purpose and nothing in the product may include or link this.
 *
 * Every function follows the sequential definition of the per-warp nested region context
 * stack (paper Section 3.2, "Region Semantics and Identity") and of scopes as selections
 * of executions (Section 3.2, "Region and scope"). All arithmetic is unsigned 64-bit.
 * Parity status: every function here is pinned by tests (hand-worked examples, brute-force
 * pairing enumeration, closed forms and invariants); nothing is "parity unpinned".
 */
#ifndef ORACLE_H_
#define ORACLE_H_
#include <cstddef>
#include <cstdint>

extern "C" {

struct OEvent { uint64_t ts; uint32_t tag; uint32_t ctx; };                     // 16 B
struct OInterval {                                                               // 48 B
  uint64_t t_begin, inclusive, exclusive;
  uint32_t region, ctx, stream, parent_region, begin_idx;
  uint16_t depth, flags;
};
struct OAmbig { uint64_t ts; uint32_t tag, ctx, stream, event_idx, kind, depth; };  // 32 B
struct OAgg {                                                                    // 576 B
  uint64_t count, sum_incl, min_incl, max_incl, sum_excl;
  uint64_t n_unmatched_begin, n_unmatched_end, n_flagged;
  uint64_t hist[64];
};
struct OOverlap { uint64_t overlap_ns, producer_ns, consumer_ns, either_ns; };   // 32 B
struct OStatus {                                                                 // 64 B
  uint32_t code, bad_stream;
  uint64_t bad_event, intervals_required, ambig_required;
  uint64_t n_ctx_mismatch, n_time_reversed, n_child_clamped, reserved;
};

// Step 1-3: stack matching, durations, ambiguity records. Host pointers throughout.
// Returns 0 or a host-detectable code; device-class conditions go to st->code, as the
// library does. interval_cap / ambig_cap: capacity of the output arrays in records.
int oracle_pair(const OEvent* events, const uint64_t* stream_offsets, uint32_t num_streams,
                uint32_t num_regions, OInterval* intervals, uint64_t interval_cap,
                uint64_t* interval_offsets, OAmbig* ambig, uint64_t ambig_cap,
                uint64_t* ambig_offsets, OStatus* st);

// Step 4: per-(region, scope) statistics. Any table may be null.
int oracle_aggregate(const OInterval* intervals, const uint64_t* interval_offsets,
                     const OAmbig* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                     uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                     uint32_t num_regions, OAgg* warp_tab, OAgg* cta_tab, OAgg* sm_tab,
                     OAgg* kernel_tab, OStatus* st);

// Step 4 (second half): per-SM overlap of producer/consumer region pairs.
int oracle_overlap(const OInterval* intervals, const uint64_t* interval_offsets,
                   uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm,
                   uint32_t num_sms, const uint32_t* pairs, uint32_t num_pairs, OOverlap* out,
                   OStatus* st);

// Scope selection (paper Section 1, the observe(region, signals, scope) query; Section 3.2
// "Region and scope"): which executions of a region count, chosen by iteration window
// (ctx_lo <= ctx <= ctx_hi), warp role (bit stream % warps_per_cta of warp_mask), SM subset
// (bit cta_sm[cta] of sm_mask) and region set (bit region of region_mask). Null masks select
// everything. Host pointers.
struct OScope {
  uint32_t ctx_lo, ctx_hi;
  uint64_t warp_mask;
  const uint32_t* sm_mask;
  const uint32_t* region_mask;
};

// oracle_aggregate over the selected intervals and ambiguity records only, plus role_tab[W][R]
// (key = stream % warps_per_cta) and iter_tab[ctx_hi - ctx_lo + 1][R] (key = ctx - ctx_lo).
// scope may be null (everything); iter_tab needs a scope.
int oracle_aggregate_scoped(const OInterval* intervals, const uint64_t* interval_offsets,
                            const OAmbig* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                            uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                            uint32_t num_regions, const OScope* scope, OAgg* warp_tab, OAgg* cta_tab,
                            OAgg* sm_tab, OAgg* kernel_tab, OAgg* role_tab, OAgg* iter_tab, OStatus* st);

// PC-to-region mapping (paper Section 3.2, the dynamic PC-to-region mapping figure): a mapping-run stream is a
// sequence of begin(region), end(region) and exec(pc, k) records; every exec credits k executions of that PC
// to the innermost region active at that point of the stream (row num_regions = outside every region). The
// stack follows the rules of oracle_pair (an end closes the innermost open frame of its region and drops the
// frames above it; an end without such a frame changes nothing; at most 64 open frames, an exec record
// counting as one more). counts is [(num_regions + 1)][num_pcs].
struct OMapEvent { uint32_t kind; uint32_t id; uint64_t count; };  // kind 0 begin, 1 end, 2 exec
int oracle_map_pc_counts(const OMapEvent* events, const uint64_t* stream_offsets, uint32_t num_streams,
                         uint32_t num_regions, uint32_t num_pcs, uint64_t* counts, OStatus* st);

// Ambiguity-aware attribution (paper Section 3.5): alpha[r][p] = n[r][p] / sum_r' n[r'][p],
// mhat[r] = sum_p alpha[r][p] * metric[p], entropy[p] = - sum_{alpha > 0} alpha ln alpha. fp64, plain loops.
// alpha may be null.
int oracle_attribute(const uint64_t* counts, uint32_t num_rows, uint32_t num_pcs, const double* metric,
                     double* mhat, double* entropy, double* alpha);

// Cross-run join (paper Sections 3.3 and 3.5: probe samples are joined to the reference run by region id and
// dynamic scope, not by timestamps; appendix: mean and 0/20/40/60/80th percentiles over repeated samples).
// Query q = reference[ref_index[q]]; its samples are all intervals of `samples` with the same
// (stream, region, ctx); values = their inclusive times, sorted; pct[j] = sorted[(j * count) / 5].
struct OJoin { uint64_t count, sum; uint64_t pct[5]; uint64_t max; };
int oracle_join_samples(const OInterval* reference, uint64_t num_reference, const uint64_t* ref_index,
                        uint32_t num_queries, const OInterval* samples, uint64_t num_samples, OJoin* out, OStatus* st);

// Ring-buffer container (one fixed slot of slot_capacity records per stream, record i at position
// i % slot_capacity, written[s] records ever written): the surviving records, oldest first, packed in CSR form.
// The paper fixes no container; this is the layout declared in the library's header.
int oracle_ring_linearise(const OEvent* ring, uint32_t slot_capacity, const uint64_t* written, uint32_t num_streams,
                          OEvent* events, uint64_t event_capacity, uint64_t* stream_offsets, uint64_t* dropped, OStatus* st);

// oracle_overlap over the selected intervals only.
int oracle_overlap_scoped(const OInterval* intervals, const uint64_t* interval_offsets,
                          uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm,
                          uint32_t num_sms, const uint32_t* pairs, uint32_t num_pairs,
                          const OScope* scope, OOverlap* out, OStatus* st);
}
#endif
