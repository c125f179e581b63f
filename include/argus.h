/*
 * argus.h — C-ABI of the region-trace synthesis hot path for NVIDIA B200 (sm_100a).
 *
 * The library turns raw per-(CTA, warp) begin/end region-marker event buffers into
 * nested, attributed region intervals, attribution-ambiguity records, per-(region,
 * execution-scope) statistics and per-SM producer/consumer overlap time.
 *
 * Paper passages the operations follow (arxiv 2609.12299, "Argus"):
 *   - Section 3.2 "Region Semantics and Identity": a region is a code span delimited by
 *     begin(id)/end(id) markers with stable ids; the transitions update a nested region
 *     context stack per warp and the innermost active region owns what happens;
 *     temporal traces recover region-labelled intervals.
 *   - Section 3.2 "Region and scope": a scope selects dynamic executions (warp role,
 *     iteration window, SM subset); here scopes are the aggregation keys warp/CTA/SM/kernel.
 *   - Section 3.1 / 3.3: the `duration` signal is the elapsed time of a region.
 *   - Section 3.5 "Synthesizing Qualified Region Reports": evidence is joined by region
 *     identity and dynamic execution context, and attribution ambiguity is reported, not
 *     hidden.
 *
 * Conventions
 *   - All structs are plain little-endian PODs, naturally aligned, with no padding.
 *   - Every pointer named "device" below is a CUDA device pointer on the current device;
 *     `cuda_stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *   - The caller owns every buffer. The operations allocate nothing, keep nothing of a call
 *     for the next one, enqueue their kernels on `cuda_stream` and return without
 *     synchronising; results are valid once the stream reaches that point, so
 *     pair -> aggregate -> overlap on one stream needs no host synchronisation.
 *   - What the library does keep: per device, the launch parameters of its kernels (looked
 *     up on first use, under a lock) and, for argus_pair_intervals_static, the address of
 *     its scratch array; process-wide, the test and measurement switches declared in
 *     argus_testing.h. Host threads may call the operations concurrently, each call with
 *     its own buffers, workspace and stream.
 *   - Return value: host-detectable errors (ARGUS_OK, ARGUS_ERR_INVALID_ARG,
 *     ARGUS_ERR_WORKSPACE, ARGUS_ERR_CUDA). Conditions found on the device are written to
 *     `status->code` (first error wins); on a device error the output arrays are
 *     unspecified, but the GPU is never trapped or hung.
 */
#ifndef ARGUS_H_
#define ARGUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ARGUS_NONE        0xFFFFFFFFu /* parent_region of a top-level interval */
#define ARGUS_MAX_DEPTH   64          /* max simultaneously open frames per stream */
#define ARGUS_MAX_REGIONS 65536       /* upper bound of num_regions */
#define ARGUS_HIST_BINS   64
#define ARGUS_MAX_PAIRS   256         /* (producer, consumer) pairs of one overlap call */

/* return / status codes */
enum {
  ARGUS_OK = 0,
  ARGUS_ERR_INVALID_ARG = 1, /* host: null pointer, bad sizes, misaligned buffer          */
  ARGUS_ERR_WORKSPACE = 2,   /* host: workspace_bytes smaller than the *_workspace_bytes query */
  ARGUS_ERR_CUDA = 3,        /* host: a CUDA runtime call failed                          */
  ARGUS_ERR_CAPACITY = 4,    /* device: interval/ambiguity capacity too small; see *_required */
  ARGUS_ERR_DEPTH = 5,       /* device: a stream would hold more than ARGUS_MAX_DEPTH open frames */
  ARGUS_ERR_BAD_REGION = 6,  /* device: tag>>1 >= num_regions                             */
  ARGUS_ERR_BAD_OFFSETS = 7, /* device: stream_offsets / interval_offsets decreasing or beyond the array */
  ARGUS_ERR_TIMEOUT = 8,     /* device: a bounded wait expired                            */
  ARGUS_ERR_STATIC_LIMIT = 9 /* host: input larger than the built-in scratch of a *_static call */
};

/* One marker event, 16 bytes. tag = region_id << 1 | is_end. ts = globaltimer ns.
 * ctx = dynamic execution context (iteration / tile / token coordinate). */
typedef struct {
  uint64_t ts;
  uint32_t tag;
  uint32_t ctx;
} argus_event_t;

/* interval flags */
#define ARGUS_FLAG_CTX_MISMATCH  1u /* end.ctx != begin.ctx (interval keeps begin's ctx)     */
#define ARGUS_FLAG_TIME_REVERSED 2u /* t_end < t_begin; inclusive saturated to 0             */
#define ARGUS_FLAG_CHILD_CLAMPED 4u /* children sum > inclusive; exclusive saturated to 0    */

/* One matched region occurrence, 48 bytes. depth = stack height before the push
 * (top level = 0); parent_region = region on top of the stack at the push or ARGUS_NONE;
 * begin_idx = index of the begin marker within its stream. */
typedef struct {
  uint64_t t_begin;
  uint64_t inclusive;
  uint64_t exclusive;
  uint32_t region;
  uint32_t ctx;
  uint32_t stream;
  uint32_t parent_region;
  uint32_t begin_idx;
  uint16_t depth;
  uint16_t flags;
} argus_interval_t;

/* ambiguity kinds */
#define ARGUS_AMBIG_UNMATCHED_END   1u /* end with no open frame of its region; depth = stack height */
#define ARGUS_AMBIG_BEGIN_MISNESTED 2u /* begin force-closed by an enclosing region's end            */
#define ARGUS_AMBIG_BEGIN_EOS       3u /* begin still open at the end of its stream                  */

/* One marker that could not be attributed to an interval, 32 bytes. */
typedef struct {
  uint64_t ts;
  uint32_t tag;
  uint32_t ctx;
  uint32_t stream;
  uint32_t event_idx; /* index of the marker within its stream */
  uint32_t kind;
  uint32_t depth;
} argus_ambiguity_t;

/* Statistics of one (scope key, region) cell, 576 bytes. min/max/hist use the inclusive
 * duration; hist bin = d ? 63 - clz64(d) : 0. An empty cell is all zero except
 * min_incl = UINT64_MAX. */
typedef struct {
  uint64_t count;
  uint64_t sum_incl;
  uint64_t min_incl;
  uint64_t max_incl;
  uint64_t sum_excl;
  uint64_t n_unmatched_begin; /* ambiguity kinds 2 and 3 at this (key, region) */
  uint64_t n_unmatched_end;   /* ambiguity kind 1 */
  uint64_t n_flagged;         /* intervals with flags != 0 */
  uint64_t hist[ARGUS_HIST_BINS];
} argus_agg_t;

/* Overlap of one (producer, consumer) pair on one SM, 32 bytes; all in ns. */
typedef struct {
  uint64_t overlap_ns;  /* |U_P  ∩ U_C| */
  uint64_t producer_ns; /* |U_P|       */
  uint64_t consumer_ns; /* |U_C|       */
  uint64_t either_ns;   /* |U_P ∪ U_C| */
} argus_overlap_t;

/* Device-resident status block, 64 bytes. */
typedef struct {
  uint32_t code;       /* ARGUS_OK or the first device error                     */
  uint32_t bad_stream; /* stream where the first error was seen                  */
  uint64_t bad_event;  /* event index within that stream (or offending count)    */
  uint64_t intervals_required;
  uint64_t ambig_required;
  uint64_t n_ctx_mismatch;
  uint64_t n_time_reversed;
  uint64_t n_child_clamped;
  uint64_t n_sequential_tiles; /* diagnostic: times the tiled kernel handed markers of a tile that is not
                                  well nested to the sequential stack machine (0 for well-formed traces) */
} argus_status_t;

/* ---------------------------------------------------------------------------------------
 * argus_pair_intervals — Section 3.2 (per-warp nested region stack; innermost region owns).
 *
 * For every stream s (events[stream_offsets[s] .. stream_offsets[s+1]), in buffer order,
 * never re-sorted by time):
 *   begin(r): push a frame (depth = current height, parent = region on top or ARGUS_NONE);
 *             more than ARGUS_MAX_DEPTH open frames -> ARGUS_ERR_DEPTH.
 *   end(r):   search the stack from the top for the innermost frame of region r.
 *             none  -> ambiguity record UNMATCHED_END (depth = height), stack unchanged.
 *             found -> frames above it are force-closed as BEGIN_MISNESTED (their
 *                      accumulated child time moves to the new top); the found frame
 *                      becomes an interval: inclusive = t_end - t_begin (0 + TIME_REVERSED
 *                      if negative), exclusive = inclusive - sum of inclusive of its
 *                      children among matched intervals (0 + CHILD_CLAMPED if negative),
 *                      ctx from the begin (CTX_MISMATCH if the end's differs).
 *   end of stream: every open frame -> BEGIN_EOS.
 * Outputs (device): intervals ordered by (stream, position of the end marker) with
 * interval_offsets[S+1]; ambiguity records ordered by (stream, event_idx) with
 * ambig_offsets[S+1]. interval_capacity >= floor(N/2) and ambig_capacity >= N always
 * suffice; otherwise ARGUS_ERR_CAPACITY reports the required counts in `status`.
 * Requirements: events 16-byte aligned; num_events = length of `events` (every
 * stream_offsets value must be <= num_events, else ARGUS_ERR_BAD_OFFSETS);
 * num_regions in [1, ARGUS_MAX_REGIONS]; every stream shorter than 2^32 events;
 * num_events < 2^48; workspace 256-byte aligned and at least
 * argus_pair_workspace_bytes(num_events, S, ambig_capacity) bytes. `status` (device, 64 B) is
 * overwritten. Empty streams and num_streams == 0 are legal.
 * ------------------------------------------------------------------------------------- */
size_t argus_pair_workspace_bytes(uint64_t num_events, uint32_t num_streams,
                                  uint64_t ambig_capacity);

int argus_pair_intervals(const argus_event_t* events /*device*/, uint64_t num_events,
                         const uint64_t* stream_offsets /*device [S+1]*/,
                         uint32_t num_streams, uint32_t num_regions,
                         argus_interval_t* intervals /*device*/, uint64_t interval_capacity,
                         uint64_t* interval_offsets /*device [S+1] out*/,
                         argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                         uint64_t* ambig_offsets /*device [S+1] out*/,
                         argus_status_t* status /*device*/, void* workspace /*device*/,
                         size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_pair_intervals_static — no counterpart in the paper: a convenience variant of
 * argus_pair_intervals for callers that cannot allocate device memory.
 *
 * Some callers run where cudaMalloc is off limits: inside a profiler or tool callback, in a
 * process whose memory pool is owned by another component, or on a path that must not touch
 * the allocator because an allocation could synchronise the device or fail late. This entry
 * point needs no workspace argument: its scratch (control block, per-stream counters, work
 * queue, event bitmap and its prefix tables, ambiguity notes) lives in a fixed array inside the library's
 * device image, about 1 MB per GPU that loads the library, held until the process exits.
 * Inputs and outputs are still the caller's buffers. The call makes no cudaMalloc, cudaFree
 * or other allocating call.
 *
 * Limits (larger requests return ARGUS_ERR_STATIC_LIMIT and do nothing):
 *   num_events <= ARGUS_STATIC_MAX_EVENTS, num_streams <= ARGUS_STATIC_MAX_STREAMS,
 *   ambig_capacity <= ARGUS_STATIC_MAX_AMBIG.
 * The first call on each device looks up the scratch array's device address (with that
 * device current); make that first call before starting any stream capture. All calls on a
 * device share the one scratch array: the parts that must start at zero are cleared at the
 * start of every call, but two calls that overlap on the GPU (different streams, no ordering
 * between them) race on it; callers must order them. Results equal argus_pair_intervals'.
 * ------------------------------------------------------------------------------------- */
#define ARGUS_STATIC_MAX_EVENTS  (1u << 20)
#define ARGUS_STATIC_MAX_STREAMS 4096u
#define ARGUS_STATIC_MAX_AMBIG   (1u << 16)

int argus_pair_intervals_static(const argus_event_t* events /*device*/, uint64_t num_events,
                                const uint64_t* stream_offsets /*device [S+1]*/,
                                uint32_t num_streams, uint32_t num_regions,
                                argus_interval_t* intervals /*device*/, uint64_t interval_capacity,
                                uint64_t* interval_offsets /*device [S+1] out*/,
                                argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                                uint64_t* ambig_offsets /*device [S+1] out*/,
                                argus_status_t* status /*device*/, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_aggregate — Section 3.2 "Region and scope" + the `duration` signal (Section 3.1).
 *
 * Reduces intervals (and, if given, ambiguity records) into dense tables of argus_agg_t,
 * one per scope level: warp_tab[S][R] (key = stream), cta_tab[C][R] (key = stream /
 * warps_per_cta, C = S / warps_per_cta), sm_tab[M][R] (key = cta_sm[cta]) and
 * kernel_tab[R]. Any table pointer may be NULL (that level is skipped). Every cell of a
 * requested table is written (empty cells: zero, min_incl = UINT64_MAX).
 * num_streams must be a multiple of warps_per_cta; cta_sm values must be < num_sms.
 * Event-derived ambiguity counters are added at the marker's (region, key).
 * ------------------------------------------------------------------------------------- */
size_t argus_aggregate_workspace_bytes(uint64_t num_intervals, uint32_t num_streams,
                                       uint32_t num_regions);

int argus_aggregate(const argus_interval_t* intervals /*device*/,
                    const uint64_t* interval_offsets /*device [S+1]*/,
                    const argus_ambiguity_t* ambig /*device, nullable*/,
                    const uint64_t* ambig_offsets /*device [S+1], nullable*/,
                    uint32_t num_streams, uint32_t warps_per_cta,
                    const uint32_t* cta_sm /*device [C]*/, uint32_t num_sms,
                    uint32_t num_regions, argus_agg_t* warp_tab /*device [S][R], nullable*/,
                    argus_agg_t* cta_tab /*device [C][R], nullable*/,
                    argus_agg_t* sm_tab /*device [M][R], nullable*/,
                    argus_agg_t* kernel_tab /*device [R], nullable*/,
                    argus_status_t* status /*device*/, void* workspace /*device*/,
                    size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_overlap — producer/consumer overlap per SM (the overlap diagnosis the paper
 * motivates in Sections 1 and 4; scope = SM subset, Section 3.2).
 *
 * For every pair k = (producer region P, consumer region Cn) and SM m: take the half-open
 * spans [t_begin, t_begin + inclusive) of all intervals of region P (resp. Cn) in streams
 * whose CTA maps to m (all depths and contexts, flagged ones included, empty spans
 * dropped); U_P, U_C = their unions. out[k][m] = { |U_P ∩ U_C|, |U_P|, |U_C|, |U_P ∪ U_C| }.
 * At most ARGUS_MAX_PAIRS pairs per call (more: ARGUS_ERR_INVALID_ARG).
 * max_intervals is an upper bound of interval_offsets[S] known on the host (for instance
 * the capacity given to argus_pair_intervals); it sizes the workspace, and a stream whose
 * offsets reach beyond it is not read (status->code = ARGUS_ERR_BAD_OFFSETS). If more spans
 * are selected than the workspace holds, status->code = ARGUS_ERR_CAPACITY.
 * ------------------------------------------------------------------------------------- */
size_t argus_overlap_workspace_bytes(uint64_t max_intervals, uint32_t num_streams,
                                     uint32_t num_pairs, uint32_t num_sms);

int argus_overlap(const argus_interval_t* intervals /*device*/, uint64_t max_intervals,
                  const uint64_t* interval_offsets /*device [S+1]*/, uint32_t num_streams,
                  uint32_t warps_per_cta, const uint32_t* cta_sm /*device [C]*/,
                  uint32_t num_sms, const uint32_t* pairs /*device [K][2]*/,
                  uint32_t num_pairs, argus_overlap_t* out /*device [K][M]*/,
                  argus_status_t* status /*device*/, void* workspace /*device*/,
                  size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * Scope selection — Section 1 (the observe(region, signals, scope) query) and Section 3.2
 * "Region and scope": the region is the code being asked about, the scope picks which of
 * its dynamic executions count, by the role of the warp, by a window of iterations or by a
 * subset of SMs.
 *
 * An interval belongs to a scope when all four tests hold:
 *   iteration window : ctx_lo <= interval.ctx <= ctx_hi  (ctx is the begin marker's)
 *   warp role        : bit (interval.stream % warps_per_cta) of warp_mask is set
 *                      (warps 64 and up of a CTA are never selected unless warp_mask is all ones)
 *   SM subset        : bit cta_sm[interval.stream / warps_per_cta] of sm_mask is set
 *   region set       : bit interval.region of region_mask is set
 * sm_mask and region_mask are DEVICE arrays of ceil(num_sms / 32) and ceil(num_regions / 32)
 * words (bit i of word i / 32); NULL selects everything. The struct itself is read on the
 * host at call time. An ambiguity record is tested the same way with its own ctx, stream and
 * tag >> 1. Inclusive and exclusive times are those pairing computed over the whole stream:
 * selection does not change them.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  uint32_t ctx_lo, ctx_hi;       /* inclusive on both ends; 0 .. UINT32_MAX selects all      */
  uint64_t warp_mask;            /* UINT64_MAX selects all                                    */
  const uint32_t* sm_mask;       /* device, nullable                                          */
  const uint32_t* region_mask;   /* device, nullable                                          */
} argus_scope_t;

#define ARGUS_MAX_ITER_ROWS 65536u /* rows of an iteration table (ctx_hi - ctx_lo + 1)        */

/* ---------------------------------------------------------------------------------------
 * argus_aggregate_scoped — argus_aggregate over the intervals (and ambiguity records) of one
 * scope, plus two tables keyed the way the paper's queries select executions:
 *   role_tab[W][R] : key = warp index inside its CTA (stream % warps_per_cta), which is the
 *                    role of the warp in a warp-specialised kernel (the GEMM example of
 *                    Section 1 measures per role and per iteration), reduced over all CTAs;
 *   iter_tab[I][R] : key = ctx - ctx_lo, I = ctx_hi - ctx_lo + 1 <= ARGUS_MAX_ITER_ROWS:
 *                    per-iteration statistics across warps (the worked example of Section 3.1
 *                    selects sixteen pipeline iterations). Needs a non-NULL scope.
 * scope == NULL selects everything; then warp/cta/sm/kernel tables equal argus_aggregate's.
 * Every cell of a requested table is written. Workspace: argus_aggregate_workspace_bytes.
 * Errors as argus_aggregate; ARGUS_ERR_INVALID_ARG also when iter_tab is given without a
 * scope or with more than ARGUS_MAX_ITER_ROWS rows, or ctx_hi < ctx_lo.
 * ------------------------------------------------------------------------------------- */
int argus_aggregate_scoped(const argus_interval_t* intervals /*device*/,
                           const uint64_t* interval_offsets /*device [S+1]*/,
                           const argus_ambiguity_t* ambig /*device, nullable*/,
                           const uint64_t* ambig_offsets /*device [S+1], nullable*/,
                           uint32_t num_streams, uint32_t warps_per_cta,
                           const uint32_t* cta_sm /*device [C]*/, uint32_t num_sms,
                           uint32_t num_regions, const argus_scope_t* scope /*host, nullable*/,
                           argus_agg_t* warp_tab /*device [S][R], nullable*/,
                           argus_agg_t* cta_tab /*device [C][R], nullable*/,
                           argus_agg_t* sm_tab /*device [M][R], nullable*/,
                           argus_agg_t* kernel_tab /*device [R], nullable*/,
                           argus_agg_t* role_tab /*device [W][R], nullable*/,
                           argus_agg_t* iter_tab /*device [I][R], nullable*/,
                           argus_status_t* status /*device*/, void* workspace /*device*/,
                           size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_overlap_scoped — argus_overlap over the intervals of one scope (for instance the
 * producer/consumer overlap of a few pipeline iterations on a subset of SMs). scope == NULL
 * selects everything. out[k][m] of an SM outside the scope is all zero. Workspace:
 * argus_overlap_workspace_bytes.
 * ------------------------------------------------------------------------------------- */
int argus_overlap_scoped(const argus_interval_t* intervals /*device*/, uint64_t max_intervals,
                         const uint64_t* interval_offsets /*device [S+1]*/,
                         uint32_t num_streams, uint32_t warps_per_cta,
                         const uint32_t* cta_sm /*device [C]*/, uint32_t num_sms,
                         const uint32_t* pairs /*device [K][2]*/, uint32_t num_pairs,
                         const argus_scope_t* scope /*host, nullable*/,
                         argus_overlap_t* out /*device [K][M]*/, argus_status_t* status /*device*/,
                         void* workspace /*device*/, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * PC-to-region attribution — Section 3.2 (the figure on dynamic PC-to-region mapping: each
 * execution of the instruction at PC p is credited to the innermost region active in its
 * warp at that moment) and Section 3.5 "Ambiguity-aware attribution" (the weights alpha,
 * the lifted metric and the association entropy).
 *
 * Mapping-run traces reuse the marker record. Regions keep ids 0 .. R-1. "The instruction
 * at PC index p executed k times here" is written as a begin/end pair of the extra region
 * id R (exec_region) placed at that point of the stream:
 *     { ts = 0, tag = R << 1,       ctx = p }     { ts = k, tag = (R << 1) | 1, ctx = p }
 * so that argus_pair_intervals (called with num_regions = R + 1) turns it into an interval
 * with region R, ctx p, inclusive k and parent_region = the innermost active region, under
 * exactly the stack rules of pairing, mis-nested and unmatched markers included. (Times of
 * real regions are meaningless in such a trace; only the counts are used.)
 *
 * argus_map_pc_counts: counts[r][p] (u64, [(R + 1)][P], row R = outside every region) =
 * sum of inclusive over the intervals with region exec_region, ctx p and parent_region r
 * (parent NONE or >= R goes to row R). Every cell is written. Intervals of exec_region
 * whose ctx >= num_pcs set status->code = ARGUS_ERR_INVALID_ARG.
 *
 * argus_attribute (fp64): with N_p = sum_r counts[r][p], alpha[r][p] = counts[r][p] / N_p
 * (0 where N_p = 0), mhat[r] = sum_p alpha[r][p] * metric[p], entropy[p] = - sum over
 * r with alpha > 0 of alpha * ln(alpha). alpha may be NULL. The sums over p are taken in a
 * fixed order (block partial sums, then their sum), so results repeat from run to run; they
 * agree with a sequential sum to rounding (relative 1e-12 of sum_p |alpha * metric|).
 * ------------------------------------------------------------------------------------- */
int argus_map_pc_counts(const argus_interval_t* intervals /*device*/,
                        const uint64_t* interval_offsets /*device [S+1]*/, uint32_t num_streams,
                        uint32_t exec_region /* = R */, uint32_t num_pcs,
                        uint64_t* counts /*device [(R+1)][P]*/, argus_status_t* status /*device*/,
                        void* cuda_stream);

size_t argus_attribute_workspace_bytes(uint32_t num_rows, uint32_t num_pcs);

int argus_attribute(const uint64_t* counts /*device [rows][P]*/, uint32_t num_rows,
                    uint32_t num_pcs, const double* metric /*device [P]*/,
                    double* mhat /*device [rows]*/, double* entropy /*device [P]*/,
                    double* alpha /*device [rows][P], nullable*/, void* workspace /*device*/,
                    size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * Cross-run join with distribution statistics — Section 3.3 (a probe measurement is joined
 * back to the reference trace through its stable region / operation id and its dynamic
 * scope), Section 3.5 "Qualified synthesis" (a probe of iteration i is matched to the same
 * operation of reference iteration i, never by comparing timestamps of different runs) and
 * the appendix on the asynchronous-timeline trace (mean and 0th / 20th / 40th / 60th / 80th
 * percentile of the repeated samples of every operation).
 *
 * Query q names one interval of the reference run, ref_index[q] (an index into `reference`).
 * Its key is (stream, region, ctx). Every interval of `samples` (the intervals of any number
 * of probe runs, in any order) with the same key is a sample of it; its value is the sample's
 * inclusive time. out[q] = number of samples, their sum (mean = sum / count), minimum ... :
 * pct[j] = sorted_values[(j * count) / 5] for j = 0..4 (0th = minimum, 80th close to the
 * maximum), all zero when there is no sample. Reference intervals that share a key share
 * their samples. At most ARGUS_JOIN_MAX_SAMPLES samples per query are ranked; a query with
 * more sets status->code = ARGUS_ERR_CAPACITY (count and sum are still exact).
 * Cost is num_queries passes over `samples`: meant for the selected operations of a query
 * (tens to thousands), not for joining whole traces.
 * ------------------------------------------------------------------------------------- */
#define ARGUS_JOIN_MAX_SAMPLES 4096u

typedef struct {
  uint64_t count, sum;   /* samples joined, sum of their inclusive times                  */
  uint64_t pct[5];       /* 0th, 20th, 40th, 60th, 80th percentile                        */
  uint64_t max;          /* largest sample                                                */
} argus_join_t;          /* 64 bytes */

int argus_join_samples(const argus_interval_t* reference /*device*/, uint64_t num_reference,
                       const uint64_t* ref_index /*device [Q]*/, uint32_t num_queries,
                       const argus_interval_t* samples /*device*/, uint64_t num_samples,
                       argus_join_t* out /*device [Q]*/, argus_status_t* status /*device*/,
                       void* cuda_stream);

/* The same when the samples are the interval arrays of num_runs probe runs, one after the
 * other in `samples`, each ordered by stream as argus_pair_intervals writes them:
 * sample_offsets[run * (S + 1) + s] .. [run * (S + 1) + s + 1] (indices into `samples`) are
 * the intervals of stream s in that run. A query then reads only its own stream's samples in
 * every run (num_runs * N / S records instead of N), which is what makes thousands of queries
 * against whole traces affordable. Offsets that decrease or leave `samples` set
 * ARGUS_ERR_BAD_OFFSETS. Same results as argus_join_samples on the same records. */
int argus_join_samples_grouped(const argus_interval_t* reference /*device*/, uint64_t num_reference,
                               const uint64_t* ref_index /*device [Q]*/, uint32_t num_queries,
                               const argus_interval_t* samples /*device*/, uint64_t num_samples,
                               const uint64_t* sample_offsets /*device [num_runs][S+1]*/,
                               uint32_t num_runs, uint32_t num_streams,
                               argus_join_t* out /*device [Q]*/, argus_status_t* status /*device*/,
                               void* cuda_stream);

/* The same join for probe-run samples in ANY order, in one pass over `samples` for all queries
 * together (Section 3.5: evidence is joined by region identity and execution context, never by
 * comparing timestamps across runs): the distinct (stream, region, ctx) keys of the queries go
 * into a hash table in the workspace, every sample is read once and looked up, matching values
 * are appended to their key's list (at most ARGUS_JOIN_MAX_SAMPLES are kept and ranked; count
 * and sum stay exact, ARGUS_ERR_CAPACITY reports the overflow), and one block per query sorts
 * and ranks. Cost: one read of `samples` whatever the number of queries. workspace: device
 * memory, 256-byte aligned, argus_join_workspace_bytes(num_queries) bytes, owned by the caller,
 * contents unspecified before and after. Same results as argus_join_samples. */
size_t argus_join_workspace_bytes(uint32_t num_queries);
int argus_join_samples_hashed(const argus_interval_t* reference /*device*/, uint64_t num_reference,
                              const uint64_t* ref_index /*device [Q]*/, uint32_t num_queries,
                              const argus_interval_t* samples /*device*/, uint64_t num_samples,
                              argus_join_t* out /*device [Q]*/, argus_status_t* status /*device*/,
                              void* workspace /*device*/, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * Ring-buffer input — a second container for the marker records of Section 3.2: tracers
 * commonly give every warp a fixed slot of slot_capacity records and let it wrap. The paper
 * does not fix a container; this one exercises the recovery path (after a wrap the surviving
 * records may start with ends whose begins were overwritten: they come out as unmatched-end
 * ambiguity records).
 *
 * ring[s * slot_capacity + (i % slot_capacity)] holds the i-th record stream s wrote;
 * written[s] counts all records it ever wrote. The surviving records of stream s are the
 * last min(written[s], slot_capacity), oldest first. argus_ring_linearise copies them into
 * `events` in packed CSR form and writes stream_offsets[S + 1] (stream_offsets[0] = 0), ready
 * for argus_pair_intervals; dropped[s] (nullable) = records lost to the wrap. If the packed
 * records exceed event_capacity nothing is copied and status->code = ARGUS_ERR_CAPACITY with
 * the required count in status->intervals_required.
 * ------------------------------------------------------------------------------------- */
int argus_ring_linearise(const argus_event_t* ring /*device [S][slot_capacity]*/,
                         uint32_t slot_capacity, const uint64_t* written /*device [S]*/,
                         uint32_t num_streams, argus_event_t* events /*device*/,
                         uint64_t event_capacity, uint64_t* stream_offsets /*device [S+1] out*/,
                         uint64_t* dropped /*device [S] out, nullable*/,
                         argus_status_t* status /*device*/, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_pair_intervals_ring — pairing straight from the ring container above, without the
 * packed copy: the pairing kernel fetches every tile of a stream from its slot with one bulk
 * copy, or two where the tile straddles the slot's end. Results (intervals, ambiguity
 * records, offsets, status) are those of argus_ring_linearise followed by
 * argus_pair_intervals; event indices (begin_idx, event_idx) count the surviving records of
 * the stream, oldest first. stream_offsets[S + 1] (out) receives the offsets the packed form
 * would have, dropped[S] (out, nullable) the records lost to the wrap. Workspace:
 * argus_pair_workspace_bytes(S * slot_capacity, S, ambig_capacity) bytes, 256-byte aligned.
 * ------------------------------------------------------------------------------------- */
int argus_pair_intervals_ring(const argus_event_t* ring /*device [S][slot_capacity]*/,
                              uint32_t slot_capacity, const uint64_t* written /*device [S]*/,
                              uint32_t num_streams, uint32_t num_regions,
                              uint64_t* stream_offsets /*device [S+1] out*/,
                              uint64_t* dropped /*device [S] out, nullable*/,
                              argus_interval_t* intervals /*device*/, uint64_t interval_capacity,
                              uint64_t* interval_offsets /*device [S+1] out*/,
                              argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                              uint64_t* ambig_offsets /*device [S+1] out*/,
                              argus_status_t* status /*device*/, void* workspace /*device*/,
                              size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------
 * argus_synthesize — the three operations above in one call, with identical results
 * (Section 3.2 for intervals and scopes; the Synthesize task of Section 3.4).
 *
 * Arguments have the meaning they have in argus_pair_intervals, argus_aggregate and
 * argus_overlap. Pairing also writes an 8-byte digest of every interval into the workspace
 * (4 bytes per event), and one pass over the digests both aggregates the intervals and
 * selects the overlap spans (up to 400 regions and 128 pairs; beyond that the three
 * operations run one after the other). Any of the four tables may be NULL; without any
 * table the overlap stage reads the interval records. num_pairs may be 0. max_overlap_spans bounds
 * the spans selected for overlap over all pairs (an interval counts once per pair and role
 * its region appears in); more than that -> ARGUS_ERR_CAPACITY with the count in
 * status->intervals_required. One status block reports the first error of any stage.
 * ------------------------------------------------------------------------------------- */
size_t argus_synthesize_workspace_bytes(uint64_t num_events, uint32_t num_streams,
                                        uint32_t num_regions, uint64_t ambig_capacity,
                                        uint32_t num_pairs, uint32_t num_sms,
                                        uint64_t max_overlap_spans);

int argus_synthesize(const argus_event_t* events /*device*/, uint64_t num_events,
                     const uint64_t* stream_offsets /*device [S+1]*/, uint32_t num_streams,
                     uint32_t num_regions, argus_interval_t* intervals /*device*/,
                     uint64_t interval_capacity, uint64_t* interval_offsets /*device [S+1] out*/,
                     argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                     uint64_t* ambig_offsets /*device [S+1] out*/, uint32_t warps_per_cta,
                     const uint32_t* cta_sm /*device [C]*/, uint32_t num_sms,
                     argus_agg_t* warp_tab /*device, nullable*/, argus_agg_t* cta_tab /*device, nullable*/,
                     argus_agg_t* sm_tab /*device, nullable*/, argus_agg_t* kernel_tab /*device, nullable*/,
                     const uint32_t* pairs /*device [K][2]*/, uint32_t num_pairs,
                     argus_overlap_t* overlap_out /*device [K][M]*/, uint64_t max_overlap_spans,
                     argus_status_t* status /*device*/, void* workspace /*device*/,
                     size_t workspace_bytes, void* cuda_stream);

/* The same from the ring container: argus_pair_intervals_ring's pairing inside the one-call
 * pipeline. stream_offsets[S + 1] and dropped[S] (nullable) are outputs as there. Workspace:
 * argus_synthesize_workspace_bytes(S * slot_capacity, ...) bytes. */
int argus_synthesize_ring(const argus_event_t* ring /*device [S][slot_capacity]*/,
                          uint32_t slot_capacity, const uint64_t* written /*device [S]*/,
                          uint32_t num_streams, uint32_t num_regions,
                          uint64_t* stream_offsets /*device [S+1] out*/,
                          uint64_t* dropped /*device [S] out, nullable*/,
                          argus_interval_t* intervals /*device*/, uint64_t interval_capacity,
                          uint64_t* interval_offsets /*device [S+1] out*/,
                          argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                          uint64_t* ambig_offsets /*device [S+1] out*/, uint32_t warps_per_cta,
                          const uint32_t* cta_sm /*device [C]*/, uint32_t num_sms,
                          argus_agg_t* warp_tab /*device, nullable*/, argus_agg_t* cta_tab /*device, nullable*/,
                          argus_agg_t* sm_tab /*device, nullable*/, argus_agg_t* kernel_tab /*device, nullable*/,
                          const uint32_t* pairs /*device [K][2]*/, uint32_t num_pairs,
                          argus_overlap_t* overlap_out /*device [K][M]*/, uint64_t max_overlap_spans,
                          argus_status_t* status /*device*/, void* workspace /*device*/,
                          size_t workspace_bytes, void* cuda_stream);

/* Copies the device status block to host memory and synchronises `cuda_stream`.
 * Returns ARGUS_OK or ARGUS_ERR_CUDA; the device-side code is in host_copy->code. */
int argus_status_fetch(const argus_status_t* dev_status, argus_status_t* host_copy,
                       void* cuda_stream);

/* Static, NUL-terminated description of a code; never NULL. */
const char* argus_strerror(int code);

/* Library version: major * 10000 + minor * 100 + patch. */
int argus_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ARGUS_H_ */
