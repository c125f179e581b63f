/*
 * argus_testing.h — test, tuning and measurement aids of the region-trace library. Not part of
 * the product ABI (argus.h): nothing here changes a result, and production callers need none
 * of it. The switches are process-wide.
 */
#ifndef ARGUS_TESTING_H_
#define ARGUS_TESTING_H_

#include "argus.h"

#ifdef __cplusplus
extern "C" {
#endif

/* argus_pair_intervals (Section 3.2, the nested region context stack per warp) with an explicit
 * kernel choice: 0 = automatic, 1 = one thread per stream (sequential stack, any input),
 * 2 = tiled kernel (CTAs walk streams tile by tile, long streams a chunk at a time, and hand
 * the markers that break the nesting to the sequential stack). Arguments, ownership and errors
 * as argus_pair_intervals; all choices produce identical output. */
int argus_pair_intervals_ex(const argus_event_t* events /*device*/, uint64_t num_events,
                            const uint64_t* stream_offsets /*device [S+1]*/,
                            uint32_t num_streams, uint32_t num_regions,
                            argus_interval_t* intervals /*device*/, uint64_t interval_capacity,
                            uint64_t* interval_offsets /*device [S+1] out*/,
                            argus_ambiguity_t* ambig /*device*/, uint64_t ambig_capacity,
                            uint64_t* ambig_offsets /*device [S+1] out*/,
                            argus_status_t* status /*device*/, void* workspace /*device*/,
                            size_t workspace_bytes, void* cuda_stream, int kernel_choice);

/* Measurement helpers (host-side bookkeeping only).
 * argus_launch_count: kernels this library has launched since it was loaded.
 * argus_profile_enable(1): from now on each operation records a CUDA event pair on its stream
 * around its dominant kernel (slot 0 = pairing kernel of argus_pair_intervals, 1 = per-stream
 * accumulation kernel of argus_aggregate, 2 = sort kernel of argus_overlap, 3 = reserved).
 * argus_profile_read: waits for the recorded events, writes per slot the summed kernel time in
 * milliseconds and the number of recorded launches (arrays of 4), and forgets them. */
unsigned long long argus_launch_count(void);
void argus_profile_enable(int on);
int argus_profile_read(double* ms_total /*host [4]*/, unsigned long long* launches /*host [4]*/);

/* argus_set_synthesize_mode: where argus_synthesize aggregates and selects overlap spans: -1 automatic,
 * 1 in one pass over the intervals' digests, 2 the three plain operations, 3 in one pass over the interval
 * records. A mode the inputs do not allow falls back to the automatic choice.
 * argus_set_tile_variant: shape of the tiled pairing kernel, 0 = the default <128 threads, 5 events per
 * thread, 7 blocks per SM>, 1..3 = <192,5,4>, <64,5,8>, <256,7,2> (tiles end at other places).
 * argus_testing_set_poll_limit: polls after which a block of the tiled pairing kernel that waits for a
 * hand-over gives up with ARGUS_ERR_TIMEOUT (default 2^19, about a second; 0 restores the default). A test
 * sets it to a few polls to see the bounded wait run out and the call return with the status set. */
void argus_set_synthesize_mode(int mode);
void argus_set_tile_variant(int variant);
void argus_testing_set_poll_limit(unsigned int polls);

#ifdef __cplusplus
}
#endif
#endif /* ARGUS_TESTING_H_ */
