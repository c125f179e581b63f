"""B200-native region-trace synthesis: marker events -> intervals -> scope statistics -> overlap.

Thin binding over the C-ABI library `libargus.so` (see include/argus.h). Every step of the path runs
in the library's CUDA kernels; this module only marshals arguments and uses PyTorch for device
memory and streams. There is no CPU fallback: if the library has not been built, every call raises.
"""
from .binding import (AGG_DTYPE, AMBIG_DTYPE, EVENT_DTYPE, INTERVAL_DTYPE, OVERLAP_DTYPE, STATUS_DTYPE, ArgusError,
                      AggregateResult, PairResult, argus_aggregate, argus_aggregate_workspace_bytes, argus_overlap,
                      argus_overlap_workspace_bytes, argus_pair_intervals, argus_pair_workspace_bytes,
                      argus_launch_count, argus_profile_enable, argus_profile_read, argus_status_fetch, argus_strerror,
                      argus_version, library_path, load_library, argus_synthesize,
                      argus_synthesize_workspace_bytes, SynthesizeResult, argus_pair_intervals_static, ArgusScope,
                      ScopedAggregateResult, argus_aggregate_scoped, argus_overlap_scoped,
                      argus_map_pc_counts, argus_attribute, argus_join_samples, argus_join_samples_grouped, argus_join_samples_hashed, JOIN_DTYPE,
                      argus_ring_linearise, argus_pair_intervals_ring, argus_synthesize_ring)

__all__ = [
    "AGG_DTYPE", "AMBIG_DTYPE", "EVENT_DTYPE", "INTERVAL_DTYPE", "OVERLAP_DTYPE", "STATUS_DTYPE", "ArgusError",
    "AggregateResult", "PairResult", "argus_aggregate", "argus_aggregate_workspace_bytes", "argus_overlap",
    "argus_overlap_workspace_bytes", "argus_pair_intervals", "argus_pair_workspace_bytes", "argus_status_fetch",
    "argus_strerror", "argus_version", "library_path", "load_library", "argus_launch_count",
    "argus_profile_enable", "argus_profile_read", "argus_synthesize", "argus_synthesize_workspace_bytes",
    "SynthesizeResult", "argus_pair_intervals_static", "ArgusScope", "ScopedAggregateResult", "argus_aggregate_scoped",
    "argus_overlap_scoped", "argus_map_pc_counts", "argus_attribute",
    "argus_join_samples", "argus_join_samples_grouped", "argus_join_samples_hashed", "JOIN_DTYPE", "argus_ring_linearise", "argus_pair_intervals_ring", "argus_synthesize_ring",
]
