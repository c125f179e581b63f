"""ctypes binding of libargus.so: same names as the C-ABI, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))

EVENT_DTYPE = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4")])
INTERVAL_DTYPE = np.dtype([("t_begin", "<u8"), ("inclusive", "<u8"), ("exclusive", "<u8"), ("region", "<u4"),
                           ("ctx", "<u4"), ("stream", "<u4"), ("parent_region", "<u4"), ("begin_idx", "<u4"),
                           ("depth", "<u2"), ("flags", "<u2")])
AMBIG_DTYPE = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4"), ("stream", "<u4"), ("event_idx", "<u4"),
                        ("kind", "<u4"), ("depth", "<u4")])
AGG_DTYPE = np.dtype([("count", "<u8"), ("sum_incl", "<u8"), ("min_incl", "<u8"), ("max_incl", "<u8"),
                      ("sum_excl", "<u8"), ("n_unmatched_begin", "<u8"), ("n_unmatched_end", "<u8"),
                      ("n_flagged", "<u8"), ("hist", "<u8", (64,))])
OVERLAP_DTYPE = np.dtype([("overlap_ns", "<u8"), ("producer_ns", "<u8"), ("consumer_ns", "<u8"), ("either_ns", "<u8")])
STATUS_DTYPE = np.dtype([("code", "<u4"), ("bad_stream", "<u4"), ("bad_event", "<u8"), ("intervals_required", "<u8"),
                         ("ambig_required", "<u8"), ("n_ctx_mismatch", "<u8"), ("n_time_reversed", "<u8"),
                         ("n_child_clamped", "<u8"), ("n_sequential_tiles", "<u8")])

KERNEL_AUTO, KERNEL_THREAD_PER_STREAM, KERNEL_TILED = 0, 1, 2


class ArgusError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {argus_strerror(code)} (code {code})")
        self.code = code


def library_path() -> str:
    return os.path.join(_HERE, "libargus.so")


_lib = None


def load_library():
    """Loads libargus.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -c 'import __graft_entry__ as g; g.build()'`; "
                           "this package has no CPU fallback")
    lib = ctypes.CDLL(path)
    vp, u32, u64, sz, ci = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_size_t, ctypes.c_int
    lib.argus_pair_workspace_bytes.argtypes = [u64, u32, u64]
    lib.argus_pair_workspace_bytes.restype = sz
    pair_args = [vp, u64, vp, u32, u32, vp, u64, vp, vp, u64, vp, vp, vp, sz, vp]
    lib.argus_pair_intervals.argtypes = pair_args
    lib.argus_pair_intervals.restype = ci
    lib.argus_pair_intervals_ex.argtypes = pair_args + [ci]
    lib.argus_pair_intervals_ex.restype = ci
    lib.argus_aggregate_workspace_bytes.argtypes = [u64, u32, u32]
    lib.argus_aggregate_workspace_bytes.restype = sz
    lib.argus_aggregate.argtypes = [vp, vp, vp, vp, u32, u32, vp, u32, u32, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.argus_aggregate.restype = ci
    lib.argus_overlap_workspace_bytes.argtypes = [u64, u32, u32, u32]
    lib.argus_overlap_workspace_bytes.restype = sz
    lib.argus_overlap.argtypes = [vp, u64, vp, u32, u32, vp, u32, vp, u32, vp, vp, vp, sz, vp]
    lib.argus_overlap.restype = ci
    lib.argus_aggregate_scoped.argtypes = [vp, vp, vp, vp, u32, u32, vp, u32, u32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.argus_aggregate_scoped.restype = ci
    lib.argus_overlap_scoped.argtypes = [vp, u64, vp, u32, u32, vp, u32, vp, u32, vp, vp, vp, vp, sz, vp]
    lib.argus_overlap_scoped.restype = ci
    lib.argus_map_pc_counts.argtypes = [vp, vp, u32, u32, u32, vp, vp, vp]
    lib.argus_map_pc_counts.restype = ci
    lib.argus_attribute_workspace_bytes.argtypes = [u32, u32]
    lib.argus_attribute_workspace_bytes.restype = sz
    lib.argus_attribute.argtypes = [vp, u32, u32, vp, vp, vp, vp, vp, sz, vp]
    lib.argus_attribute.restype = ci
    lib.argus_join_samples.argtypes = [vp, u64, vp, u32, vp, u64, vp, vp, vp]
    lib.argus_join_samples_grouped.argtypes = [vp, u64, vp, u32, vp, u64, vp, u32, u32, vp, vp, vp]
    lib.argus_join_samples_grouped.restype = ci
    lib.argus_join_samples.restype = ci
    lib.argus_join_workspace_bytes.argtypes = [u32]
    lib.argus_join_workspace_bytes.restype = sz
    lib.argus_join_samples_hashed.argtypes = [vp, u64, vp, u32, vp, u64, vp, vp, vp, sz, vp]
    lib.argus_join_samples_hashed.restype = ci
    lib.argus_ring_linearise.argtypes = [vp, u32, vp, u32, vp, u64, vp, vp, vp, vp]
    lib.argus_ring_linearise.restype = ci
    lib.argus_pair_intervals_ring.argtypes = [vp, u32, vp, u32, u32, vp, vp, vp, u64, vp, vp, u64, vp, vp, vp, sz, vp]
    lib.argus_pair_intervals_ring.restype = ci
    lib.argus_status_fetch.argtypes = [vp, vp, vp]
    lib.argus_status_fetch.restype = ci
    lib.argus_strerror.argtypes = [ci]
    lib.argus_strerror.restype = ctypes.c_char_p
    lib.argus_version.argtypes = []
    lib.argus_version.restype = ci
    lib.argus_launch_count.argtypes = []
    lib.argus_launch_count.restype = ctypes.c_ulonglong
    lib.argus_profile_enable.argtypes = [ci]
    lib.argus_profile_enable.restype = None
    lib.argus_profile_read.argtypes = [vp, vp]
    lib.argus_profile_read.restype = ci
    lib.argus_pair_intervals_static.argtypes = [vp, u64, vp, u32, u32, vp, u64, vp, vp, u64, vp, vp, vp]
    lib.argus_pair_intervals_static.restype = ci
    lib.argus_synthesize_workspace_bytes.argtypes = [u64, u32, u32, u64, u32, u32, u64]
    lib.argus_synthesize_workspace_bytes.restype = sz
    lib.argus_synthesize.argtypes = [vp, u64, vp, u32, u32, vp, u64, vp, vp, u64, vp, u32, vp, u32, vp, vp, vp, vp, vp, u32,
                                     vp, u64, vp, vp, sz, vp]
    lib.argus_synthesize.restype = ci
    lib.argus_synthesize_ring.argtypes = [vp, u32, vp, u32, u32, vp, vp, vp, u64, vp, vp, u64, vp, u32, vp, u32, vp, vp, vp, vp, vp,
                                          u32, vp, u64, vp, vp, sz, vp]
    lib.argus_synthesize_ring.restype = ci
    _lib = lib
    return lib


def argus_set_tile_variant(v: int) -> None:
    """Tuning aid: selects an alternative tile shape of the tiled pairing kernel (0 = default)."""
    lib = load_library()
    lib.argus_set_tile_variant.argtypes = [ctypes.c_int]
    lib.argus_set_tile_variant.restype = None
    lib.argus_set_tile_variant(int(v))


def argus_set_synthesize_mode(mode: int) -> None:
    """Where argus_synthesize aggregates: -1 automatic, 1 in one pass over the intervals' digests, 2 the plain
    calls, 3 in one pass over the interval records (test aid; results are identical)."""
    load_library().argus_set_synthesize_mode(int(mode))


def argus_launch_count() -> int:
    return int(load_library().argus_launch_count())


def argus_profile_enable(on: bool) -> None:
    load_library().argus_profile_enable(1 if on else 0)


def argus_profile_read():
    """Returns ({slot: total ms}, {slot: launches}) for the slots pair / aggregate / overlap."""
    ms = (ctypes.c_double * 4)()
    n = (ctypes.c_ulonglong * 4)()
    rc = load_library().argus_profile_read(ctypes.addressof(ms), ctypes.addressof(n))
    if rc != 0:
        raise ArgusError(rc, "argus_profile_read")
    names = ("pair", "aggregate", "overlap", "reserved")
    return {k: ms[i] for i, k in enumerate(names)}, {k: int(n[i]) for i, k in enumerate(names)}


def argus_strerror(code: int) -> str:
    return load_library().argus_strerror(int(code)).decode()


def argus_version() -> int:
    return load_library().argus_version()


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream_ptr(device):
    return torch.cuda.current_stream(device).cuda_stream


def _bytes(n: int, device) -> torch.Tensor:
    return torch.empty(max(int(n), 1), dtype=torch.uint8, device=device)


def argus_pair_workspace_bytes(num_events: int, num_streams: int, ambig_capacity: int) -> int:
    return load_library().argus_pair_workspace_bytes(num_events, num_streams, ambig_capacity)


def argus_aggregate_workspace_bytes(num_intervals: int, num_streams: int, num_regions: int) -> int:
    return load_library().argus_aggregate_workspace_bytes(num_intervals, num_streams, num_regions)


def argus_overlap_workspace_bytes(max_intervals: int, num_streams: int, num_pairs: int, num_sms: int) -> int:
    return load_library().argus_overlap_workspace_bytes(max_intervals, num_streams, num_pairs, num_sms)


def argus_status_fetch(status: torch.Tensor) -> np.void:
    """Synchronises the current stream and returns the status block as a numpy record."""
    host = np.zeros(1, dtype=STATUS_DTYPE)
    rc = load_library().argus_status_fetch(status.data_ptr(), host.ctypes.data, _stream_ptr(status.device))
    if rc != 0:
        raise ArgusError(rc, "argus_status_fetch")
    return host[0]


@dataclass
class PairResult:
    intervals: torch.Tensor          # uint8 [interval_capacity * 48]
    interval_offsets: torch.Tensor   # int64 [S + 1]
    ambig: torch.Tensor              # uint8 [ambig_capacity * 32]
    ambig_offsets: torch.Tensor      # int64 [S + 1]
    status: torch.Tensor             # uint8 [64]
    interval_capacity: int
    ambig_capacity: int
    workspace: torch.Tensor

    def fetch_status(self):
        return argus_status_fetch(self.status)

    def intervals_numpy(self) -> np.ndarray:
        n = min(int(self.interval_offsets[-1].item()), self.interval_capacity)
        return self.intervals[: n * 48].cpu().numpy().view(INTERVAL_DTYPE)

    def ambig_numpy(self) -> np.ndarray:
        n = min(int(self.ambig_offsets[-1].item()), self.ambig_capacity)
        return self.ambig[: n * 32].cpu().numpy().view(AMBIG_DTYPE)


def argus_pair_intervals(events: torch.Tensor, stream_offsets: torch.Tensor, num_regions: int,
                         interval_capacity: int | None = None, ambig_capacity: int | None = None,
                         out: PairResult | None = None, kernel: int = KERNEL_AUTO) -> PairResult:
    """events: device tensor holding N 16-byte records; stream_offsets: device int64 [S+1].
    Enqueues on the current stream of the events' device and returns device tensors (no sync)."""
    lib = load_library()
    dev = events.device
    if dev.type != "cuda":
        raise ValueError("events must be a CUDA tensor")
    n = events.numel() * events.element_size() // 16
    S = stream_offsets.numel() - 1
    icap = n // 2 if interval_capacity is None else int(interval_capacity)
    acap = n if ambig_capacity is None else int(ambig_capacity)
    if out is None:
        ws_bytes = lib.argus_pair_workspace_bytes(n, S, acap)
        out = PairResult(_bytes(icap * 48, dev), torch.empty(S + 1, dtype=torch.int64, device=dev),
                         _bytes(acap * 32, dev), torch.empty(S + 1, dtype=torch.int64, device=dev),
                         _bytes(64, dev), icap, acap, _bytes(ws_bytes, dev))
    rc = lib.argus_pair_intervals_ex(_ptr(events), n, _ptr(stream_offsets), S, num_regions, _ptr(out.intervals),
                                     out.interval_capacity, _ptr(out.interval_offsets), _ptr(out.ambig),
                                     out.ambig_capacity, _ptr(out.ambig_offsets), _ptr(out.status),
                                     _ptr(out.workspace), out.workspace.numel(), _stream_ptr(dev), kernel)
    if rc != 0:
        raise ArgusError(rc, "argus_pair_intervals")
    return out


def argus_pair_intervals_static(events: torch.Tensor, stream_offsets: torch.Tensor, num_regions: int,
                                interval_capacity: int | None = None, ambig_capacity: int | None = None) -> PairResult:
    """Pairing through the entry point that needs no workspace: for callers that cannot allocate device
    memory, its scratch is a fixed array inside the library (inputs up to 2^20 events, 4096 streams,
    2^16 ambiguity records). This wrapper still allocates the OUTPUT tensors with torch; a caller that
    cannot allocate passes its own buffers to the C function directly."""
    lib = load_library()
    dev = events.device
    n = events.numel() * events.element_size() // 16
    S = stream_offsets.numel() - 1
    icap = n // 2 if interval_capacity is None else int(interval_capacity)
    acap = min(n, 1 << 16) if ambig_capacity is None else int(ambig_capacity)
    out = PairResult(_bytes(icap * 48, dev), torch.empty(S + 1, dtype=torch.int64, device=dev), _bytes(acap * 32, dev),
                     torch.empty(S + 1, dtype=torch.int64, device=dev), _bytes(64, dev), icap, acap, _bytes(1, dev))
    rc = lib.argus_pair_intervals_static(_ptr(events), n, _ptr(stream_offsets), S, num_regions, _ptr(out.intervals), icap,
                                         _ptr(out.interval_offsets), _ptr(out.ambig), acap, _ptr(out.ambig_offsets),
                                         _ptr(out.status), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_pair_intervals_static")
    return out


@dataclass
class AggregateResult:
    warp: torch.Tensor | None    # uint8 [S * R * 576]
    cta: torch.Tensor | None
    sm: torch.Tensor | None
    kernel: torch.Tensor | None
    status: torch.Tensor
    workspace: torch.Tensor
    shape: dict

    def table_numpy(self, level: str) -> np.ndarray:
        t = getattr(self, level)
        keys, regions = self.shape[level]
        return t[: keys * regions * 576].cpu().numpy().view(AGG_DTYPE).reshape(self.shape[level])  # (a table without keys is empty)


def argus_aggregate(intervals: torch.Tensor, interval_offsets: torch.Tensor, ambig: torch.Tensor | None,
                    ambig_offsets: torch.Tensor | None, warps_per_cta: int, cta_sm: torch.Tensor, num_sms: int,
                    num_regions: int, levels=("warp", "cta", "sm", "kernel"),
                    out: AggregateResult | None = None) -> AggregateResult:
    lib = load_library()
    dev = intervals.device
    S = interval_offsets.numel() - 1
    C = S // warps_per_cta if warps_per_cta else 0
    keys = {"warp": S, "cta": C, "sm": num_sms, "kernel": 1}
    if out is None:
        tabs = {lv: (_bytes(keys[lv] * num_regions * 576, dev) if lv in levels else None) for lv in keys}
        ws = _bytes(lib.argus_aggregate_workspace_bytes(intervals.numel() // 48, S, num_regions), dev)
        out = AggregateResult(tabs["warp"], tabs["cta"], tabs["sm"], tabs["kernel"], _bytes(64, dev), ws,
                              {lv: (keys[lv], num_regions) for lv in keys})
    rc = lib.argus_aggregate(_ptr(intervals), _ptr(interval_offsets), _ptr(ambig), _ptr(ambig_offsets), S,
                             warps_per_cta, _ptr(cta_sm), num_sms, num_regions, _ptr(out.warp), _ptr(out.cta),
                             _ptr(out.sm), _ptr(out.kernel), _ptr(out.status), _ptr(out.workspace),
                             out.workspace.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_aggregate")
    return out


def argus_overlap(intervals: torch.Tensor, max_intervals: int, interval_offsets: torch.Tensor, warps_per_cta: int,
                  cta_sm: torch.Tensor, num_sms: int, pairs: torch.Tensor, workspace: torch.Tensor | None = None,
                  workspace_bytes: int | None = None):
    """pairs: device int32/uint32 [K, 2]. Returns (out uint8 [K * M * 32], status uint8 [64])."""
    lib = load_library()
    dev = intervals.device
    S = interval_offsets.numel() - 1
    K = pairs.numel() // 2
    if workspace is None:
        need = workspace_bytes if workspace_bytes is not None else lib.argus_overlap_workspace_bytes(max_intervals, S, K, num_sms)
        workspace = _bytes(need, dev)
    out = _bytes(K * num_sms * 32, dev)
    status = _bytes(64, dev)
    rc = lib.argus_overlap(_ptr(intervals), max_intervals, _ptr(interval_offsets), S, warps_per_cta, _ptr(cta_sm),
                           num_sms, _ptr(pairs), K, _ptr(out), _ptr(status), _ptr(workspace), workspace.numel(),
                           _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_overlap")
    return out, status


class _ScopeStruct(ctypes.Structure):  # argus_scope_t
    _fields_ = [("ctx_lo", ctypes.c_uint32), ("ctx_hi", ctypes.c_uint32), ("warp_mask", ctypes.c_uint64),
                ("sm_mask", ctypes.c_void_p), ("region_mask", ctypes.c_void_p)]


@dataclass
class ArgusScope:
    """argus_scope_t: which executions of a region count. `sm_mask` / `region_mask` are device int32
    tensors of ceil(n / 32) words (bit i of word i // 32), or None for "all"."""
    ctx_lo: int = 0
    ctx_hi: int = 0xFFFFFFFF
    warp_mask: int = 0xFFFFFFFFFFFFFFFF
    sm_mask: torch.Tensor | None = None
    region_mask: torch.Tensor | None = None

    @staticmethod
    def bitmask(selected, n: int, device) -> torch.Tensor:
        """Device mask of n bits with the bits in `selected` set (argument marshalling only)."""
        words = np.zeros((n + 31) // 32, dtype=np.uint32)
        for i in selected:
            words[int(i) // 32] |= np.uint32(1 << (int(i) % 32))
        return torch.from_numpy(words.view(np.int32)).to(device)

    def _struct(self) -> _ScopeStruct:
        return _ScopeStruct(self.ctx_lo, self.ctx_hi, self.warp_mask, _ptr(self.sm_mask), _ptr(self.region_mask))


@dataclass
class ScopedAggregateResult(AggregateResult):
    role: torch.Tensor | None = None   # uint8 [W * R * 576]
    iter: torch.Tensor | None = None   # uint8 [(ctx_hi - ctx_lo + 1) * R * 576]


def argus_aggregate_scoped(intervals: torch.Tensor, interval_offsets: torch.Tensor, ambig: torch.Tensor | None,
                           ambig_offsets: torch.Tensor | None, warps_per_cta: int, cta_sm: torch.Tensor, num_sms: int,
                           num_regions: int, scope: ArgusScope | None,
                           levels=("warp", "cta", "sm", "kernel", "role")) -> ScopedAggregateResult:
    """levels may also name "iter" (needs a scope; one row per ctx of its window)."""
    lib = load_library()
    dev = intervals.device
    S = interval_offsets.numel() - 1
    C = S // warps_per_cta if warps_per_cta else 0
    n_iter = scope.ctx_hi - scope.ctx_lo + 1 if (scope is not None and "iter" in levels) else 0
    keys = {"warp": S, "cta": C, "sm": num_sms, "kernel": 1, "role": warps_per_cta, "iter": max(n_iter, 0)}
    tabs = {lv: (_bytes(max(keys[lv], 1) * num_regions * 576, dev) if lv in levels else None) for lv in keys}
    ws = _bytes(lib.argus_aggregate_workspace_bytes(intervals.numel() // 48, S, num_regions), dev)
    out = ScopedAggregateResult(tabs["warp"], tabs["cta"], tabs["sm"], tabs["kernel"], _bytes(64, dev), ws,
                                {lv: (keys[lv], num_regions) for lv in keys}, tabs["role"], tabs["iter"])
    sc = scope._struct() if scope is not None else None
    rc = lib.argus_aggregate_scoped(_ptr(intervals), _ptr(interval_offsets), _ptr(ambig), _ptr(ambig_offsets), S,
                                    warps_per_cta, _ptr(cta_sm), num_sms, num_regions,
                                    ctypes.addressof(sc) if sc is not None else None, _ptr(out.warp), _ptr(out.cta),
                                    _ptr(out.sm), _ptr(out.kernel), _ptr(out.role), _ptr(out.iter), _ptr(out.status),
                                    _ptr(out.workspace), out.workspace.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_aggregate_scoped")
    return out


def argus_overlap_scoped(intervals: torch.Tensor, max_intervals: int, interval_offsets: torch.Tensor, warps_per_cta: int,
                         cta_sm: torch.Tensor, num_sms: int, pairs: torch.Tensor, scope: ArgusScope | None):
    """Returns (out uint8 [K * M * 32], status uint8 [64])."""
    lib = load_library()
    dev = intervals.device
    S = interval_offsets.numel() - 1
    K = pairs.numel() // 2
    workspace = _bytes(lib.argus_overlap_workspace_bytes(max_intervals, S, K, num_sms), dev)
    out = _bytes(K * num_sms * 32, dev)
    status = _bytes(64, dev)
    sc = scope._struct() if scope is not None else None
    rc = lib.argus_overlap_scoped(_ptr(intervals), max_intervals, _ptr(interval_offsets), S, warps_per_cta, _ptr(cta_sm),
                                  num_sms, _ptr(pairs), K, ctypes.addressof(sc) if sc is not None else None, _ptr(out),
                                  _ptr(status), _ptr(workspace), workspace.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_overlap_scoped")
    return out, status


def argus_map_pc_counts(intervals: torch.Tensor, interval_offsets: torch.Tensor, exec_region: int, num_pcs: int):
    """Returns (counts int64 tensor [(exec_region + 1), num_pcs] (bit pattern of u64), status uint8 [64])."""
    lib = load_library()
    dev = intervals.device
    S = interval_offsets.numel() - 1
    counts = torch.empty((exec_region + 1, num_pcs), dtype=torch.int64, device=dev)
    status = _bytes(64, dev)
    rc = lib.argus_map_pc_counts(_ptr(intervals), _ptr(interval_offsets), S, exec_region, num_pcs, _ptr(counts),
                                 _ptr(status), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_map_pc_counts")
    return counts, status


def argus_attribute(counts: torch.Tensor, metric: torch.Tensor, want_alpha: bool = True):
    """counts: int64 [rows, P] (u64 bit pattern); metric: float64 [P]. Returns (mhat [rows], entropy [P],
    alpha [rows, P] or None), float64 device tensors."""
    lib = load_library()
    dev = counts.device
    rows, P = counts.shape
    mhat = torch.empty(rows, dtype=torch.float64, device=dev)
    entropy = torch.empty(P, dtype=torch.float64, device=dev)
    alpha = torch.empty((rows, P), dtype=torch.float64, device=dev) if want_alpha else None
    ws = _bytes(lib.argus_attribute_workspace_bytes(rows, P), dev)
    rc = lib.argus_attribute(_ptr(counts), rows, P, _ptr(metric), _ptr(mhat), _ptr(entropy), _ptr(alpha), _ptr(ws),
                             ws.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_attribute")
    return mhat, entropy, alpha


JOIN_DTYPE = np.dtype([("count", "<u8"), ("sum", "<u8"), ("pct", "<u8", (5,)), ("max", "<u8")])  # argus_join_t


def argus_join_samples(reference: torch.Tensor, ref_index: torch.Tensor, samples: torch.Tensor):
    """reference, samples: uint8 tensors of 48-byte interval records; ref_index: int64 [Q].
    Returns (out uint8 [Q * 64] of argus_join_t, status uint8 [64])."""
    lib = load_library()
    dev = reference.device
    Q = ref_index.numel()
    out = _bytes(Q * 64, dev)
    status = _bytes(64, dev)
    rc = lib.argus_join_samples(_ptr(reference), reference.numel() // 48, _ptr(ref_index), Q, _ptr(samples),
                                samples.numel() // 48, _ptr(out), _ptr(status), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_join_samples")
    return out, status


def argus_join_samples_hashed(reference: torch.Tensor, ref_index: torch.Tensor, samples: torch.Tensor,
                              workspace: torch.Tensor | None = None):
    """As argus_join_samples, in one pass over `samples` for all queries together (samples in any order)."""
    lib = load_library()
    dev = reference.device
    Q = ref_index.numel()
    out = _bytes(Q * 64, dev)
    status = _bytes(64, dev)
    need = lib.argus_join_workspace_bytes(Q)
    if workspace is None:
        workspace = _bytes(max(need, 256), dev)
    rc = lib.argus_join_samples_hashed(_ptr(reference), reference.numel() // 48, _ptr(ref_index), Q, _ptr(samples),
                                       samples.numel() // 48, _ptr(out), _ptr(status), _ptr(workspace), workspace.numel(),
                                       _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_join_samples_hashed")
    return out, status


def argus_join_samples_grouped(reference: torch.Tensor, ref_index: torch.Tensor, samples: torch.Tensor,
                               sample_offsets: torch.Tensor, num_streams: int):
    """As argus_join_samples, with `samples` = the interval arrays of several probe runs one after the other and
    sample_offsets int64 [num_runs, S + 1] = where each stream's intervals of each run lie in `samples`."""
    lib = load_library()
    dev = reference.device
    Q = ref_index.numel()
    out = _bytes(Q * 64, dev)
    status = _bytes(64, dev)
    runs = sample_offsets.numel() // (num_streams + 1)
    rc = lib.argus_join_samples_grouped(_ptr(reference), reference.numel() // 48, _ptr(ref_index), Q, _ptr(samples),
                                        samples.numel() // 48, _ptr(sample_offsets), runs, num_streams, _ptr(out), _ptr(status),
                                        _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_join_samples_grouped")
    return out, status


def argus_ring_linearise(ring: torch.Tensor, slot_capacity: int, written: torch.Tensor, event_capacity: int | None = None):
    """ring: uint8 [S * slot_capacity * 16]; written: int64 [S] (records each stream ever wrote).
    Returns (events uint8 [event_capacity * 16], stream_offsets int64 [S + 1], dropped int64 [S], status)."""
    lib = load_library()
    dev = ring.device
    S = written.numel()
    cap = S * slot_capacity if event_capacity is None else int(event_capacity)
    events = _bytes(cap * 16, dev)
    offsets = torch.empty(S + 1, dtype=torch.int64, device=dev)
    dropped = torch.empty(max(S, 1), dtype=torch.int64, device=dev)
    status = _bytes(64, dev)
    rc = lib.argus_ring_linearise(_ptr(ring), slot_capacity, _ptr(written), S, _ptr(events), cap, _ptr(offsets),
                                  _ptr(dropped), _ptr(status), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_ring_linearise")
    return events, offsets, dropped[:S], status


def argus_pair_intervals_ring(ring: torch.Tensor, slot_capacity: int, written: torch.Tensor, num_regions: int,
                              interval_capacity: int | None = None, ambig_capacity: int | None = None):
    """Pairing straight from a ring container (see argus_ring_linearise for the layout), without the packed copy.
    Returns (PairResult, stream_offsets int64 [S + 1] of the packed form, dropped int64 [S])."""
    lib = load_library()
    dev = ring.device
    S = written.numel()
    bound = S * slot_capacity
    icap = bound // 2 if interval_capacity is None else int(interval_capacity)
    acap = bound if ambig_capacity is None else int(ambig_capacity)
    out = PairResult(_bytes(icap * 48, dev), torch.empty(S + 1, dtype=torch.int64, device=dev),
                     _bytes(acap * 32, dev), torch.empty(S + 1, dtype=torch.int64, device=dev),
                     _bytes(64, dev), icap, acap, _bytes(lib.argus_pair_workspace_bytes(bound, S, acap), dev))
    offsets = torch.empty(S + 1, dtype=torch.int64, device=dev)
    dropped = torch.empty(max(S, 1), dtype=torch.int64, device=dev)
    rc = lib.argus_pair_intervals_ring(_ptr(ring), slot_capacity, _ptr(written), S, num_regions, _ptr(offsets), _ptr(dropped),
                                       _ptr(out.intervals), out.interval_capacity, _ptr(out.interval_offsets), _ptr(out.ambig),
                                       out.ambig_capacity, _ptr(out.ambig_offsets), _ptr(out.status), _ptr(out.workspace),
                                       out.workspace.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_pair_intervals_ring")
    return out, offsets, dropped[:S]


@dataclass
class SynthesizeResult:
    pair: PairResult
    agg: AggregateResult
    overlap: torch.Tensor | None   # uint8 [K * M * 32]
    status: torch.Tensor
    workspace: torch.Tensor
    max_overlap_spans: int

    def fetch_status(self):
        return argus_status_fetch(self.status)

    def overlap_numpy(self, num_sms: int) -> np.ndarray:
        return self.overlap.cpu().numpy().view(OVERLAP_DTYPE).reshape(-1, num_sms)


def argus_synthesize_workspace_bytes(num_events: int, num_streams: int, num_regions: int, ambig_capacity: int,
                                     num_pairs: int, num_sms: int, max_overlap_spans: int) -> int:
    lib = load_library()
    return lib.argus_synthesize_workspace_bytes(num_events, num_streams, num_regions, ambig_capacity, num_pairs, num_sms,
                                                max_overlap_spans)


def _synthesize_buffers(dev, n, S, K, num_regions, warps_per_cta, num_sms, interval_capacity, ambig_capacity, max_overlap_spans,
                        levels) -> SynthesizeResult:
    """Output tensors and workspace of the one-call pipeline for a trace of at most n events."""
    icap = n // 2 if interval_capacity is None else int(interval_capacity)
    acap = n if ambig_capacity is None else int(ambig_capacity)
    mos = (2 * K * icap if max_overlap_spans is None else int(max_overlap_spans)) if K else 0
    C = S // warps_per_cta if warps_per_cta else 0
    keys = {"warp": S, "cta": C, "sm": num_sms, "kernel": 1}
    tabs = {lv: (_bytes(keys[lv] * num_regions * 576, dev) if lv in levels else None) for lv in keys}
    status = _bytes(64, dev)
    pr = PairResult(_bytes(icap * 48, dev), torch.empty(S + 1, dtype=torch.int64, device=dev), _bytes(acap * 32, dev),
                    torch.empty(S + 1, dtype=torch.int64, device=dev), status, icap, acap, _bytes(1, dev))
    ag = AggregateResult(tabs["warp"], tabs["cta"], tabs["sm"], tabs["kernel"], status, _bytes(1, dev),
                         {lv: (keys[lv], num_regions) for lv in keys})
    ws = _bytes(argus_synthesize_workspace_bytes(n, S, num_regions, acap, K, num_sms, mos), dev)
    return SynthesizeResult(pr, ag, _bytes(K * num_sms * 32, dev) if K else None, status, ws, mos)


def argus_synthesize_ring(ring: torch.Tensor, slot_capacity: int, written: torch.Tensor, num_regions: int, warps_per_cta: int,
                          cta_sm: torch.Tensor, num_sms: int, pairs: torch.Tensor | None = None,
                          interval_capacity: int | None = None, ambig_capacity: int | None = None,
                          max_overlap_spans: int | None = None, levels=("warp", "cta", "sm", "kernel")):
    """The one-call pipeline on a ring container (see argus_ring_linearise for the layout).
    Returns (SynthesizeResult, stream_offsets int64 [S + 1] of the packed form, dropped int64 [S])."""
    lib = load_library()
    dev = ring.device
    S = written.numel()
    K = 0 if pairs is None else pairs.numel() // 2
    out = _synthesize_buffers(dev, S * slot_capacity, S, K, num_regions, warps_per_cta, num_sms, interval_capacity,
                              ambig_capacity, max_overlap_spans, levels)
    offsets = torch.empty(S + 1, dtype=torch.int64, device=dev)
    dropped = torch.empty(max(S, 1), dtype=torch.int64, device=dev)
    p, a = out.pair, out.agg
    rc = lib.argus_synthesize_ring(_ptr(ring), slot_capacity, _ptr(written), S, num_regions, _ptr(offsets), _ptr(dropped),
                                   _ptr(p.intervals), p.interval_capacity, _ptr(p.interval_offsets), _ptr(p.ambig),
                                   p.ambig_capacity, _ptr(p.ambig_offsets), warps_per_cta, _ptr(cta_sm), num_sms, _ptr(a.warp),
                                   _ptr(a.cta), _ptr(a.sm), _ptr(a.kernel), _ptr(pairs), K, _ptr(out.overlap),
                                   out.max_overlap_spans, _ptr(out.status), _ptr(out.workspace), out.workspace.numel(),
                                   _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_synthesize_ring")
    return out, offsets, dropped[:S]


def argus_synthesize(events: torch.Tensor, stream_offsets: torch.Tensor, num_regions: int, warps_per_cta: int,
                     cta_sm: torch.Tensor, num_sms: int, pairs: torch.Tensor | None = None,
                     interval_capacity: int | None = None, ambig_capacity: int | None = None,
                     max_overlap_spans: int | None = None, levels=("warp", "cta", "sm", "kernel"),
                     out: SynthesizeResult | None = None) -> SynthesizeResult:
    """Whole hot path in one call (pair -> aggregate -> overlap); enqueues on the current stream."""
    lib = load_library()
    dev = events.device
    n = events.numel() * events.element_size() // 16
    S = stream_offsets.numel() - 1
    K = 0 if pairs is None else pairs.numel() // 2
    if out is None:
        out = _synthesize_buffers(dev, n, S, K, num_regions, warps_per_cta, num_sms, interval_capacity, ambig_capacity,
                                  max_overlap_spans, levels)
    p, a = out.pair, out.agg
    rc = lib.argus_synthesize(_ptr(events), n, _ptr(stream_offsets), S, num_regions, _ptr(p.intervals), p.interval_capacity,
                              _ptr(p.interval_offsets), _ptr(p.ambig), p.ambig_capacity, _ptr(p.ambig_offsets), warps_per_cta,
                              _ptr(cta_sm), num_sms, _ptr(a.warp), _ptr(a.cta), _ptr(a.sm), _ptr(a.kernel), _ptr(pairs), K,
                              _ptr(out.overlap), out.max_overlap_spans, _ptr(out.status), _ptr(out.workspace),
                              out.workspace.numel(), _stream_ptr(dev))
    if rc != 0:
        raise ArgusError(rc, "argus_synthesize")
    return out
