"""ctypes loader of the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package; the product never does. Record layouts are retyped here, independently of the CUDA
binding. See oracle.h for what each function computes and which paper passages it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))

EVENT = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4")])
INTERVAL = np.dtype([("t_begin", "<u8"), ("inclusive", "<u8"), ("exclusive", "<u8"), ("region", "<u4"),
                     ("ctx", "<u4"), ("stream", "<u4"), ("parent_region", "<u4"), ("begin_idx", "<u4"),
                     ("depth", "<u2"), ("flags", "<u2")])
AMBIG = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4"), ("stream", "<u4"), ("event_idx", "<u4"),
                  ("kind", "<u4"), ("depth", "<u4")])
AGG = np.dtype([("count", "<u8"), ("sum_incl", "<u8"), ("min_incl", "<u8"), ("max_incl", "<u8"),
                ("sum_excl", "<u8"), ("n_unmatched_begin", "<u8"), ("n_unmatched_end", "<u8"),
                ("n_flagged", "<u8"), ("hist", "<u8", (64,))])
OVERLAP = np.dtype([("overlap_ns", "<u8"), ("producer_ns", "<u8"), ("consumer_ns", "<u8"), ("either_ns", "<u8")])
STATUS = np.dtype([("code", "<u4"), ("bad_stream", "<u4"), ("bad_event", "<u8"), ("intervals_required", "<u8"),
                   ("ambig_required", "<u8"), ("n_ctx_mismatch", "<u8"), ("n_time_reversed", "<u8"),
                   ("n_child_clamped", "<u8"), ("reserved", "<u8")])
assert (EVENT.itemsize, INTERVAL.itemsize, AMBIG.itemsize, AGG.itemsize, OVERLAP.itemsize, STATUS.itemsize) == \
    (16, 48, 32, 576, 32, 64)

NONE = 0xFFFFFFFF


def build(force: bool = False) -> str:
    """Compiles oracle.cpp into liboracle.so next to it (g++, -O2)."""
    src = os.path.join(_HERE, "oracle.cpp")
    out = os.path.join(_HERE, "liboracle.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < max(
            os.path.getmtime(src), os.path.getmtime(os.path.join(_HERE, "oracle.h"))):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", out, src])
    return out


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, u32, u64 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64
        lib.oracle_pair.argtypes = [vp, vp, u32, u32, vp, u64, vp, vp, u64, vp, vp]
        lib.oracle_aggregate.argtypes = [vp, vp, vp, vp, u32, u32, vp, u32, u32, vp, vp, vp, vp, vp]
        lib.oracle_overlap.argtypes = [vp, vp, u32, u32, vp, u32, vp, u32, vp, vp]
        lib.oracle_aggregate_scoped.argtypes = [vp, vp, vp, vp, u32, u32, vp, u32, u32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_overlap_scoped.argtypes = [vp, vp, u32, u32, vp, u32, vp, u32, vp, vp, vp]
        lib.oracle_ring_linearise.argtypes = [vp, u32, vp, u32, vp, u64, vp, vp, vp]
        lib.oracle_ring_linearise.restype = ctypes.c_int
        lib.oracle_join_samples.argtypes = [vp, u64, vp, u32, vp, u64, vp, vp]
        lib.oracle_join_samples.restype = ctypes.c_int
        lib.oracle_map_pc_counts.argtypes = [vp, vp, u32, u32, u32, vp, vp]
        lib.oracle_attribute.argtypes = [vp, u32, u32, vp, vp, vp, vp]
        for f in (lib.oracle_pair, lib.oracle_aggregate, lib.oracle_overlap, lib.oracle_aggregate_scoped,
                  lib.oracle_overlap_scoped, lib.oracle_map_pc_counts, lib.oracle_attribute):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data


def pair(events: np.ndarray, stream_offsets: np.ndarray, num_regions: int, interval_cap: int | None = None,
         ambig_cap: int | None = None):
    """Returns (rc, intervals, interval_offsets, ambig, ambig_offsets, status)."""
    events = np.ascontiguousarray(events, dtype=EVENT)
    offs = np.ascontiguousarray(stream_offsets, dtype=np.uint64)
    S = len(offs) - 1
    n = len(events)
    icap = n // 2 if interval_cap is None else interval_cap
    acap = n if ambig_cap is None else ambig_cap
    iv = np.zeros(icap, dtype=INTERVAL)
    am = np.zeros(acap, dtype=AMBIG)
    ioffs = np.zeros(S + 1, dtype=np.uint64)
    aoffs = np.zeros(S + 1, dtype=np.uint64)
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_pair(_ptr(events), _ptr(offs), S, num_regions, _ptr(iv), icap, _ptr(ioffs), _ptr(am), acap,
                             _ptr(aoffs), _ptr(st))
    ni = min(int(ioffs[S]), icap)
    na = min(int(aoffs[S]), acap)
    return rc, iv[:ni], ioffs, am[:na], aoffs, st[0]


def aggregate(intervals, interval_offsets, ambig, ambig_offsets, warps_per_cta, cta_sm, num_sms, num_regions,
              levels=("warp", "cta", "sm", "kernel")):
    """Returns (rc, {level: table [keys, R]}, status)."""
    iv = np.ascontiguousarray(intervals, dtype=INTERVAL)
    ioffs = np.ascontiguousarray(interval_offsets, dtype=np.uint64)
    S = len(ioffs) - 1
    am = None if ambig is None else np.ascontiguousarray(ambig, dtype=AMBIG)
    aoffs = None if ambig_offsets is None else np.ascontiguousarray(ambig_offsets, dtype=np.uint64)
    cs = np.ascontiguousarray(cta_sm, dtype=np.uint32)
    C = S // warps_per_cta if warps_per_cta else 0
    keys = {"warp": S, "cta": C, "sm": num_sms, "kernel": 1}
    tabs = {lv: (np.zeros((keys[lv], num_regions), dtype=AGG) if lv in levels else None) for lv in keys}
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_aggregate(_ptr(iv), _ptr(ioffs), _ptr(am), _ptr(aoffs), S, warps_per_cta, _ptr(cs), num_sms,
                                  num_regions, _ptr(tabs["warp"]), _ptr(tabs["cta"]), _ptr(tabs["sm"]),
                                  _ptr(tabs["kernel"]), _ptr(st))
    return rc, {k: v for k, v in tabs.items() if v is not None}, st[0]


def overlap(intervals, interval_offsets, warps_per_cta, cta_sm, num_sms, pairs):
    """Returns (rc, out [K, M], status)."""
    iv = np.ascontiguousarray(intervals, dtype=INTERVAL)
    ioffs = np.ascontiguousarray(interval_offsets, dtype=np.uint64)
    S = len(ioffs) - 1
    cs = np.ascontiguousarray(cta_sm, dtype=np.uint32)
    pr = np.ascontiguousarray(pairs, dtype=np.uint32).reshape(-1, 2)
    out = np.zeros((len(pr), num_sms), dtype=OVERLAP)
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_overlap(_ptr(iv), _ptr(ioffs), S, warps_per_cta, _ptr(cs), num_sms, _ptr(pr), len(pr),
                                _ptr(out), _ptr(st))
    return rc, out, st[0]


class _OScope(ctypes.Structure):
    _fields_ = [("ctx_lo", ctypes.c_uint32), ("ctx_hi", ctypes.c_uint32), ("warp_mask", ctypes.c_uint64),
                ("sm_mask", ctypes.c_void_p), ("region_mask", ctypes.c_void_p)]


def _bitmask(selected, n):
    """Bit i of word i // 32 set for every i in `selected` (an iterable of indices < n)."""
    words = np.zeros((n + 31) // 32, dtype=np.uint32)
    for i in selected:
        assert 0 <= int(i) < n
        words[int(i) // 32] |= np.uint32(1 << (int(i) % 32))
    return words


def _scope_struct(scope, num_sms, num_regions):
    """scope: None or a dict with optional keys ctx (lo, hi), warps (indices inside a CTA), sms, regions.
    Returns (struct or None, arrays to keep alive)."""
    if scope is None:
        return None, ()
    lo, hi = scope.get("ctx", (0, 0xFFFFFFFF))
    warps = scope.get("warps")
    wm = 0xFFFFFFFFFFFFFFFF if warps is None else sum(1 << int(w) for w in set(warps))
    sm = None if scope.get("sms") is None else _bitmask(scope["sms"], num_sms)
    rg = None if scope.get("regions") is None else _bitmask(scope["regions"], num_regions)
    return _OScope(int(lo), int(hi), wm, _ptr(sm), _ptr(rg)), (sm, rg)


def aggregate_scoped(intervals, interval_offsets, ambig, ambig_offsets, warps_per_cta, cta_sm, num_sms, num_regions,
                     scope=None, levels=("warp", "cta", "sm", "kernel", "role", "iter")):
    """Returns (rc, {level: table [keys, R]}, status); level "iter" needs a scope with a ctx window."""
    iv = np.ascontiguousarray(intervals, dtype=INTERVAL)
    ioffs = np.ascontiguousarray(interval_offsets, dtype=np.uint64)
    S = len(ioffs) - 1
    am = None if ambig is None else np.ascontiguousarray(ambig, dtype=AMBIG)
    aoffs = None if ambig_offsets is None else np.ascontiguousarray(ambig_offsets, dtype=np.uint64)
    cs = np.ascontiguousarray(cta_sm, dtype=np.uint32)
    C = S // warps_per_cta if warps_per_cta else 0
    sc, keep = _scope_struct(scope, num_sms, num_regions)
    n_iter = 0
    if "iter" in levels and scope is not None and "ctx" in scope:
        n_iter = int(scope["ctx"][1]) - int(scope["ctx"][0]) + 1
        if tuple(int(x) for x in scope["ctx"]) == (0, 0xFFFFFFFF):
            n_iter = 0       # the all-selecting window: no iteration table
        elif n_iter > 65536:
            n_iter = 1       # too many rows: the call is refused before it touches the table
    keys = {"warp": S, "cta": C, "sm": num_sms, "kernel": 1, "role": warps_per_cta, "iter": n_iter}
    tabs = {lv: (np.zeros((keys[lv], num_regions), dtype=AGG) if lv in levels and (lv != "iter" or n_iter > 0) else None)
            for lv in keys}
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_aggregate_scoped(_ptr(iv), _ptr(ioffs), _ptr(am), _ptr(aoffs), S, warps_per_cta, _ptr(cs), num_sms,
                                         num_regions, None if sc is None else ctypes.addressof(sc), _ptr(tabs["warp"]),
                                         _ptr(tabs["cta"]), _ptr(tabs["sm"]), _ptr(tabs["kernel"]), _ptr(tabs["role"]),
                                         _ptr(tabs["iter"]), _ptr(st))
    del keep
    return rc, {k: v for k, v in tabs.items() if v is not None}, st[0]


def overlap_scoped(intervals, interval_offsets, warps_per_cta, cta_sm, num_sms, pairs, scope=None, num_regions=65536):
    """Returns (rc, out [K, M], status)."""
    iv = np.ascontiguousarray(intervals, dtype=INTERVAL)
    ioffs = np.ascontiguousarray(interval_offsets, dtype=np.uint64)
    S = len(ioffs) - 1
    cs = np.ascontiguousarray(cta_sm, dtype=np.uint32)
    pr = np.ascontiguousarray(pairs, dtype=np.uint32).reshape(-1, 2)
    out = np.zeros((len(pr), num_sms), dtype=OVERLAP)
    st = np.zeros(1, dtype=STATUS)
    sc, keep = _scope_struct(scope, num_sms, num_regions)
    rc = _load().oracle_overlap_scoped(_ptr(iv), _ptr(ioffs), S, warps_per_cta, _ptr(cs), num_sms, _ptr(pr), len(pr),
                                       None if sc is None else ctypes.addressof(sc), _ptr(out), _ptr(st))
    del keep
    return rc, out, st[0]


MAP_EVENT = np.dtype([("kind", "<u4"), ("id", "<u4"), ("count", "<u8")])  # kind 0 begin, 1 end, 2 exec
assert MAP_EVENT.itemsize == 16


def map_pc_counts(map_events, stream_offsets, num_regions, num_pcs):
    """Returns (rc, counts [(R + 1), P] uint64, status); row R = outside every region."""
    ev = np.ascontiguousarray(map_events, dtype=MAP_EVENT)
    offs = np.ascontiguousarray(stream_offsets, dtype=np.uint64)
    counts = np.zeros((num_regions + 1, num_pcs), dtype=np.uint64)
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_map_pc_counts(_ptr(ev), _ptr(offs), len(offs) - 1, num_regions, num_pcs, _ptr(counts), _ptr(st))
    return rc, counts, st[0]


def attribute(counts, metric, want_alpha=True):
    """Returns (rc, mhat [rows], entropy [P], alpha [rows, P] or None), all float64."""
    n = np.ascontiguousarray(counts, dtype=np.uint64)
    rows, P = n.shape
    m = np.ascontiguousarray(metric, dtype=np.float64)
    mhat, ent = np.zeros(rows, np.float64), np.zeros(P, np.float64)
    alpha = np.zeros((rows, P), np.float64) if want_alpha else None
    rc = _load().oracle_attribute(_ptr(n), rows, P, _ptr(m), _ptr(mhat), _ptr(ent), _ptr(alpha))
    return rc, mhat, ent, alpha


JOIN = np.dtype([("count", "<u8"), ("sum", "<u8"), ("pct", "<u8", (5,)), ("max", "<u8")])
assert JOIN.itemsize == 64


def join_samples(reference, ref_index, samples):
    """Returns (rc, out [Q] of JOIN, status)."""
    ref = np.ascontiguousarray(reference, dtype=INTERVAL)
    idx = np.ascontiguousarray(ref_index, dtype=np.uint64)
    smp = np.ascontiguousarray(samples, dtype=INTERVAL)
    out = np.zeros(len(idx), dtype=JOIN)
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_join_samples(_ptr(ref), len(ref), _ptr(idx), len(idx), _ptr(smp), len(smp), _ptr(out), _ptr(st))
    return rc, out, st[0]


def ring_linearise(ring, slot_capacity, written, event_capacity=None):
    """ring: EVENT array [S * slot_capacity]; written: [S]. Returns (rc, events, stream_offsets, dropped, status)."""
    rg = np.ascontiguousarray(ring, dtype=EVENT)
    wr = np.ascontiguousarray(written, dtype=np.uint64)
    S = len(wr)
    cap = int(np.minimum(wr, slot_capacity).sum()) if event_capacity is None else int(event_capacity)
    ev = np.zeros(max(cap, 1), dtype=EVENT)
    offs = np.zeros(S + 1, dtype=np.uint64)
    dropped = np.zeros(max(S, 1), dtype=np.uint64)
    st = np.zeros(1, dtype=STATUS)
    rc = _load().oracle_ring_linearise(_ptr(rg), slot_capacity, _ptr(wr), S, _ptr(ev), cap, _ptr(offs), _ptr(dropped), _ptr(st))
    return rc, ev[:int(offs[-1])] if int(offs[-1]) <= cap else ev[:0], offs, dropped[:S], st[0]
