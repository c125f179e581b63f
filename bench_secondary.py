"""Timings of the entry points beyond the benchmark's step, on one GPU, with CUDA events (the secondary
suite of bench.py):

    python bench.py --suite secondary --what scoped   # argus_aggregate_scoped / argus_overlap_scoped on trace 3
    python bench.py --suite secondary --what pcmap    # PC-to-region mapping and attribution on a mapping run
    python bench.py --suite secondary --what ring     # pairing from a ring container: packed copy first, or directly
    python bench.py --suite secondary --what join     # cross-run join against a whole trace: per query, grouped, hashed

Each line printed is one JSON object: what ran, its time (best of the repetitions after warm-up), the
algorithmic bytes it has to move and the fraction of the measured HBM copy bandwidth that amounts to.
Inputs are synthetic and generated on the device; they are larger than the 126 MB L2.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

import paper_2609_12299_b200.binding as argus
from paper_2609_12299_b200 import tracegen as tg
from paper_2609_12299_b200.tracegen.mapping import mapping_trace

_ROOT = os.path.dirname(os.path.abspath(__file__))


def _peak_gbs() -> float:
    path = os.path.join(_ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"])
    return 6650.0


def _time(fn, reps=5, warmup=2):
    best = float("inf")
    for i in range(warmup + reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        torch.cuda.synchronize()
        if i >= warmup:
            best = min(best, e0.elapsed_time(e1))
        del out
    return best


def _line(what, ms, alg_bytes, **extra):
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    print(json.dumps({"what": what, "ms": round(ms, 4), "algorithmic_bytes": int(alg_bytes), "achieved_GBps": round(gbs, 1),
                      "frac_of_measured_hbm": round(gbs / _peak_gbs(), 4), **extra}), flush=True)


def run_scoped(iters: int):
    spec = tg.config(3).scaled(iters=iters) if iters else tg.config(3)
    dev = torch.device("cuda", 0)
    d_ev, d_off = tg.generate_cuda(spec, dev)
    n = d_ev.numel() // 16
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(dev)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(dev)
    W, R, M = spec.warps_per_cta, spec.num_regions, spec.num_sms
    p = argus.argus_pair_intervals(d_ev, d_off, R, interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096))
    assert int(p.fetch_status()["code"]) == 0
    del d_ev
    torch.cuda.empty_cache()
    iv_bytes = p.intervals.numel()
    lo = spec.iters // 2
    args = (p.intervals, p.interval_offsets, p.ambig, p.ambig_offsets, W, cta_sm, M, R)
    cases = [
        ("argus_aggregate (four levels, nothing filtered)", lambda: argus.argus_aggregate(*args), 1.0),
        ("argus_aggregate_scoped, scope = everything, + role table", lambda: argus.argus_aggregate_scoped(*args, None), 1.0),
        ("argus_aggregate_scoped, 16 iterations, 3 of 16 warp roles, 4 regions, + role and iteration tables",
         lambda: argus.argus_aggregate_scoped(*args, argus.ArgusScope(lo, lo + 15, 0b100011, None,
                                                                      argus.ArgusScope.bitmask(range(4), R, dev)),
                                              levels=("kernel", "role", "iter")), 3.0 / 16.0),
        ("argus_aggregate_scoped, 16 iterations of all regions, + role and iteration tables (iteration table by global atomics)",
         lambda: argus.argus_aggregate_scoped(*args, argus.ArgusScope(lo, lo + 15),
                                              levels=("warp", "cta", "sm", "kernel", "role", "iter")), 1.0),
        ("argus_overlap_scoped, 16 iterations", lambda: argus.argus_overlap_scoped(p.intervals, n // 2, p.interval_offsets, W,
                                                                                   cta_sm, M, pairs,
                                                                                   argus.ArgusScope(lo, lo + 15)), 1.0),
    ]
    for what, fn, passes in cases:
        _line(what, _time(fn), iv_bytes * passes, intervals=iv_bytes // 48, workload=spec.name,
              note="algorithmic bytes = interval bytes of the streams the scope reads x passes over them")


def run_pcmap(iters: int, num_pcs: int, execs_per_begin: int):
    spec = tg.config(3).scaled(iters=iters)
    dev = torch.device("cuda", 0)
    d_ev, d_off = tg.generate_cuda(spec, dev)
    R = spec.num_regions
    m_ev, m_off = mapping_trace(d_ev, d_off, R, num_pcs, execs_per_begin)
    del d_ev
    torch.cuda.empty_cache()
    n = m_ev.numel() // 16
    state = {}

    def pair():
        state["p"] = argus.argus_pair_intervals(m_ev, m_off, R + 1, interval_capacity=n // 2, ambig_capacity=4096,
                                                out=state.get("p"))
        return None

    ms_pair = _time(pair)
    p = state["p"]
    assert int(p.fetch_status()["code"]) == 0
    _line("argus_pair_intervals on the mapping run (whole call)", ms_pair, 40.0 * n, events=n, workload="decode mapping run",
          regions=R + 1, pcs=num_pcs)
    ms_map = _time(lambda: argus.argus_map_pc_counts(p.intervals, p.interval_offsets, R, num_pcs))
    counts, status = argus.argus_map_pc_counts(p.intervals, p.interval_offsets, R, num_pcs)
    assert int(argus.argus_status_fetch(status)["code"]) == 0
    n_exec = int((counts != 0).sum().item())
    _line("argus_map_pc_counts (counts cleared, then one pass over the intervals)", ms_map,
          24.0 * n + (R + 1) * num_pcs * 8, intervals=n // 2, nonzero_cells=n_exec)
    metric = torch.rand(num_pcs, dtype=torch.float64, device=dev)
    ms_attr = _time(lambda: argus.argus_attribute(counts, metric, want_alpha=True))
    _line("argus_attribute with alpha output", ms_attr, (R + 1) * num_pcs * 16 + num_pcs * 16, rows=R + 1, pcs=num_pcs)
    ms_attr2 = _time(lambda: argus.argus_attribute(counts, metric, want_alpha=False))
    _line("argus_attribute without alpha output", ms_attr2, (R + 1) * num_pcs * 8 + num_pcs * 16, rows=R + 1, pcs=num_pcs)


def run_ring(iters: int, shift_tokens: int):
    """Trace 3 held in a ring container (one slot per stream, exactly as long as the stream): pairing after
    argus_ring_linearise against argus_pair_intervals_ring, which reads the slots directly."""
    spec = tg.config(3).scaled(iters=iters) if iters else tg.config(3)
    dev = torch.device("cuda", 0)
    d_ev, d_off = tg.generate_cuda(spec, dev)
    n = d_ev.numel() // 16
    S = spec.num_streams
    cap = n // S                                      # every stream of this trace has the same length
    shift = (cap // spec.iters) * shift_tokens        # records written before the survivors: a whole number of tokens
    written = torch.full((S,), cap + shift, dtype=torch.int64, device=dev)
    R = spec.num_regions
    state = {}

    def two_steps():
        ev, offs, _, st = argus.argus_ring_linearise(d_ev, cap, written)
        state["p"] = argus.argus_pair_intervals(ev, offs, R, interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096),
                                                out=state.get("p"))
        return ev

    ms2 = _time(two_steps, reps=3, warmup=1)
    st = state["p"].fetch_status()
    assert int(st["code"]) == 0, st
    _line("argus_ring_linearise + argus_pair_intervals", ms2, 72.0 * n, events=n, workload=spec.name, shift_records=shift,
          sequential_tiles=int(st["n_sequential_tiles"]), note="algorithmic bytes: 32 B/event for the copy + 40 B/event for pairing")
    del state["p"]
    torch.cuda.empty_cache()
    ms1 = _time(lambda: argus.argus_pair_intervals_ring(d_ev, cap, written, R, interval_capacity=n // 2,
                                                         ambig_capacity=max(n // 64, 4096)), reps=3, warmup=1)
    pr, _, _ = argus.argus_pair_intervals_ring(d_ev, cap, written, R, interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096))
    st = pr.fetch_status()
    assert int(st["code"]) == 0, st
    _line("argus_pair_intervals_ring (allocations included)", ms1, 40.0 * n, events=n, workload=spec.name, shift_records=shift,
          sequential_tiles=int(st["n_sequential_tiles"]))
    del pr
    torch.cuda.empty_cache()
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(dev)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(dev)
    kw = dict(interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096), max_overlap_spans=n // 8)
    ms3 = _time(lambda: argus.argus_synthesize_ring(d_ev, cap, written, R, spec.warps_per_cta, cta_sm, spec.num_sms, pairs, **kw),
                reps=3, warmup=1)
    res, _, _ = argus.argus_synthesize_ring(d_ev, cap, written, R, spec.warps_per_cta, cta_sm, spec.num_sms, pairs, **kw)
    assert int(res.fetch_status()["code"]) == 0
    _line("argus_synthesize_ring (allocations included)", ms3, 40.0 * n, events=n, workload=spec.name, shift_records=shift)


def run_join(iters: int, queries: int):
    """Cross-run join on the decode trace: the run's own intervals serve as reference and as one probe run."""
    spec = tg.config(3).scaled(iters=iters) if iters else tg.config(3)
    dev = torch.device("cuda", 0)
    d_ev, d_off = tg.generate_cuda(spec, dev)
    n = d_ev.numel() // 16
    p = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions, interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096))
    assert int(p.fetch_status()["code"]) == 0
    del d_ev
    torch.cuda.empty_cache()
    n_iv = int(p.interval_offsets[-1].item())
    iv = p.intervals[: n_iv * 48]
    g = torch.Generator(device="cpu").manual_seed(7)
    idx = torch.randint(0, n_iv, (queries,), generator=g, dtype=torch.int64).to(dev)
    few = idx[:8].contiguous()
    ms = _time(lambda: argus.argus_join_samples(iv, few, iv), reps=2, warmup=1)
    _line("argus_join_samples, 8 queries (every query reads the 32 key bytes of every sample)", ms, 8 * 32.0 * n_iv,
          intervals=n_iv, workload=spec.name)
    offs = p.interval_offsets.view(1, -1).contiguous()
    ms = _time(lambda: argus.argus_join_samples_grouped(iv, idx, iv, offs, spec.num_streams), reps=3, warmup=1)
    _line(f"argus_join_samples_grouped, {queries} queries (every query reads its own stream's samples)", ms,
          queries * 32.0 * n_iv / spec.num_streams, intervals=n_iv, workload=spec.name)
    ws = torch.empty(argus.load_library().argus_join_workspace_bytes(queries), dtype=torch.uint8, device=dev)
    ms = _time(lambda: argus.argus_join_samples_hashed(iv, idx, iv, ws), reps=3, warmup=1)
    _line(f"argus_join_samples_hashed, {queries} queries (one pass over the samples in whatever order they lie)", ms,
          48.0 * n_iv, intervals=n_iv, workload=spec.name)


def run(what: str, iters: int = 0, queries: int = 2000, shift_tokens: int = 100, pcs: int = 70_560, execs_per_begin: int = 2):
    argus.load_library()
    if what == "scoped":
        run_scoped(iters)
    elif what == "ring":
        run_ring(iters, shift_tokens)
    elif what == "join":
        run_join(iters, queries)
    elif what == "pcmap":
        run_pcmap(iters or 24, pcs, execs_per_begin)
    else:
        raise ValueError(what)
