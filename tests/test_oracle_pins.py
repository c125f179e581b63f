"""Pins of the CPU oracle against things other than itself: hand-worked examples (tests/golden),
brute-force enumeration of pairings, closed forms for well-formed streams, library routines
(numpy group-by, tick counting) and invariants. No GPU needed."""
import itertools

import numpy as np
import pytest

import oracle
from helpers import (NONE, ambig_tuples, closed_form_wellformed, enumerate_matchings, interval_tuples, load_example,
                     make_events, random_wellformed, single_stream)
from paper_2609_12299_b200 import tracegen as tg

EXAMPLES = ["example_a_wellformed.txt", "example_b_dropped_end.txt", "example_c_dup_stray_trunc.txt",
            "example_e_ctx_ignored.txt", "example_f_greedy.txt", "example_g_boundary.txt", "example_h_flags.txt"]


@pytest.mark.parametrize("name", EXAMPLES)
def test_hand_worked_examples(name):
    ev, want_iv, want_am = load_example(name)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, single_stream(ev), 8)
    assert rc == 0 and st["code"] == 0
    assert interval_tuples(iv) == want_iv
    assert ambig_tuples(am) == want_am
    assert list(ioffs) == [0, len(want_iv)] and list(aoffs) == [0, len(want_am)]
    assert all(int(r["stream"]) == 0 for r in iv) and all(int(r["stream"]) == 0 for r in am)
    # the ambiguity record repeats the marker itself
    for r in am:
        e = ev[int(r["event_idx"])]
        assert (int(r["ts"]), int(r["tag"]), int(r["ctx"])) == (int(e["ts"]), int(e["tag"]), int(e["ctx"]))


def test_example_a_aggregates():
    ev, _, _ = load_example("example_a_wellformed.txt")
    _, iv, ioffs, am, aoffs, _ = oracle.pair(ev, single_stream(ev), 3)
    rc, tabs, st = oracle.aggregate(iv, ioffs, am, aoffs, 1, np.array([0], np.uint32), 1, 3)
    assert rc == 0
    k = tabs["kernel"][0]
    want = {0: (1, 30, 30, 30, 14, {4: 1}), 1: (2, 16, 8, 8, 16, {3: 2}), 2: (1, 0, 0, 0, 0, {0: 1})}
    for r, (count, s, mn, mx, ex, hist) in want.items():
        assert (int(k[r]["count"]), int(k[r]["sum_incl"]), int(k[r]["min_incl"]), int(k[r]["max_incl"]),
                int(k[r]["sum_excl"])) == (count, s, mn, mx, ex)
        h = np.zeros(64, np.uint64)
        for b, c in hist.items():
            h[b] = c
        assert np.array_equal(k[r]["hist"], h)
    # one stream, one CTA, one SM: every level holds the same numbers
    for lv in ("warp", "cta", "sm"):
        assert tabs[lv][0].tobytes() == k.tobytes()


def test_example_d_overlap():
    spans, expect = [], None
    import os
    from helpers import GOLDEN
    for line in open(os.path.join(GOLDEN, "example_d_overlap.txt")):
        tok = line.split()
        if tok and tok[0] == "span":
            spans.append(tuple(int(x) for x in tok[1:]))
        elif tok and tok[0] == "expect":
            expect = tuple(int(x) for x in tok[1:])
    nstreams = 3
    iv = np.zeros(len(spans), dtype=oracle.INTERVAL)
    spans.sort(key=lambda s: s[0])
    for i, (s, region, t, incl) in enumerate(spans):
        iv[i]["stream"], iv[i]["region"], iv[i]["t_begin"], iv[i]["inclusive"] = s, region, t, incl
    ioffs = np.zeros(nstreams + 1, np.uint64)
    for s, *_ in spans:
        ioffs[s + 1:] += 1
    rc, out, st = oracle.overlap(iv, ioffs, 1, np.zeros(3, np.uint32), 1, [(0, 1), (1, 0), (0, 0)])
    assert rc == 0
    assert tuple(int(out[0, 0][f]) for f in ("overlap_ns", "producer_ns", "consumer_ns", "either_ns")) == expect
    # roles swapped; self-overlap equals the producer's own measure
    assert int(out[1, 0]["overlap_ns"]) == expect[0] and int(out[1, 0]["producer_ns"]) == expect[2]
    assert int(out[2, 0]["overlap_ns"]) == int(out[2, 0]["producer_ns"]) == expect[1]


def test_brute_force_wellformed_unique_perfect_matching():
    rng = np.random.default_rng(1)
    for trial in range(40):
        ev = random_wellformed(rng, int(rng.integers(1, 6)), 3, max_height=4)
        rc, iv, _, am, _, st = oracle.pair(ev, single_stream(ev), 3)
        assert len(am) == 0 and len(iv) == len(ev) // 2
        perfect = [m for m in enumerate_matchings(ev) if len(m) == len(ev) // 2]
        # innermost-first (stack) matching is one of the perfect non-crossing matchings; when the
        # region ids of nested frames differ it is the only one
        ends = [i for i in range(len(ev)) if int(ev["tag"][i]) & 1]
        got = frozenset((int(r["begin_idx"]), e) for r, e in zip(iv, ends))
        assert got in perfect
        regions_distinct_on_paths = True
        stack = []
        for t in ev["tag"]:
            if int(t) & 1:
                stack.pop()
            else:
                if (int(t) >> 1) in stack:
                    regions_distinct_on_paths = False
                stack.append(int(t) >> 1)
        if regions_distinct_on_paths:
            # with no region nested in itself, the perfect non-crossing matching is unique
            assert perfect == [got]


def test_brute_force_any_stream_is_valid_matching():
    rng = np.random.default_rng(2)
    for trial in range(60):
        n = int(rng.integers(1, 11))
        rows, t = [], 0
        for _ in range(n):
            t += int(rng.integers(0, 5))
            rows.append((t, "BE"[int(rng.integers(0, 2))], int(rng.integers(0, 3)), 0))
        ev = make_events(rows)
        rc, iv, _, am, _, st = oracle.pair(ev, single_stream(ev), 3)
        assert st["code"] == 0
        amb_idx = {int(r["event_idx"]) for r in am}
        ends = [i for i in range(n) if (int(ev["tag"][i]) & 1) and i not in amb_idx]
        assert len(ends) == len(iv)
        got = frozenset((int(r["begin_idx"]), e) for r, e in zip(iv, ends))
        assert got in enumerate_matchings(ev)
        # I1: begins = intervals + unmatched begins; ends = intervals + unmatched ends (per region)
        for region in range(3):
            nb = sum(1 for tg_ in ev["tag"] if int(tg_) == region << 1)
            ne = sum(1 for tg_ in ev["tag"] if int(tg_) == (region << 1 | 1))
            ni = sum(1 for r in iv if int(r["region"]) == region)
            ub = sum(1 for r in am if int(r["tag"]) >> 1 == region and int(r["kind"]) in (2, 3))
            ue = sum(1 for r in am if int(r["tag"]) >> 1 == region and int(r["kind"]) == 1)
            assert nb == ni + ub and ne == ni + ue
        assert list(am["event_idx"]) == sorted(am["event_idx"])


def test_closed_form_wellformed():
    rng = np.random.default_rng(3)
    for trial in range(25):
        ev = random_wellformed(rng, int(rng.integers(1, 60)), 5, max_height=7, t0=1_700_000_000_000_000_000)
        rc, iv, _, am, _, st = oracle.pair(ev, single_stream(ev), 5)
        assert len(am) == 0 and st["code"] == 0
        want = closed_form_wellformed(ev)
        got = [(int(r["inclusive"]), int(r["exclusive"]), int(r["depth"])) for r in iv]
        assert got == want
        assert all(int(r["flags"]) == 0 for r in iv)


def _forest_checks(ev, iv, am):
    """I2/I3 on one stream: inclusive >= exclusive; for unflagged intervals exclusive + children = inclusive,
    children being the matched intervals directly below in the forest of matched intervals."""
    amb_idx = {int(r["event_idx"]) for r in am}
    ends = [i for i in range(len(ev)) if (int(ev["tag"][i]) & 1) and i not in amb_idx]
    spans = [(int(r["begin_idx"]), e, k) for k, (r, e) in enumerate(zip(iv, ends))]
    child_sum = [0] * len(iv)
    root_incl = 0
    for (b, e, k) in spans:
        # parent in the matched forest: the tightest interval strictly containing (b, e)
        best = None
        for (b2, e2, k2) in spans:
            if b2 < b and e < e2 and (best is None or b2 > best[0]):
                best = (b2, e2, k2)
        if best is None:
            root_incl += int(iv[k]["inclusive"])
        else:
            child_sum[best[2]] += int(iv[k]["inclusive"])
    for k, r in enumerate(iv):
        assert int(r["inclusive"]) >= int(r["exclusive"])
        if int(r["flags"]) & 4 == 0:
            assert int(r["exclusive"]) + child_sum[k] == int(r["inclusive"])
    if all(int(r["flags"]) & 6 == 0 for r in iv):
        assert sum(int(r["exclusive"]) for r in iv) == root_incl


def test_forest_invariants_on_malformed_streams():
    rng = np.random.default_rng(4)
    for trial in range(30):
        ev = random_wellformed(rng, int(rng.integers(5, 40)), 4, max_height=5)
        keep = np.ones(len(ev), bool)
        drop = rng.random(len(ev)) < 0.15
        keep[drop] = False
        ev2 = ev[keep]
        if rng.random() < 0.5 and len(ev2) > 3:
            ev2 = ev2[: int(rng.integers(1, len(ev2)))]
        rc, iv, _, am, _, st = oracle.pair(ev2, single_stream(ev2), 4)
        assert st["code"] == 0
        _forest_checks(ev2, iv, am)


def test_ground_truth_recovery_after_end_deletion():
    # P2: with only end markers deleted and no region nested in itself, every surviving end matches its
    # original begin: intervals == number of ends, no UNMATCHED_END, and each (begin_idx, t_begin, inclusive)
    # appears in the clean trace (indices shift only by deleted ends before the begin).
    rng = np.random.default_rng(5)
    for trial in range(20):
        ev = random_wellformed(rng, 40, 12, max_height=6, self_nest=False)
        _, iv0, _, _, _, _ = oracle.pair(ev, single_stream(ev), 12)
        clean = {(int(r["t_begin"]), int(r["region"]), int(r["depth"])): int(r["inclusive"]) for r in iv0}
        is_end = (ev["tag"] & 1).astype(bool)
        drop = is_end & (rng.random(len(ev)) < 0.2)
        ev2 = ev[~drop]
        _, iv, _, am, _, st = oracle.pair(ev2, single_stream(ev2), 12)
        assert len(iv) == int((ev2["tag"] & 1).sum())
        assert all(int(r["kind"]) != 1 for r in am)
        ts_count = {}
        for r in iv0:
            ts_count[int(r["t_begin"])] = ts_count.get(int(r["t_begin"]), 0) + 1
        for r in iv:
            key = (int(r["t_begin"]), int(r["region"]))
            matches = [v for (t, reg, d), v in clean.items() if (t, reg) == key]
            assert int(r["inclusive"]) in matches


def test_tracegen_malformed_end_deletion_recovers_config():
    # same property on the GEMM-shaped generator trace: program draws are independent of defect draws,
    # so the clean trace with the same seed is the ground truth
    base = tg.TraceSpec(tg.GEMM, 2, 30, 0, seed=77)
    ev0, offs0 = tg.generate_host(base)
    ev1, offs1 = tg.generate_host(tg.TraceSpec(tg.GEMM, 2, 30, 0, seed=77, p_drop_end=0.02))
    assert len(ev1) < len(ev0)
    _, iv0, _, am0, _, _ = oracle.pair(ev0, offs0, 5)
    _, iv1, io1, am1, _, _ = oracle.pair(ev1, offs1, 5)
    assert len(am0) == 0
    assert len(iv1) == int((ev1["tag"] & 1).sum())
    assert all(int(r["kind"]) != 1 for r in am1)
    clean = {(int(r["stream"]), int(r["t_begin"]), int(r["region"]), int(r["ctx"]), int(r["inclusive"])) for r in iv0}
    for r in iv1:
        assert (int(r["stream"]), int(r["t_begin"]), int(r["region"]), int(r["ctx"]), int(r["inclusive"])) in clean
    # duplicated begins only: the multiset of (region, ctx, t_begin, inclusive) equals the clean trace's
    ev2, offs2 = tg.generate_host(tg.TraceSpec(tg.GEMM, 2, 30, 0, seed=77, p_dup_begin=0.02))
    assert len(ev2) > len(ev0)
    _, iv2, _, am2, _, _ = oracle.pair(ev2, offs2, 5)
    key = lambda iv: sorted((int(r["stream"]), int(r["region"]), int(r["ctx"]), int(r["t_begin"]), int(r["inclusive"]))
                            for r in iv)
    assert key(iv2) == key(iv0)
    assert len(am2) == len(ev2) - len(ev0)


def test_aggregate_matches_numpy_groupby_and_rollup():
    spec = tg.TraceSpec(tg.GEMM, 4, 25, 0, seed=9, p_drop_end=0.01, p_dup_begin=0.01, p_trunc=0.1)
    ev, offs = tg.generate_host(spec)
    _, iv, ioffs, am, aoffs, _ = oracle.pair(ev, offs, spec.num_regions)
    cta_sm = np.array([0, 1, 1, 0], np.uint32)
    rc, tabs, st = oracle.aggregate(iv, ioffs, am, aoffs, spec.warps_per_cta, cta_sm, 2, spec.num_regions)
    assert rc == 0 and st["code"] == 0
    R, W = spec.num_regions, spec.warps_per_cta
    level_key = {"warp": lambda s: s, "cta": lambda s: s // W, "sm": lambda s: cta_sm[s // W], "kernel": lambda s: 0 * s}
    for lv, fn in level_key.items():
        tab = tabs[lv]
        keys = fn(iv["stream"].astype(np.int64))
        cell = keys * R + iv["region"].astype(np.int64)
        ncell = tab.shape[0] * R
        assert np.array_equal(tab["count"].ravel(), np.bincount(cell, minlength=ncell).astype(np.uint64))
        for field, src in (("sum_incl", "inclusive"), ("sum_excl", "exclusive")):
            acc = np.zeros(ncell, np.uint64)
            np.add.at(acc, cell, iv[src])
            assert np.array_equal(tab[field].ravel(), acc)
        mn = np.full(ncell, np.iinfo(np.uint64).max, np.uint64)
        np.minimum.at(mn, cell, iv["inclusive"])
        mx = np.zeros(ncell, np.uint64)
        np.maximum.at(mx, cell, iv["inclusive"])
        assert np.array_equal(tab["min_incl"].ravel(), mn) and np.array_equal(tab["max_incl"].ravel(), mx)
        # floor(log2) through exact integer bit_length, bins of 0 and 1 both 0
        bins = np.array([max(int(d).bit_length() - 1, 0) for d in iv["inclusive"]], np.int64)
        hist = np.zeros((ncell, 64), np.uint64)
        np.add.at(hist, (cell, bins), 1)
        assert np.array_equal(tab["hist"].reshape(ncell, 64), hist)
        assert np.array_equal(tab["n_flagged"].ravel(), np.bincount(cell[iv["flags"] != 0], minlength=ncell).astype(np.uint64))
        akeys = fn(am["stream"].astype(np.int64)) * R + (am["tag"] >> 1).astype(np.int64)
        ub = np.bincount(akeys[am["kind"] != 1], minlength=ncell).astype(np.uint64)
        ue = np.bincount(akeys[am["kind"] == 1], minlength=ncell).astype(np.uint64)
        assert np.array_equal(tab["n_unmatched_begin"].ravel(), ub)
        assert np.array_equal(tab["n_unmatched_end"].ravel(), ue)
        assert np.array_equal(tab["hist"].sum(-1), tab["count"])  # I6
    # I5 roll-up: kernel = sum of SM = sum of CTA = sum of warp; min/max by min/max
    for field in ("count", "sum_incl", "sum_excl", "n_flagged", "n_unmatched_begin", "n_unmatched_end", "hist"):
        k = tabs["kernel"][field][0]
        for lv in ("warp", "cta", "sm"):
            assert np.array_equal(tabs[lv][field].sum(0, dtype=np.uint64), k)
    for lv in ("warp", "cta", "sm"):
        assert np.array_equal(tabs[lv]["min_incl"].min(0), tabs["kernel"]["min_incl"][0])
        assert np.array_equal(tabs[lv]["max_incl"].max(0), tabs["kernel"]["max_incl"][0])
    # empty cells: zero with min = UINT64_MAX
    empty = tabs["warp"][tabs["warp"]["count"] == 0]
    assert np.all(empty["min_incl"] == np.iinfo(np.uint64).max) and np.all(empty["max_incl"] == 0)


def test_overlap_matches_tick_counting():
    rng = np.random.default_rng(6)
    for trial in range(20):
        S, W, M, R = 8, 2, 2, 3
        cta_sm = np.array([0, 1, 1, 0], np.uint32)
        rows = []
        for s in range(S):
            for _ in range(int(rng.integers(0, 6))):
                rows.append((s, int(rng.integers(0, R)), 100 + int(rng.integers(0, 60)), int(rng.integers(0, 25))))
        rows.sort(key=lambda r: r[0])
        iv = np.zeros(len(rows), oracle.INTERVAL)
        ioffs = np.zeros(S + 1, np.uint64)
        for i, (s, region, t, d) in enumerate(rows):
            iv[i]["stream"], iv[i]["region"], iv[i]["t_begin"], iv[i]["inclusive"] = s, region, t, d
            ioffs[s + 1:] += 1
        pairs = [(0, 1), (1, 2), (2, 2), (1, 0)]
        rc, out, st = oracle.overlap(iv, ioffs, W, cta_sm, M, pairs)
        assert rc == 0
        for k, (P, C) in enumerate(pairs):
            for m in range(M):
                tick_p, tick_c = np.zeros(256, bool), np.zeros(256, bool)
                for (s, region, t, d) in rows:
                    if cta_sm[s // W] != m:
                        continue
                    if region == P:
                        tick_p[t:t + d] = True
                    if region == C:
                        tick_c[t:t + d] = True
                o = out[k, m]
                assert int(o["producer_ns"]) == tick_p.sum() and int(o["consumer_ns"]) == tick_c.sum()
                assert int(o["overlap_ns"]) == (tick_p & tick_c).sum()
                assert int(o["either_ns"]) == (tick_p | tick_c).sum()
                assert int(o["overlap_ns"]) <= min(int(o["producer_ns"]), int(o["consumer_ns"]))  # I7


def test_time_shift_and_concatenation_invariance():
    rng = np.random.default_rng(7)
    a = random_wellformed(rng, 30, 4)
    b = random_wellformed(rng, 20, 4, t0=50_000)
    _, iva, _, _, _, _ = oracle.pair(a, single_stream(a), 4)
    _, ivb, _, _, _, _ = oracle.pair(b, single_stream(b), 4)
    shifted = a.copy()
    shifted["ts"] += 12345
    _, ivs, _, _, _, _ = oracle.pair(shifted, single_stream(shifted), 4)
    assert np.array_equal(ivs["t_begin"], iva["t_begin"] + 12345)
    for f in ("inclusive", "exclusive", "region", "depth", "parent_region", "begin_idx", "ctx"):
        assert np.array_equal(ivs[f], iva[f])
    # I10: two well-formed streams in one stream buffer back to back = outputs back to back
    ab = np.concatenate([a, b])
    _, ivab, _, amab, _, _ = oracle.pair(ab, single_stream(ab), 4)
    assert len(amab) == 0 and len(ivab) == len(iva) + len(ivb)
    for f in ("t_begin", "inclusive", "exclusive", "region", "depth", "parent_region", "ctx"):
        assert np.array_equal(ivab[f], np.concatenate([iva[f], ivb[f]]))
    assert np.array_equal(ivab["begin_idx"][len(iva):], ivb["begin_idx"] + len(a))
    # as two streams: offsets and stream ids
    offs = np.array([0, len(a), len(a) + len(b)], np.uint64)
    _, iv2, io2, _, ao2, _ = oracle.pair(ab, offs, 4)
    assert list(io2) == [0, len(iva), len(iva) + len(ivb)] and list(ao2) == [0, 0, 0]
    assert np.array_equal(iv2["begin_idx"][len(iva):], ivb["begin_idx"])
    assert set(iv2["stream"][len(iva):]) == {1}


def test_error_codes_and_edges():
    # empty input, empty streams, offsets that do not start at zero
    ev = make_events([(1, "B", 0, 0), (2, "E", 0, 0), (5, "B", 1, 3), (9, "E", 1, 3)])
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, np.array([2, 2, 4, 4], np.uint64), 2)
    assert st["code"] == 0 and list(ioffs) == [0, 0, 1, 1] and int(iv[0]["region"]) == 1 and int(iv[0]["stream"]) == 1
    assert int(iv[0]["begin_idx"]) == 0
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev[:0], np.array([0], np.uint64), 2)
    assert rc == 0 and st["code"] == 0 and len(iv) == 0
    # bad region
    rc, *_, st = oracle.pair(ev, single_stream(ev), 1)
    assert st["code"] == 6 and int(st["bad_event"]) == 2
    # depth overflow at the 65th open frame; 64 are fine
    deep = make_events([(i, "B", 0, 0) for i in range(64)])
    rc, iv, _, am, _, st = oracle.pair(deep, single_stream(deep), 1)
    assert st["code"] == 0 and len(am) == 64 and [int(d) for d in am["depth"]] == list(range(64))
    deep = make_events([(i, "B", 0, 0) for i in range(65)])
    rc, *_, st = oracle.pair(deep, single_stream(deep), 1)
    assert st["code"] == 5 and int(st["bad_event"]) == 64
    # capacity: required counts are reported
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, single_stream(ev), 2, interval_cap=1)
    assert st["code"] == 4 and int(st["intervals_required"]) == 2
    # decreasing offsets
    rc, *_, st = oracle.pair(ev, np.array([0, 3, 2], np.uint64), 2)
    assert st["code"] == 7
    # status counters
    evh, _, _ = load_example("example_h_flags.txt")
    *_, st = oracle.pair(evh, single_stream(evh), 3)
    assert (int(st["n_ctx_mismatch"]), int(st["n_time_reversed"]), int(st["n_child_clamped"])) == (1, 1, 1)


def test_full_config_invariants_tiny_and_scaled():
    # config 0 at full size; the others scaled down, same structure
    specs = [tg.config(0), tg.config(1).scaled(3, 40), tg.config(2).scaled(2, 2), tg.config(3).scaled(2, 3),
             tg.config(4).scaled(6, 60)]
    heights = {tg.TINY: 3, tg.GEMM: 3, tg.ATTENTION: 4, tg.DECODE: 5}
    for spec in specs:
        ev, offs = tg.generate_host(spec)
        rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions)
        assert rc == 0 and st["code"] == 0
        nb = int(((ev["tag"] & 1) == 0).sum())
        ne = len(ev) - nb
        assert nb == len(iv) + int((am["kind"] != 1).sum()) and ne == len(iv) + int((am["kind"] == 1).sum())
        assert int(ioffs[-1]) == len(iv) and int(aoffs[-1]) == len(am)
        assert np.all(iv["inclusive"] >= iv["exclusive"])
        if spec.well_formed:
            assert len(am) == 0 and np.all(iv["flags"] == 0) and len(iv) * 2 == len(ev)
            assert int(iv["depth"].max()) == heights[spec.kind] - 1
            # I3 per stream: sum of exclusive = sum of inclusive of top-level intervals
            for s in range(spec.num_streams):
                seg = iv[int(ioffs[s]):int(ioffs[s + 1])]
                assert int(seg["exclusive"].sum(dtype=np.uint64)) == int(seg["inclusive"][seg["depth"] == 0].sum(dtype=np.uint64))
            top = iv[iv["depth"] == 0]
            assert np.all(top["parent_region"] == NONE)
        else:
            assert len(am) > 0
