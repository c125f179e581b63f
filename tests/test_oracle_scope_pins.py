"""Pins of the oracle's scope selection (aggregate_scoped, overlap_scoped): a hand-worked example,
the unscoped functions (pinned elsewhere) as the all-selecting special case, additivity over
partitions of a scope dimension, and counts / sums redone with numpy masks and bincount."""
import os

import numpy as np
import pytest

import oracle
from helpers import GOLDEN
from paper_2609_12299_b200 import tracegen as tg

ALL32 = 0xFFFFFFFF
ADD_FIELDS = ("count", "sum_incl", "sum_excl", "n_unmatched_begin", "n_unmatched_end", "n_flagged", "hist")


def _parse_list(tok):
    return None if tok == "all" else [int(x) for x in tok]


def load_scope_example():
    ivs, scopes, expect, overlap = [], {}, {}, {}
    with open(os.path.join(GOLDEN, "example_i_scope.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] == "iv":
                ivs.append(tuple(int(x) for x in tok[1:]))
            elif tok[0] == "scope":
                i_w, i_s, i_r = tok.index("warps"), tok.index("sms"), tok.index("regions")
                sc = {"ctx": (int(tok[3]), int(tok[4]))}
                for key, lo, hi in (("warps", i_w, i_s), ("sms", i_s, i_r), ("regions", i_r, len(tok))):
                    sel = _parse_list(tok[lo + 1] if tok[lo + 1] == "all" else tok[lo + 1:hi])
                    if sel is not None:
                        sc[key] = sel
                scopes[tok[1]] = sc
            elif tok[0] == "expect":
                expect.setdefault(tok[1], {})[(tok[2], int(tok[3]), int(tok[4]))] = tuple(int(x) for x in tok[5:])
            elif tok[0] == "overlap":
                overlap.setdefault(tok[1], {})[int(tok[2])] = tuple(int(x) for x in tok[3:])
    S = 4
    iv = np.zeros(len(ivs), dtype=oracle.INTERVAL)
    ioffs = np.zeros(S + 1, dtype=np.uint64)
    for i, (s, r, ctx, t0, incl, excl) in enumerate(sorted(ivs, key=lambda v: v[0])):
        iv[i]["stream"], iv[i]["region"], iv[i]["ctx"] = s, r, ctx
        iv[i]["t_begin"], iv[i]["inclusive"], iv[i]["exclusive"] = t0, incl, excl
        iv[i]["parent_region"] = oracle.NONE
        ioffs[s + 1:] += 1
    return iv, ioffs, scopes, expect, overlap


def test_hand_worked_scopes():
    iv, ioffs, scopes, expect, overlap = load_scope_example()
    cta_sm = np.array([0, 1], dtype=np.uint32)
    for name, cells in expect.items():
        rc, tabs, st = oracle.aggregate_scoped(iv, ioffs, None, None, 2, cta_sm, 2, 3, scope=scopes[name])
        assert rc == 0 and int(st["code"]) == 0
        listed = {lv for (lv, _, _) in cells}
        for lv in listed:
            tab = tabs[lv]
            for key in range(tab.shape[0]):
                for r in range(3):
                    c = tab[key, r]
                    got = (int(c["count"]), int(c["sum_incl"]), int(c["min_incl"]), int(c["max_incl"]), int(c["sum_excl"]))
                    want = cells.get((lv, key, r), (0, 0, 2**64 - 1, 0, 0))
                    assert got == want, (name, lv, key, r, got, want)
    for name, rows in overlap.items():
        rc, out, st = oracle.overlap_scoped(iv, ioffs, 2, cta_sm, 2, [(0, 1)], scope=scopes[name], num_regions=3)
        assert rc == 0
        for m, want in rows.items():
            o = out[0, m]
            assert (int(o["overlap_ns"]), int(o["producer_ns"]), int(o["consumer_ns"]), int(o["either_ns"])) == want, (name, m)


@pytest.fixture(scope="module")
def tiny():
    """The tiny benchmark trace with a few defects, so that ambiguity records exist."""
    spec = tg.TraceSpec(kind=tg.TINY, num_ctas=4, iters=626, inner=0, seed=77, p_dup_begin=0.02, p_drop_end=0.03,
                        p_trunc=0.1, name="tiny-defects")
    ev, offs = tg.generate_host(spec)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions)
    assert rc == 0 and int(st["code"]) == 0 and len(am) > 0
    return spec, iv, ioffs, am, aoffs


def _agg(tiny, scope, levels=("warp", "cta", "sm", "kernel", "role", "iter")):
    spec, iv, ioffs, am, aoffs = tiny
    rc, tabs, st = oracle.aggregate_scoped(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms,
                                           spec.num_regions, scope=scope, levels=levels)
    assert rc == 0 and int(st["code"]) == 0
    return tabs


def test_everything_selected_is_the_unscoped_aggregate(tiny):
    spec, iv, ioffs, am, aoffs = tiny
    rc, ref, st = oracle.aggregate(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.num_regions)
    assert rc == 0
    for scope in (None, {}, {"ctx": (0, ALL32), "warps": range(spec.warps_per_cta), "sms": range(spec.num_sms),
                             "regions": range(spec.num_regions)}):
        tabs = _agg(tiny, scope, levels=("warp", "cta", "sm", "kernel", "role"))
        for lv in ("warp", "cta", "sm", "kernel"):
            assert tabs[lv].tobytes() == ref[lv].tobytes(), lv
        # role rows: the warp rows with the same index inside their CTA, combined
        W = spec.warps_per_cta
        for w in range(W):
            rows = ref["warp"][w::W]
            for f in ADD_FIELDS:
                assert np.array_equal(tabs["role"][w][f], rows[f].sum(0, dtype=np.uint64)), (w, f)
            assert np.array_equal(tabs["role"][w]["min_incl"], rows["min_incl"].min(0))
            assert np.array_equal(tabs["role"][w]["max_incl"], rows["max_incl"].max(0))


def _assert_partition_adds_up(whole, parts):
    for f in ADD_FIELDS:
        assert np.array_equal(sum(p[f].astype(object) for p in parts).astype(np.uint64), whole[f]), f
    assert np.array_equal(np.minimum.reduce([p["min_incl"] for p in parts]), whole["min_incl"])
    assert np.array_equal(np.maximum.reduce([p["max_incl"] for p in parts]), whole["max_incl"])


def test_partitions_of_each_scope_dimension_add_up(tiny):
    spec = tiny[0]
    whole = _agg(tiny, None, levels=("kernel",))["kernel"]
    ctxs = np.unique(np.concatenate([tiny[1]["ctx"], tiny[3]["ctx"]]))
    mid = int(ctxs[len(ctxs) // 2])
    parts = [{"ctx": (0, mid)}, {"ctx": (mid + 1, ALL32)}]
    _assert_partition_adds_up(whole, [_agg(tiny, p, ("kernel",))["kernel"] for p in parts])
    parts = [{"warps": [0, 3]}, {"warps": [1]}, {"warps": [2]}]
    _assert_partition_adds_up(whole, [_agg(tiny, p, ("kernel",))["kernel"] for p in parts])
    parts = [{"sms": [0]}, {"sms": [1]}]
    _assert_partition_adds_up(whole, [_agg(tiny, p, ("kernel",))["kernel"] for p in parts])
    # a region mask keeps the selected columns untouched and empties the others
    sel = [1, 4, 6]
    t = _agg(tiny, {"regions": sel}, ("kernel",))["kernel"]
    for r in range(spec.num_regions):
        if r in sel:
            assert t[0, r].tobytes() == whole[0, r].tobytes()
        else:
            assert int(t[0, r]["count"]) == 0 and int(t[0, r]["min_incl"]) == 2**64 - 1
            assert int(t[0, r]["n_unmatched_begin"]) + int(t[0, r]["n_unmatched_end"]) == 0


def test_counts_and_sums_redone_with_numpy_masks(tiny):
    spec, iv, ioffs, am, aoffs = tiny
    W, R = spec.warps_per_cta, spec.num_regions
    ctx_lo, ctx_hi = 3, 11
    scope = {"ctx": (ctx_lo, ctx_hi), "warps": [0, 2, 3], "sms": [1], "regions": [0, 2, 3, 5, 7]}
    tabs = _agg(tiny, scope)

    def mask(stream, ctx, region):
        return ((ctx >= ctx_lo) & (ctx <= ctx_hi) & np.isin(stream % W, scope["warps"]) &
                np.isin(spec.cta_sm[stream // W], scope["sms"]) & np.isin(region, scope["regions"]))

    m = mask(iv["stream"], iv["ctx"], iv["region"])
    assert 0 < m.sum() < len(iv)
    sel = iv[m]
    ker = tabs["kernel"][0]
    assert np.array_equal(ker["count"], np.bincount(sel["region"], minlength=R))
    for field, src in (("sum_incl", "inclusive"), ("sum_excl", "exclusive")):
        want = np.zeros(R, dtype=np.uint64)
        np.add.at(want, sel["region"], sel[src])
        assert np.array_equal(ker[field], want)
    assert np.array_equal(ker["n_flagged"], np.bincount(sel["region"][sel["flags"] != 0], minlength=R))
    bins = np.where(sel["inclusive"] > 0, np.floor(np.log2(np.maximum(sel["inclusive"], 1).astype(np.float64))), 0).astype(int)
    assert np.array_equal(ker["hist"], np.bincount(sel["region"] * 64 + bins, minlength=R * 64).reshape(R, 64))
    am_m = mask(am["stream"], am["ctx"], am["tag"] >> 1)
    sel_am = am[am_m]
    assert np.array_equal(ker["n_unmatched_end"], np.bincount((sel_am["tag"] >> 1)[sel_am["kind"] == 1], minlength=R))
    assert np.array_equal(ker["n_unmatched_begin"], np.bincount((sel_am["tag"] >> 1)[sel_am["kind"] != 1], minlength=R))
    # per-warp, per-role and per-iteration keys
    assert np.array_equal(tabs["warp"]["count"], np.bincount(sel["stream"].astype(np.int64) * R + sel["region"],
                                                             minlength=spec.num_streams * R).reshape(-1, R))
    assert np.array_equal(tabs["role"]["count"], np.bincount((sel["stream"] % W).astype(np.int64) * R + sel["region"],
                                                             minlength=W * R).reshape(W, R))
    n_it = ctx_hi - ctx_lo + 1
    assert tabs["iter"].shape == (n_it, R)
    assert np.array_equal(tabs["iter"]["count"], np.bincount((sel["ctx"] - ctx_lo).astype(np.int64) * R + sel["region"],
                                                             minlength=n_it * R).reshape(n_it, R))
    # every keyed table adds up to the kernel table of the same scope
    for lv in ("warp", "cta", "sm", "role", "iter"):
        _assert_partition_adds_up(tabs["kernel"], list(tabs[lv][:, None, :]))


def test_scoped_overlap_special_cases(tiny):
    spec, iv, ioffs, _, _ = tiny
    W, M = spec.warps_per_cta, spec.num_sms
    pairs = spec.overlap_pairs
    rc, ref, _ = oracle.overlap(iv, ioffs, W, spec.cta_sm, M, pairs)
    rc2, out, _ = oracle.overlap_scoped(iv, ioffs, W, spec.cta_sm, M, pairs, scope=None, num_regions=spec.num_regions)
    assert rc == 0 and rc2 == 0 and out.tobytes() == ref.tobytes() and int(ref["overlap_ns"].sum()) > 0
    # SM subset: the other SM's row is zero, the selected one is unchanged
    _, out, _ = oracle.overlap_scoped(iv, ioffs, W, spec.cta_sm, M, pairs, scope={"sms": [1]}, num_regions=spec.num_regions)
    assert out[:, 1].tobytes() == ref[:, 1].tobytes() and not out[:, 0].tobytes().strip(b"\0")
    # without the producer's region nothing overlaps and the consumer's union is unchanged
    k = 0
    P, Cn = int(pairs[k][0]), int(pairs[k][1])
    keep = [r for r in range(spec.num_regions) if r != P]
    _, out, _ = oracle.overlap_scoped(iv, ioffs, W, spec.cta_sm, M, pairs[k:k + 1], scope={"regions": keep},
                                      num_regions=spec.num_regions)
    assert not out["producer_ns"].any() and not out["overlap_ns"].any()
    assert np.array_equal(out["consumer_ns"], ref[k:k + 1]["consumer_ns"]) and np.array_equal(out["either_ns"], out["consumer_ns"])
    # a window can only shrink the unions; windows that split the contexts bound the whole from below
    ctxs = np.unique(iv["ctx"])
    mid = int(ctxs[len(ctxs) // 2])
    _, lo, _ = oracle.overlap_scoped(iv, ioffs, W, spec.cta_sm, M, pairs, scope={"ctx": (0, mid)}, num_regions=spec.num_regions)
    _, hi, _ = oracle.overlap_scoped(iv, ioffs, W, spec.cta_sm, M, pairs, scope={"ctx": (mid + 1, ALL32)}, num_regions=spec.num_regions)
    for f in ("producer_ns", "consumer_ns", "either_ns"):
        assert np.all(lo[f] <= ref[f]) and np.all(hi[f] <= ref[f]) and np.all(lo[f] + hi[f] >= ref[f])


def test_scope_argument_errors(tiny):
    spec, iv, ioffs, am, aoffs = tiny
    rc, _, _ = oracle.aggregate_scoped(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms,
                                       spec.num_regions, scope={"ctx": (5, 4)})
    assert rc == 1
    rc, _, _ = oracle.aggregate_scoped(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms,
                                       spec.num_regions, scope={"ctx": (0, 70000)})
    assert rc == 1  # an iteration table of more than 65536 rows
    rc, _, _ = oracle.overlap_scoped(iv, ioffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.overlap_pairs,
                                     scope={"ctx": (5, 4)}, num_regions=spec.num_regions)
    assert rc == 1
