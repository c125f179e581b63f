"""Parity at the full benchmark sizes, in the launch configuration bench.py times (argus_synthesize on
a trace generated in GPU memory): EVERY CTA is regenerated on the host (the generator is bit-identical
on host and device), run through the CPU oracle on its own and compared bit for bit (intervals,
ambiguity records, warp and CTA rows, SM row and overlap), one CTA per host thread so that host memory
stays bounded; the oracle's per-CTA tables are merged in plain numpy (sum / min / max) and compared with
the SM- and kernel-scope tables; properties that hold at any size are checked on the whole output."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from paper_2609_12299_b200 import tracegen as tg

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_full(spec):
    d_ev, d_off = tg.generate_cuda(spec, DEV)
    n = d_ev.numel() // 16
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs,
                                 interval_capacity=n // 2, ambig_capacity=max(n // 64, 4096),
                                 max_overlap_spans=max(n // 8, 1 << 16))
    st = res.fetch_status()
    assert int(st["code"]) == 0, st
    return res, st, n, d_off.cpu().numpy().view(np.uint64)


def _check_cta(spec, res, offs, c, host):
    """Everything the path produced for CTA `c` against the oracle run on that CTA alone."""
    W, R = spec.warps_per_cta, spec.num_regions
    s0, s1 = c * W, (c + 1) * W
    ev = tg.host_streams(spec, offs, s0, s1, nthreads=1)
    sub = (offs[s0:s1 + 1] - offs[s0]).astype(np.uint64)
    rc, o_iv, o_ioffs, o_am, o_aoffs, o_st = oracle.pair(ev, sub, R, ambig_cap=max(len(ev) // 16, 4096))
    assert rc == 0 and int(o_st["code"]) == 0
    del ev
    ioffs, aoffs = host["ioffs"], host["aoffs"]
    assert np.array_equal(ioffs[s0:s1 + 1] - ioffs[s0], o_ioffs)
    assert np.array_equal(aoffs[s0:s1 + 1] - aoffs[s0], o_aoffs)
    g_iv = res.pair.intervals[int(ioffs[s0]) * 48:int(ioffs[s1]) * 48].cpu().numpy().view(argus.INTERVAL_DTYPE)
    want = o_iv.copy()
    want["stream"] += s0
    assert g_iv.tobytes() == want.tobytes(), f"intervals of CTA {c} differ"
    g_am = res.pair.ambig[int(aoffs[s0]) * 32:int(aoffs[s1]) * 32].cpu().numpy().view(argus.AMBIG_DTYPE)
    want_am = o_am.copy()
    want_am["stream"] += s0
    assert g_am.tobytes() == want_am.tobytes(), f"ambiguity records of CTA {c} differ"
    _, o_tabs, _ = oracle.aggregate(o_iv, o_ioffs, o_am, o_aoffs, W, np.zeros(1, np.uint32), 1, R)
    row = R * 576
    g_warp = res.agg.warp[s0 * row:s1 * row].cpu().numpy().view(argus.AGG_DTYPE).reshape(W, R)
    assert g_warp.tobytes() == o_tabs["warp"].tobytes(), f"warp rows of CTA {c} differ"
    g_cta = res.agg.cta[c * row:(c + 1) * row].cpu().numpy().view(argus.AGG_DTYPE).reshape(1, R)
    assert g_cta.tobytes() == o_tabs["cta"].tobytes(), f"CTA row {c} differs"
    if np.array_equal(spec.cta_sm, np.arange(spec.num_ctas)):  # one CTA per SM: SM row and overlap are this CTA's
        g_sm = res.agg.sm[c * row:(c + 1) * row].cpu().numpy().view(argus.AGG_DTYPE).reshape(1, R)
        assert g_sm.tobytes() == o_tabs["sm"].tobytes(), f"SM row {c} differs"
        _, o_ov, _ = oracle.overlap(o_iv, o_ioffs, W, np.zeros(1, np.uint32), 1, spec.overlap_pairs)
        g_ov = host["overlap"][:, c]
        assert g_ov.tobytes() == o_ov[:, 0].tobytes(), f"overlap of SM {c} differs"
    return len(o_iv), len(o_am), o_tabs["cta"][0].copy()


_ADD = ("count", "sum_incl", "sum_excl", "n_unmatched_begin", "n_unmatched_end", "n_flagged", "hist")


def _merge(rows):
    """Rows of per-CTA oracle tables ([k][R]) into one row: additive fields summed, min / max taken."""
    out = rows[0].copy()
    for f in _ADD:
        out[f] = np.sum([r[f] for r in rows], axis=0, dtype=np.uint64)
    out["min_incl"] = np.min([r["min_incl"] for r in rows], axis=0)
    out["max_incl"] = np.max([r["max_incl"] for r in rows], axis=0)
    return out


def _check_every_cta(spec, res, offs):
    """All CTAs against the oracle (one CTA per host thread), then the SM and kernel tables against the merged
    per-CTA oracle tables. Returns the intervals and ambiguity records compared."""
    host = {"ioffs": res.pair.interval_offsets.cpu().numpy().view(np.uint64),
            "aoffs": res.pair.ambig_offsets.cpu().numpy().view(np.uint64), "overlap": res.overlap_numpy(spec.num_sms)}
    with ThreadPoolExecutor(max_workers=min(os.cpu_count() or 1, 16)) as pool:
        done = list(pool.map(lambda c: _check_cta(spec, res, offs, c, host), range(spec.num_ctas)))
    rows = [d[2] for d in done]
    sm_want = np.stack([_merge([rows[c] for c in range(spec.num_ctas) if spec.cta_sm[c] == m]) for m in range(spec.num_sms)])
    assert res.agg.table_numpy("sm").tobytes() == sm_want.tobytes(), "SM table differs from the merged oracle tables"
    ker_want = _merge(rows)[None]
    assert res.agg.table_numpy("kernel").tobytes() == ker_want.tobytes(), "kernel table differs from the merged oracle tables"
    assert int(host["ioffs"][-1]) == sum(d[0] for d in done) and int(host["aoffs"][-1]) == sum(d[1] for d in done)
    return sum(d[0] for d in done), sum(d[1] for d in done)


def _check_global(spec, res, st, n, well_formed):
    """Size-independent properties of the whole output."""
    S, R = spec.num_streams, spec.num_regions
    ioffs = res.pair.interval_offsets.cpu().numpy().view(np.uint64)
    total = int(ioffs[-1])
    assert int(st["intervals_required"]) == total
    if well_formed:
        assert total * 2 == n and int(st["ambig_required"]) == 0 and int(st["n_sequential_tiles"]) == 0
    warp = res.agg.table_numpy("warp")
    cta, sm, ker = res.agg.table_numpy("cta"), res.agg.table_numpy("sm"), res.agg.table_numpy("kernel")
    assert int(ker["count"].sum()) == total
    assert np.array_equal(warp["count"].sum(1), np.diff(ioffs))       # per-stream counts = CSR offsets
    for f in ("count", "sum_incl", "sum_excl", "n_flagged", "n_unmatched_begin", "n_unmatched_end", "hist"):
        for tab in (warp, cta, sm):
            assert np.array_equal(tab[f].sum(0, dtype=np.uint64), ker[f][0]), f
    for tab in (warp, cta, sm):
        assert np.array_equal(tab["min_incl"].min(0), ker["min_incl"][0])
        assert np.array_equal(tab["max_incl"].max(0), ker["max_incl"][0])
    assert np.array_equal(ker["hist"].sum(-1), ker["count"])
    assert int((ker["n_unmatched_begin"] + ker["n_unmatched_end"]).sum()) == int(st["ambig_required"])
    ov = res.overlap_numpy(spec.num_sms)
    assert np.all(ov["overlap_ns"] <= np.minimum(ov["producer_ns"], ov["consumer_ns"]))
    assert np.array_equal(ov["either_ns"], ov["producer_ns"] + ov["consumer_ns"] - ov["overlap_ns"])
    del warp


def test_decode_megakernel_full_size():
    """The bench workload: 1.23 G events (19.65 GB), 202 regions; all 148 CTAs."""
    spec = tg.config(3)
    res, st, n, offs = _run_full(spec)
    assert n == 1_228_177_408
    _check_global(spec, res, st, n, well_formed=True)
    ni, na = _check_every_cta(spec, res, offs)
    assert ni == spec.num_streams * 259_328 and na == 0
    del res
    torch.cuda.empty_cache()


def test_attention_full_size():
    spec = tg.config(2)
    res, st, n, offs = _run_full(spec)
    assert n == 153_513_888
    _check_global(spec, res, st, n, well_formed=True)
    _check_every_cta(spec, res, offs)
    ov = res.overlap_numpy(spec.num_sms)
    assert np.all(ov["overlap_ns"] > 0)  # producer and consumer spans do overlap on every SM in this trace
    del res
    torch.cuda.empty_cache()


def test_persistent_gemm_full_size():
    spec = tg.config(1)
    res, st, n, offs = _run_full(spec)
    assert n == 68_672_000
    _check_global(spec, res, st, n, well_formed=True)
    _check_every_cta(spec, res, offs)
    del res
    torch.cuda.empty_cache()


def test_malformed_full_size():
    """Dropped ends, duplicated begins and truncated streams at full size: ambiguity records, the
    second (re-basing) pass and the sequential redo of tiles that are not well nested."""
    spec = tg.config(4)
    res, st, n, offs = _run_full(spec)
    assert int(st["ambig_required"]) > 0 and int(st["n_sequential_tiles"]) > 0
    _check_global(spec, res, st, n, well_formed=False)
    lens = np.diff(offs)
    truncated = np.nonzero(lens < np.where(np.arange(spec.num_streams) % 12 < 2, 72000, 32000) * 0.99)[0]
    assert len(truncated) > 0
    ni, na = _check_every_cta(spec, res, offs)
    assert na == int(st["ambig_required"]) > 0
    del res
    torch.cuda.empty_cache()


def test_decode_full_size_scoped_aggregate():
    """Scope selection at the bench size: 16 of the 256 iterations, three warp roles, on the 614 M intervals
    the path produced; sampled CTAs against the oracle, size-independent properties on the whole tables."""
    spec = tg.config(3)
    res, st, n, offs = _run_full(spec)
    W, R, M = spec.warps_per_cta, spec.num_regions, spec.num_sms
    lo, hi, warps = 100, 115, [0, 1, 5]
    scope = argus.ArgusScope(ctx_lo=lo, ctx_hi=hi, warp_mask=sum(1 << w for w in warps))
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    sc = argus.argus_aggregate_scoped(res.pair.intervals, res.pair.interval_offsets, res.pair.ambig, res.pair.ambig_offsets,
                                      W, cta_sm, M, R, scope, levels=("warp", "cta", "sm", "kernel", "role", "iter"))
    assert int(argus.argus_status_fetch(sc.status)["code"]) == 0
    ker, role, it = sc.table_numpy("kernel"), sc.table_numpy("role"), sc.table_numpy("iter")
    warp = sc.table_numpy("warp")
    assert it.shape == (16, R) and role.shape == (W, R)
    for f in ("count", "sum_incl", "sum_excl", "n_flagged", "hist"):
        for tab in (warp, role, it, sc.table_numpy("cta"), sc.table_numpy("sm")):
            assert np.array_equal(tab[f].sum(0, dtype=np.uint64), ker[f][0]), f
    assert not role["count"][[w for w in range(W) if w not in warps]].any()
    # every stream runs the same program: 16 iterations x 1013 intervals in each selected stream
    assert np.array_equal(warp["count"].sum(1), np.where(np.isin(np.arange(spec.num_streams) % W, warps), 16 * 1013, 0))
    assert np.all(it["count"].sum(1) == 1013 * len(warps) * spec.num_ctas)
    for c in (0, 91):
        s0, s1 = c * W, (c + 1) * W
        ev = tg.host_streams(spec, offs, s0, s1)
        sub = (offs[s0:s1 + 1] - offs[s0]).astype(np.uint64)
        rc, o_iv, o_ioffs, o_am, o_aoffs, _ = oracle.pair(ev, sub, R)
        assert rc == 0
        rc, want, _ = oracle.aggregate_scoped(o_iv, o_ioffs, o_am, o_aoffs, W, np.zeros(1, np.uint32), 1, R,
                                              scope={"ctx": (lo, hi), "warps": warps}, levels=("warp", "cta"))
        assert rc == 0
        assert warp[s0:s1].tobytes() == want["warp"].tobytes(), f"warp rows of CTA {c} differ"
        assert sc.table_numpy("cta")[c:c + 1].tobytes() == want["cta"].tobytes(), f"CTA row {c} differs"
    del res, sc
    torch.cuda.empty_cache()
