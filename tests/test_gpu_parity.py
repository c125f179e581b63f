"""Parity of the CUDA path (through the C-ABI) against the CPU oracle: bit-exact, element by element.
Everything here needs a GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from helpers import load_example, make_events, random_wellformed
from paper_2609_12299_b200 import tracegen as tg
from paper_2609_12299_b200.binding import KERNEL_THREAD_PER_STREAM, KERNEL_TILED

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KERNELS = [KERNEL_THREAD_PER_STREAM, KERNEL_TILED]


def to_dev(ev, offs):
    d_ev = torch.from_numpy(np.ascontiguousarray(ev).view(np.uint8).reshape(-1).copy()).to(DEV)
    d_off = torch.from_numpy(np.ascontiguousarray(offs, dtype=np.uint64).view(np.int64).copy()).to(DEV)
    return d_ev, d_off


def run_pair(ev, offs, R, kernel, **kw):
    d_ev, d_off = to_dev(ev, offs)
    pr = argus.argus_pair_intervals(d_ev, d_off, R, kernel=kernel, **kw)
    return pr, pr.fetch_status()


def assert_pair_matches(ev, offs, R, kernel, **kw):
    pr, st = run_pair(ev, offs, R, kernel, **kw)
    rc, o_iv, o_ioffs, o_am, o_aoffs, o_st = oracle.pair(ev, offs, R)
    assert rc == 0 and int(o_st["code"]) == 0
    assert int(st["code"]) == 0, f"device status {st}"
    assert np.array_equal(pr.interval_offsets.cpu().numpy().view(np.uint64), o_ioffs)
    assert np.array_equal(pr.ambig_offsets.cpu().numpy().view(np.uint64), o_aoffs)
    g_iv, g_am = pr.intervals_numpy(), pr.ambig_numpy()
    if g_iv.tobytes() != o_iv.tobytes():
        bad = np.nonzero(g_iv != o_iv)[0]
        raise AssertionError(f"{len(bad)} intervals differ; first at {bad[0]}: gpu {g_iv[bad[0]]} oracle {o_iv[bad[0]]}")
    if g_am.tobytes() != o_am.tobytes():
        bad = np.nonzero(g_am != o_am)[0]
        raise AssertionError(f"{len(bad)} ambiguity records differ; first at {bad[0]}: gpu {g_am[bad[0]]} oracle {o_am[bad[0]]}")
    for f in ("intervals_required", "ambig_required", "n_ctx_mismatch", "n_time_reversed", "n_child_clamped"):
        assert int(st[f]) == int(o_st[f]), f
    pr.last_status = st
    return pr, (o_iv, o_ioffs, o_am, o_aoffs)


EXAMPLES = ["example_a_wellformed.txt", "example_b_dropped_end.txt", "example_c_dup_stray_trunc.txt",
            "example_e_ctx_ignored.txt", "example_f_greedy.txt", "example_g_boundary.txt", "example_h_flags.txt"]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("name", EXAMPLES)
def test_hand_worked_examples(name, kernel):
    ev, _, _ = load_example(name)
    assert_pair_matches(ev, np.array([0, len(ev)], np.uint64), 8, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_tracegen_host_equals_device_and_config0(kernel):
    spec = tg.config(0)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = tg.generate_cuda(spec, DEV)
    assert d_ev.cpu().numpy().tobytes() == ev.tobytes()
    assert np.array_equal(d_off.cpu().numpy().view(np.uint64), offs)
    assert_pair_matches(ev, offs, spec.num_regions, kernel)


@pytest.mark.parametrize("idx,ctas,iters", [(1, 5, 60), (2, 3, 2), (3, 2, 3), (4, 6, 80)])
def test_tracegen_host_equals_device_scaled(idx, ctas, iters):
    spec = tg.config(idx).scaled(ctas, iters)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = tg.generate_cuda(spec, DEV)
    assert np.array_equal(d_off.cpu().numpy().view(np.uint64), offs)
    assert d_ev.cpu().numpy().tobytes() == ev.tobytes()


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("idx,ctas,iters", [(1, 7, 300), (2, 3, 3), (3, 3, 9), (4, 9, 400)])
def test_scaled_configs_full_pipeline(idx, ctas, iters, kernel):
    """Pair + aggregate + overlap on scaled-down versions of configs 1-4 (several tiles per stream and a ragged tail)."""
    spec = tg.config(idx).scaled(ctas, iters)
    ev, offs = tg.generate_host(spec)
    pr, (o_iv, o_ioffs, o_am, o_aoffs) = assert_pair_matches(ev, offs, spec.num_regions, kernel)
    if kernel == KERNEL_TILED and spec.well_formed:
        # well-formed traces must stay on the parallel path of the tiled kernel
        assert int(pr.last_status["n_sequential_tiles"]) == 0
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    ag = argus.argus_aggregate(pr.intervals, pr.interval_offsets, pr.ambig, pr.ambig_offsets, spec.warps_per_cta, cta_sm,
                               spec.num_sms, spec.num_regions)
    assert int(argus.argus_status_fetch(ag.status)["code"]) == 0
    _, o_tabs, _ = oracle.aggregate(o_iv, o_ioffs, o_am, o_aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms,
                                    spec.num_regions)
    for lv in ("warp", "cta", "sm", "kernel"):
        assert ag.table_numpy(lv).tobytes() == o_tabs[lv].tobytes(), lv
    pairs_np = np.concatenate([spec.overlap_pairs, spec.overlap_pairs[:, ::-1], [[0, 0]]]).astype(np.uint32)
    pairs = torch.from_numpy(pairs_np.view(np.int32)).to(DEV)
    ov, ov_st = argus.argus_overlap(pr.intervals, pr.interval_capacity, pr.interval_offsets, spec.warps_per_cta, cta_sm,
                                    spec.num_sms, pairs)
    assert int(argus.argus_status_fetch(ov_st)["code"]) == 0
    _, o_ov, _ = oracle.overlap(o_iv, o_ioffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, pairs_np)
    assert ov.cpu().numpy().view(argus.OVERLAP_DTYPE).reshape(o_ov.shape).tobytes() == o_ov.tobytes()


@pytest.mark.parametrize("kernel", KERNELS)
def test_random_malformed_streams(kernel):
    rng = np.random.default_rng(11)
    evs, offs = [], [0]
    for s in range(96):
        n_pairs = int(rng.integers(0, 3000 if s % 7 == 0 else 200))
        ev = random_wellformed(rng, n_pairs, 6, max_height=int(rng.integers(1, 12))) if n_pairs else make_events([])
        mode = s % 4
        if mode == 1 and len(ev):
            ev = ev[rng.random(len(ev)) > 0.02]              # drop markers of either kind
        elif mode == 2 and len(ev):
            ev = np.repeat(ev, 1 + (rng.random(len(ev)) < 0.02))  # duplicate markers
        elif mode == 3 and len(ev) > 2:
            ev = ev[int(rng.integers(0, len(ev))):]            # cut the head: leading unmatched ends
            if rng.random() < 0.5:
                ev = ev.copy()
                ev["ts"][rng.random(len(ev)) < 0.05] -= 500   # timestamps that run backwards
                ev["ctx"][rng.random(len(ev)) < 0.05] += 1
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    ev = np.concatenate(evs)
    assert_pair_matches(ev, np.array(offs, np.uint64), 6, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_deep_and_adversarial_streams(kernel):
    rows = [(i, "B", i % 3, 0) for i in range(64)] + [(100 + i, "E", (63 - i) % 3, 0) for i in range(64)]
    deep = make_events(rows)                                           # full depth, well formed
    only_ends = make_events([(i, "E", i % 4, 1) for i in range(5000)])  # every marker ambiguous
    only_begins = make_events([(i, "B", 0, 1) for i in range(64)])
    sawtooth = make_events([(i, "BE"[i % 2], 0, i) for i in range(6001)])  # ctx mismatch on every interval, odd length
    wide = make_events([(7 * i, "B", 1, 0) for i in range(40)] + [(1000, "E", 0, 0)] +
                       [(2000 + i, "E", 1, 0) for i in range(40)])    # stray end under a deep stack
    evs = [deep, only_ends, only_begins, sawtooth, wide, make_events([])]
    offs = np.cumsum([0] + [len(e) for e in evs]).astype(np.uint64)
    assert_pair_matches(np.concatenate(evs), offs, 4, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_edges_and_error_codes(kernel):
    ev = make_events([(1, "B", 0, 0), (2, "E", 0, 0), (5, "B", 1, 3), (9, "E", 1, 3)])
    # offsets that do not start at zero, empty streams
    assert_pair_matches(ev, np.array([2, 2, 4, 4], np.uint64), 2, kernel)
    # no events at all, but streams exist
    assert_pair_matches(ev[:0], np.array([0, 0, 0], np.uint64), 2, kernel)
    # bad region id
    pr, st = run_pair(ev, np.array([0, 4], np.uint64), 1, kernel)
    assert int(st["code"]) == 6 and int(st["bad_stream"]) == 0 and int(st["bad_event"]) == 2
    # 65 open frames
    deep = make_events([(i, "B", 0, 0) for i in range(65)])
    pr, st = run_pair(deep, np.array([0, 65], np.uint64), 1, kernel)
    assert int(st["code"]) == 5 and int(st["bad_event"]) == 64
    # interval capacity too small: required count reported
    many = make_events([(i, "BE"[i % 2], 0, 0) for i in range(200)])
    pr, st = run_pair(many, np.array([0, 200], np.uint64), 1, kernel, interval_capacity=10)
    assert int(st["code"]) == 4 and int(st["intervals_required"]) == 100
    # ambiguity capacity too small
    ends = make_events([(i, "E", 0, 0) for i in range(100)])
    pr, st = run_pair(ends, np.array([0, 100], np.uint64), 1, kernel, ambig_capacity=7)
    assert int(st["code"]) == 4 and int(st["ambig_required"]) == 100
    # decreasing offsets, offsets beyond the buffer
    pr, st = run_pair(ev, np.array([0, 3, 2], np.uint64), 2, kernel)
    assert int(st["code"]) == 7
    pr, st = run_pair(ev, np.array([0, 9], np.uint64), 2, kernel)
    assert int(st["code"]) == 7
    # the context stays usable after every error
    assert_pair_matches(ev, np.array([0, 4], np.uint64), 2, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_exact_capacity_with_malformed_trace(kernel):
    """Capacity equal to the true interval count: provisional positions overflow, the second pass fixes them."""
    spec = tg.config(4).scaled(3, 120)
    ev, offs = tg.generate_host(spec)
    _, o_iv, _, o_am, _, _ = oracle.pair(ev, offs, spec.num_regions)
    assert_pair_matches(ev, offs, spec.num_regions, kernel, interval_capacity=len(o_iv), ambig_capacity=len(o_am))


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("where", ["first", "middle", "last"])
def test_one_malformed_stream_among_wellformed_ones(kernel, where):
    """One stream loses an end marker: the streams before it keep their place in the interval array (the second
    pass leaves them alone), the ones after it move up by one."""
    spec = tg.config(3).scaled(3, 4)
    ev, offs = tg.generate_host(spec)
    S = spec.num_streams
    k = {"first": 0, "middle": S // 2, "last": S - 1}[where]
    lo, hi = int(offs[k]), int(offs[k + 1])
    ends = np.nonzero(ev["tag"][lo:hi] & 1)[0]
    drop = lo + int(ends[len(ends) // 2])
    ev2 = np.delete(ev, drop)
    offs2 = offs.copy()
    offs2[k + 1:] -= 1
    pr, (o_iv, _, o_am, _) = assert_pair_matches(ev2, offs2, spec.num_regions, kernel)
    assert len(o_am) >= 1 and len(o_iv) < len(ev2) // 2 + 1
    # and through the one-call pipeline (digests follow the intervals)
    _synthesize_matches(spec, ev2, offs2)


def test_invalid_arguments_raise():
    ev = make_events([(1, "B", 0, 0), (2, "E", 0, 0)])
    d_ev, d_off = to_dev(ev, np.array([0, 2], np.uint64))
    with pytest.raises(argus.ArgusError):
        argus.argus_pair_intervals(d_ev, d_off, 0)
    with pytest.raises(argus.ArgusError):
        argus.argus_pair_intervals(d_ev, d_off, 70000)
    pr = argus.argus_pair_intervals(d_ev, d_off, 1)
    cta_sm = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(argus.ArgusError):
        argus.argus_aggregate(pr.intervals, pr.interval_offsets, None, None, 2, cta_sm, 1, 1)  # S % W != 0
    small_ws = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(argus.ArgusError) as e:
        argus.argus_pair_intervals(d_ev, d_off, 1, out=argus.PairResult(pr.intervals, pr.interval_offsets, pr.ambig,
                                   pr.ambig_offsets, pr.status, 1, 2, small_ws))
    assert e.value.code == 2


def test_aggregate_large_region_count_and_null_tables():
    """num_regions too large for a shared-memory table (global-row path) and nullable outputs."""
    rng = np.random.default_rng(5)
    R = 600
    evs, offs = [], [0]
    for s in range(8):
        ev = random_wellformed(rng, 500, R, max_height=5)
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    ev, offs = np.concatenate(evs), np.array(offs, np.uint64)
    pr, (o_iv, o_ioffs, o_am, o_aoffs) = assert_pair_matches(ev, offs, R, KERNEL_THREAD_PER_STREAM)
    cta_sm_np = np.array([1, 0, 1, 2], np.uint32)
    cta_sm = torch.from_numpy(cta_sm_np.view(np.int32)).to(DEV)
    _, o_tabs, _ = oracle.aggregate(o_iv, o_ioffs, o_am, o_aoffs, 2, cta_sm_np, 3, R)
    ag = argus.argus_aggregate(pr.intervals, pr.interval_offsets, pr.ambig, pr.ambig_offsets, 2, cta_sm, 3, R)
    for lv in ("warp", "cta", "sm", "kernel"):
        assert ag.table_numpy(lv).tobytes() == o_tabs[lv].tobytes(), lv
    ag2 = argus.argus_aggregate(pr.intervals, pr.interval_offsets, None, None, 2, cta_sm, 3, R, levels=("kernel",))
    assert ag2.table_numpy("kernel").tobytes() == o_tabs["kernel"].tobytes()
    ag3 = argus.argus_aggregate(pr.intervals, pr.interval_offsets, None, None, 2, cta_sm, 3, R, levels=("sm",))
    assert ag3.table_numpy("sm").tobytes() == o_tabs["sm"].tobytes()


def test_overlap_random_spans_and_capacity():
    rng = np.random.default_rng(8)
    S, W, M, R = 24, 3, 4, 5
    cta_sm_np = rng.integers(0, M, S // W).astype(np.uint32)
    rows = []
    for s in range(S):
        for _ in range(int(rng.integers(0, 3000 if s % 5 == 0 else 50))):
            rows.append((s, int(rng.integers(0, R)), int(rng.integers(0, 1 << 40)) + (1 << 60), int(rng.integers(0, 1 << 30))))
    rows.sort(key=lambda r: r[0])
    iv = np.zeros(len(rows), argus.INTERVAL_DTYPE)
    arr = np.array(rows, dtype=np.uint64)
    iv["stream"], iv["region"], iv["t_begin"], iv["inclusive"] = arr[:, 0], arr[:, 1], arr[:, 2], arr[:, 3]
    ioffs = np.zeros(S + 1, np.uint64)
    ioffs[1:] = np.cumsum(np.bincount(arr[:, 0].astype(np.int64), minlength=S))
    pairs_np = np.array([(0, 1), (1, 0), (2, 2), (3, 4), (4, 0)], np.uint32)
    _, o_ov, _ = oracle.overlap(iv, ioffs, W, cta_sm_np, M, pairs_np)
    d_iv = torch.from_numpy(iv.view(np.uint8).reshape(-1).copy()).to(DEV)
    d_off = torch.from_numpy(ioffs.view(np.int64).copy()).to(DEV)
    cta_sm = torch.from_numpy(cta_sm_np.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(pairs_np.view(np.int32)).to(DEV)
    ov, st = argus.argus_overlap(d_iv, len(iv), d_off, W, cta_sm, M, pairs)
    assert int(argus.argus_status_fetch(st)["code"]) == 0
    assert ov.cpu().numpy().view(argus.OVERLAP_DTYPE).reshape(o_ov.shape).tobytes() == o_ov.tobytes()
    # a workspace too small for the selected spans is reported, not overrun
    ov, st = argus.argus_overlap(d_iv, len(iv), d_off, W, cta_sm, M, pairs, workspace_bytes=64 * 1024)
    assert int(argus.argus_status_fetch(st)["code"]) == 4


@pytest.mark.parametrize("shape", ["even", "same-start", "crowded-with-outliers", "huge-range", "one-bucket-over"])
def test_overlap_segment_sort_paths(shape):
    """Large segments are sorted by buckets of start time, or by the full network when the starts crowd:
    starts spread evenly; thousands of equal starts; nearly all starts in a narrow window with a few far outliers;
    starts over the whole 64-bit range; one bucket just over its capacity."""
    rng = np.random.default_rng(len(shape))
    S, W, M, R = 4, 2, 2, 2
    n = 20000
    cta_sm_np = np.array([0, 1], np.uint32)
    iv = np.zeros(S * n, argus.INTERVAL_DTYPE)
    for s in range(S):
        if shape == "even":
            t = (1 << 50) + np.sort(rng.integers(0, 1 << 34, n)).astype(np.uint64)
        elif shape == "same-start":
            t = np.full(n, 777, np.uint64)
            t[: n // 2] += rng.integers(0, 3, n // 2).astype(np.uint64)
        elif shape == "crowded-with-outliers":
            t = (1 << 40) + rng.integers(0, 5000, n).astype(np.uint64)
            t[:5] = (1 << 62) + rng.integers(0, 100, 5).astype(np.uint64)
        elif shape == "huge-range":
            t = rng.integers(0, 1 << 63, n).astype(np.uint64) * np.uint64(2) + rng.integers(0, 2, n).astype(np.uint64)
            t = np.minimum(t, np.uint64((1 << 64) - (1 << 33)))
        else:
            t = np.arange(n, dtype=np.uint64) * np.uint64(1000)
            t[100:230] = t[100]          # 130 equal starts: more than a bucket holds
        sl = slice(s * n, (s + 1) * n)
        iv["stream"][sl] = s
        iv["region"][sl] = rng.integers(0, R, n)
        iv["t_begin"][sl] = t
        iv["inclusive"][sl] = rng.integers(0, 1 << 20, n)
    ioffs = (np.arange(S + 1) * n).astype(np.uint64)
    pairs_np = np.array([(0, 1), (1, 1)], np.uint32)
    _, o_ov, _ = oracle.overlap(iv, ioffs, W, cta_sm_np, M, pairs_np)
    d_iv = torch.from_numpy(iv.view(np.uint8).reshape(-1).copy()).to(DEV)
    d_off = torch.from_numpy(ioffs.view(np.int64).copy()).to(DEV)
    ov, st = argus.argus_overlap(d_iv, len(iv), d_off, W, torch.from_numpy(cta_sm_np.view(np.int32)).to(DEV), M,
                                 torch.from_numpy(pairs_np.view(np.int32)).to(DEV))
    assert int(argus.argus_status_fetch(st)["code"]) == 0
    assert ov.cpu().numpy().view(argus.OVERLAP_DTYPE).reshape(o_ov.shape).tobytes() == o_ov.tobytes()


def _synthesize_matches(spec, ev, offs, **kw):
    d_ev, d_off = to_dev(ev, offs)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs_np = np.concatenate([spec.overlap_pairs, spec.overlap_pairs[:, ::-1], [[0, 0]]]).astype(np.uint32)
    pairs = torch.from_numpy(pairs_np.view(np.int32)).to(DEV)
    res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs, **kw)
    st = res.fetch_status()
    assert int(st["code"]) == 0, st
    rc, o_iv, o_ioffs, o_am, o_aoffs, o_st = oracle.pair(ev, offs, spec.num_regions)
    assert res.pair.intervals_numpy().tobytes() == o_iv.tobytes()
    assert res.pair.ambig_numpy().tobytes() == o_am.tobytes()
    assert np.array_equal(res.pair.interval_offsets.cpu().numpy().view(np.uint64), o_ioffs)
    assert np.array_equal(res.pair.ambig_offsets.cpu().numpy().view(np.uint64), o_aoffs)
    _, o_tabs, _ = oracle.aggregate(o_iv, o_ioffs, o_am, o_aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms,
                                    spec.num_regions)
    for lv in kw.get("levels", ("warp", "cta", "sm", "kernel")):
        got, want = res.agg.table_numpy(lv), o_tabs[lv]
        if got.tobytes() != want.tobytes():
            bad = np.argwhere(got != want)
            raise AssertionError(f"{lv}: {len(bad)} cells differ; first {bad[0]}: gpu {got[tuple(bad[0])]} oracle {want[tuple(bad[0])]}")
    _, o_ov, _ = oracle.overlap(o_iv, o_ioffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, pairs_np)
    assert res.overlap_numpy(spec.num_sms).tobytes() == o_ov.tobytes()
    return res, st


@pytest.fixture(params=[-1, 1, 2, 3], ids=["auto", "one-pass-digests", "plain-calls", "one-pass-records"])
def synth_mode(request):
    """Where argus_synthesize aggregates and selects overlap spans; results must not depend on it."""
    from paper_2609_12299_b200.binding import argus_set_synthesize_mode
    argus_set_synthesize_mode(request.param)
    yield request.param
    argus_set_synthesize_mode(-1)


@pytest.mark.parametrize("idx,ctas,iters", [(0, 4, 626), (1, 7, 300), (2, 3, 3), (3, 3, 9), (4, 9, 400)])
def test_synthesize_matches_oracle_in_every_mode(idx, ctas, iters, synth_mode):
    """One-call pipeline in each of its modes."""
    spec = tg.config(idx).scaled(ctas, iters)
    ev, offs = tg.generate_host(spec)
    res, st = _synthesize_matches(spec, ev, offs)
    if spec.well_formed:
        assert int(st["n_sequential_tiles"]) == 0


@pytest.mark.parametrize("levels", [("kernel",), ("sm",), ("cta", "kernel"), ("warp",), ()])
def test_synthesize_table_subsets(levels, synth_mode):
    """Any subset of the four tables may be asked for (none: intervals and overlap only)."""
    spec = tg.config(3).scaled(2, 5)
    ev, offs = tg.generate_host(spec)
    _synthesize_matches(spec, ev, offs, levels=levels)


def test_synthesize_wide_histogram_and_flags(synth_mode):
    """Durations spread over many log2 bins (outside the 16-bin shared-memory window), flagged intervals,
    min/max extremes and a region that never occurs."""
    rng = np.random.default_rng(21)
    spec = tg.TraceSpec(tg.GEMM, 2, 1)  # only for warps_per_cta / cta_sm / pairs
    S = spec.num_streams
    evs, offs = [], [0]
    for s in range(S):
        rows, t = [], 1 << 40
        for i in range(int(rng.integers(200, 3000))):
            r = int(rng.integers(0, 4))
            d = int(2 ** rng.uniform(0, 50)) if rng.random() < 0.9 else 0
            rows.append((t, "B", r, i))
            inner = int(rng.integers(0, d + 1))
            if rng.random() < 0.5:
                rows.append((t + 1, "B", (r + 1) % 4, i))
                rows.append((t + 1 + inner, "E", (r + 1) % 4, i + (1 if rng.random() < 0.05 else 0)))
            t_end = t + d - (2 * d if rng.random() < 0.02 else 0)
            rows.append((t_end, "E", r, i))
            t += d + int(rng.integers(0, 100))
        ev = make_events(rows)
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    _synthesize_matches(spec, np.concatenate(evs), np.array(offs, np.uint64))


def test_synthesize_hot_regions_long_streams(synth_mode):
    """Streams long enough for the digest pass to give the most frequent regions their per-lane copies: two regions
    own most intervals; durations just below and above the digest's 23 bits, so that the 32-bit sums of the
    copies carry, bins fall outside a region's window, and wide digests send lanes to the records."""
    rng = np.random.default_rng(77)
    spec = tg.TraceSpec(tg.GEMM, 1, 1)  # only for warps_per_cta / cta_sm / pairs
    S = spec.num_streams
    evs, offs = [], [0]
    for s in range(S):
        n = 120000 if s % 3 == 0 else 9000
        region = rng.choice(5, size=n, p=[0.45, 0.4, 0.05, 0.05, 0.05]).astype(np.uint64)
        kind = rng.random(n)
        dur = np.where(kind < 0.6, rng.integers(1 << 21, 1 << 23, n),
                       np.where(kind < 0.9, rng.integers(0, 300, n),
                                np.where(kind < 0.97, rng.integers(1 << 23, 1 << 36, n), 2 ** rng.integers(0, 23, n)))).astype(np.uint64)
        gap = rng.integers(0, 50, n).astype(np.uint64)
        t_begin = (np.uint64(1) << np.uint64(33)) + np.concatenate([[0], np.cumsum(dur + gap)[:-1]]).astype(np.uint64)
        ev = np.zeros(2 * n, argus.EVENT_DTYPE)
        ev["ts"][0::2] = t_begin
        ev["ts"][1::2] = t_begin + dur
        ev["tag"][0::2] = (region << np.uint64(1)).astype(np.uint32)
        ev["tag"][1::2] = ((region << np.uint64(1)) | np.uint64(1)).astype(np.uint32)
        ctx = np.arange(n, dtype=np.uint32)
        ev["ctx"][0::2] = ctx
        ev["ctx"][1::2] = ctx + (rng.random(n) < 0.01)  # a few context mismatches: flagged intervals
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    _synthesize_matches(spec, np.concatenate(evs), np.array(offs, np.uint64))


@pytest.mark.parametrize("R", [300, 500])
def test_synthesize_many_regions(R):
    """300 regions: more than the pairing kernel's table holds (one pass over the intervals instead);
    500: more than the compact aggregation table holds (the plain calls)."""
    rng = np.random.default_rng(5)
    spec = tg.TraceSpec(tg.TINY, 2, 1)
    evs, offs = [], [0]
    for s in range(spec.num_streams):
        ev = random_wellformed(rng, 400, R, max_height=5)
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    ev, offs = np.concatenate(evs), np.array(offs, np.uint64)

    class Spec:  # same fields _synthesize_matches reads
        num_regions, warps_per_cta, cta_sm, num_sms = R, 4, spec.cta_sm, spec.num_sms
        overlap_pairs = np.array([(1, 2), (7, R - 1)], np.uint32)
    _synthesize_matches(Spec, ev, offs)


def test_synthesize_overlap_span_capacity():
    spec = tg.config(2).scaled(2, 2)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = to_dev(ev, offs)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs,
                                 max_overlap_spans=512)
    st = res.fetch_status()
    assert int(st["code"]) == 4 and int(st["intervals_required"]) > 512


@pytest.mark.parametrize("idx,ctas,iters", [(0, 4, 626), (1, 7, 300), (2, 3, 3), (3, 3, 9), (4, 9, 400)])
def test_outputs_repeat_byte_for_byte(idx, ctas, iters):
    """The same call twice on fresh buffers: every output byte is the same (all device-side accumulation is integer
    atomics, ranks come from prefix sums, spans are sorted before they are measured)."""
    spec = tg.config(idx).scaled(ctas, iters)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = to_dev(ev, offs)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    runs = []
    for _ in range(2):
        res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs)
        assert int(res.fetch_status()["code"]) == 0
        runs.append([res.pair.intervals_numpy().tobytes(), res.pair.ambig_numpy().tobytes(),
                     res.pair.interval_offsets.cpu().numpy().tobytes(), res.pair.ambig_offsets.cpu().numpy().tobytes(),
                     res.overlap.cpu().numpy().tobytes(), res.status.cpu().numpy().tobytes()] +
                    [res.agg.table_numpy(lv).tobytes() for lv in ("warp", "cta", "sm", "kernel")])
    assert runs[0] == runs[1]


def _fuzz_case(seed):
    """A random trace shape: stream count, region count, SM map, pairs; streams of random length, some empty, some
    corrupted (dropped and duplicated markers, flipped kinds, changed regions, time running backwards, huge gaps)."""
    rng = np.random.default_rng(1000 + seed)
    W = int(rng.choice([1, 2, 4, 8, 16]))
    C = int(rng.integers(1, 7))
    S = W * C
    R = int(rng.choice([1, 2, 5, 37, 300, 500]))
    M = int(rng.integers(1, 5))
    evs, offs = [], [0]
    for s in range(S):
        kind = rng.random()
        n_pairs = 0 if kind < 0.1 else int(rng.integers(1, 1500 if kind < 0.9 else 12000))
        ev = random_wellformed(rng, n_pairs, R, max_height=int(rng.integers(1, 9)), t0=int(rng.integers(0, 1 << 45)))
        if len(ev) and rng.random() < 0.5:      # corrupt it
            n = len(ev)
            keep = rng.random(n) > 0.003
            ev = ev[keep]
            n = len(ev)
            if n:
                flip = rng.random(n) < 0.002
                ev["tag"][flip] ^= 1
                chg = rng.random(n) < 0.002
                ev["tag"][chg] = (rng.integers(0, R, int(chg.sum())).astype(np.uint32) << 1) | (ev["tag"][chg] & 1)
                back = rng.random(n) < 0.002
                ev["ts"][back] -= np.minimum(ev["ts"][back], rng.integers(1, 1000, int(back.sum())).astype(np.uint64))
                jump = rng.random(n) < 0.001
                ev["ts"] += np.cumsum(np.where(jump, rng.integers(1 << 30, 1 << 40, n), 0)).astype(np.uint64)
                dup = np.nonzero(rng.random(n) < 0.002)[0]
                ev = np.insert(ev, dup, ev[dup])
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    K = int(rng.integers(0, 5))

    class Spec:
        num_regions, warps_per_cta, num_sms = R, W, M
        cta_sm = rng.integers(0, M, C).astype(np.uint32)
        overlap_pairs = rng.integers(0, R, (K, 2)).astype(np.uint32)
    ev = np.concatenate(evs) if evs else np.zeros(0, argus.EVENT_DTYPE)
    return Spec, ev.astype(argus.EVENT_DTYPE), np.array(offs, np.uint64)


@pytest.mark.parametrize("seed", list(range(16)) + [305])   # 305: a stream that opens a 65th frame
def test_synthesize_random_shapes(seed, synth_mode):
    spec, ev, offs = _fuzz_case(seed)
    rc, _, _, _, _, o_st = oracle.pair(ev, offs, spec.num_regions)
    if int(o_st["code"]) != 0:   # the random corruption opened more than 64 frames: the same error is reported
        d_ev, d_off = to_dev(ev, offs)
        cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
        st = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, None).fetch_status()
        assert int(st["code"]) == int(o_st["code"])
        return
    _synthesize_matches(spec, ev, offs)


def test_synthesize_empty_inputs(synth_mode):
    """Streams without events, and no streams at all: empty outputs, zeroed tables, status clean."""
    spec = tg.TraceSpec(tg.TINY, 2, 1)   # 8 streams, 4 warps per CTA
    ev = make_events([])
    _synthesize_matches(spec, ev, np.zeros(spec.num_streams + 1, np.uint64))

    class NoStreams:
        num_regions, warps_per_cta, num_sms = 3, 4, 2
        cta_sm = np.zeros(0, np.uint32)
        overlap_pairs = np.array([(0, 1)], np.uint32)
    _synthesize_matches(NoStreams, ev, np.zeros(1, np.uint64))


def test_synthesize_interval_capacity_too_small(synth_mode):
    """Fewer interval slots than the trace needs: the call reports ARGUS_ERR_CAPACITY with the required count, the
    later stages read nothing beyond the array, and the same buffers work again with enough room."""
    spec = tg.config(1).scaled(2, 40)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = to_dev(ev, offs)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    need = len(ev) // 2
    res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs,
                                 interval_capacity=need // 3)
    st = res.fetch_status()
    assert int(st["code"]) == 4 and int(st["intervals_required"]) == need
    _synthesize_matches(spec, ev, offs)


def test_synthesize_ambiguity_capacity_too_small(synth_mode):
    """Fewer ambiguity slots than a malformed trace needs: ARGUS_ERR_CAPACITY with the required count; the offsets the
    call leaves behind stay inside the arrays, so the aggregation behind it (no host check in between) reads nothing
    beyond them; the same buffers work again with enough room."""
    spec = tg.config(4).scaled(3, 300)
    ev, offs = tg.generate_host(spec)
    rc, o_iv, o_ioffs, o_am, o_aoffs, o_st = oracle.pair(ev, offs, spec.num_regions)
    assert len(o_am) > 40
    d_ev, d_off = to_dev(ev, offs)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    cap = len(o_am) // 3
    res = argus.argus_synthesize(d_ev, d_off, spec.num_regions, spec.warps_per_cta, cta_sm, spec.num_sms, pairs,
                                 ambig_capacity=cap)
    st = res.fetch_status()
    assert int(st["code"]) == 4 and int(st["ambig_required"]) == len(o_am)
    assert int(res.pair.ambig_offsets.cpu().numpy().view(np.uint64).max()) <= cap
    # the plain chain: pairing that overflows, then aggregation of what it left, without looking at the status
    pr = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions, ambig_capacity=cap, interval_capacity=len(o_iv) // 2)
    ag = argus.argus_aggregate(pr.intervals, pr.interval_offsets, pr.ambig, pr.ambig_offsets, spec.warps_per_cta, cta_sm,
                               spec.num_sms, spec.num_regions)
    torch.cuda.synchronize()
    assert int(pr.fetch_status()["code"]) == 4
    assert int(pr.interval_offsets.cpu().numpy().view(np.uint64).max()) <= len(o_iv) // 2
    _synthesize_matches(spec, ev, offs)


def test_overlap_offsets_beyond_the_interval_array_are_reported():
    spec = tg.config(1).scaled(2, 40)
    ev, offs = tg.generate_host(spec)
    d_ev, d_off = to_dev(ev, offs)
    pr = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions)
    cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(DEV)
    pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(DEV)
    n_iv = int(pr.interval_offsets[-1].item())
    _, st = argus.argus_overlap(pr.intervals, n_iv // 2, pr.interval_offsets, spec.warps_per_cta, cta_sm, spec.num_sms, pairs)
    assert int(argus.argus_status_fetch(st)["code"]) == 7  # ARGUS_ERR_BAD_OFFSETS


def test_maximum_region_count():
    """num_regions at its upper bound (65536): pairing, the global-row aggregation path and the one-call
    pipeline (which cannot host such a table in shared memory and runs the three plain calls)."""
    R = 65536
    rng = np.random.default_rng(33)
    spec = tg.TraceSpec(tg.TINY, 2, 1)
    evs, offs = [], [0]
    for s in range(spec.num_streams):
        ev = random_wellformed(rng, 300, 7, max_height=4)
        ev = ev.copy()
        ev["tag"] = ((ev["tag"] >> 1) * 10922 + (R - 1 - 6 * 10922)).astype(np.uint32) << 1 | (ev["tag"] & 1)  # ids up to R-1
        evs.append(ev)
        offs.append(offs[-1] + len(ev))
    ev, offs = np.concatenate(evs), np.array(offs, np.uint64)
    assert int((ev["tag"] >> 1).max()) == R - 1

    class Spec:
        num_regions, warps_per_cta, cta_sm, num_sms = R, 4, spec.cta_sm, spec.num_sms
        overlap_pairs = np.array([(R - 1, R - 1 - 10922)], np.uint32)
    _synthesize_matches(Spec, ev, offs)
    # one region too many is rejected on the host
    d_ev, d_off = to_dev(ev, offs)
    with pytest.raises(argus.ArgusError):
        argus.argus_pair_intervals(d_ev, d_off, R + 1)


def test_single_long_stream_and_many_empty_streams():
    """One stream of many tiles among empty ones (ragged CSR), and a stream that ends inside a tile."""
    rng = np.random.default_rng(34)
    long_ev = random_wellformed(rng, 20000, 5, max_height=9)
    short_ev = random_wellformed(rng, 3, 5)
    evs = [make_events([])] * 5 + [long_ev] + [make_events([])] * 3 + [short_ev] + [make_events([])] * 2
    offs = np.cumsum([0] + [len(e) for e in evs]).astype(np.uint64)
    for kernel in KERNELS:
        assert_pair_matches(np.concatenate(evs), offs, 5, kernel)


def test_long_streams_walked_in_chunks():
    """Streams several chunks long (the tiled kernel hands a stream from CTA to CTA every 32 K events, with the
    open frames and their child time in a record): deep stacks carried across hand-overs, defects, a stream
    shorter than a chunk beside them, and more CTAs than streams (idle CTAs wait for hand-overs)."""
    rng = np.random.default_rng(35)
    evs = [random_wellformed(rng, 150_000, 6, max_height=40), random_wellformed(rng, 5_000, 6, max_height=3),
           random_wellformed(rng, 70_000, 6, max_height=12)]
    # defects in the third stream: dropped ends and duplicated begins
    ev = evs[2]
    keep = np.ones(len(ev), bool)
    ends = np.nonzero(ev["tag"] & 1)[0]
    keep[rng.choice(ends, 40, replace=False)] = False
    ev = ev[keep]
    dup = np.sort(rng.choice(np.nonzero((ev["tag"] & 1) == 0)[0], 25, replace=False))
    evs[2] = np.insert(ev, dup, ev[dup])
    offs = np.cumsum([0] + [len(e) for e in evs]).astype(np.uint64)
    pr, _ = assert_pair_matches(np.concatenate(evs), offs, 6, KERNEL_TILED)
    assert int(pr.last_status["ambig_required"]) > 0


@pytest.mark.parametrize("kernel", KERNELS)
def test_marker_with_all_ones_tag_is_a_bad_region(kernel):
    """A tag of all ones is an end marker of region 2^31 - 1, not an absent event: reported like any region id out of range."""
    rng = np.random.default_rng(37)
    ev = random_wellformed(rng, 900, 5, max_height=4)
    ev["tag"][1234] = 0xFFFFFFFF
    offs = np.array([0, len(ev)], np.uint64)
    rc, *_, o_st = oracle.pair(ev, offs, 5)
    d_ev, d_off = to_dev(ev, offs)
    pr = argus.argus_pair_intervals(d_ev, d_off, 5, kernel=kernel)
    st = pr.fetch_status()
    assert int(o_st["code"]) == 6 and int(st["code"]) == 6
    assert (int(st["bad_stream"]), int(st["bad_event"])) == (int(o_st["bad_stream"]), int(o_st["bad_event"])) == (0, 1234)


@pytest.mark.parametrize("kernel", KERNELS)
def test_child_time_beyond_32_bits_inside_a_tile(kernel):
    """The tiled kernel gathers what a window adds to a frame's child time in 32 bits and hands anything larger to
    the sequential machine: children that add up to more than 2^32 ticks under one parent, a single interval longer
    than 2^32 ticks, both inside one tile, and a frame carried over many tiles whose child time passes 2^32 on the way."""
    rows, t = [], 1_700_000_000_000_000_000
    rows.append((t, "B", 0, 1))
    for i in range(6):                       # six children of 1.2e9 ticks each: 7.2e9 > 2^32 under region 0
        rows.append((t + 10, "B", 1, 1)); t += 1_200_000_000; rows.append((t, "E", 1, 1))
    rows.append((t + 5, "B", 2, 1)); t += 9_000_000_000; rows.append((t, "E", 2, 1))   # one interval of 9e9 ticks
    rows.append((t + 7, "E", 0, 1))
    rows.append((t + 8, "B", 3, 2))          # a frame that stays open over several tiles
    for i in range(4000):
        rows.append((t + 9, "B", 1, 2)); t += 3_000_000; rows.append((t, "E", 1, 2))  # 4000 x 3e6 = 1.2e10 in all
    rows.append((t + 1, "E", 3, 2))
    ev = make_events(rows)
    offs = np.array([0, len(ev)], np.uint64)
    pr, _ = assert_pair_matches(ev, offs, 4, kernel)
    iv = pr.intervals_numpy()
    assert int(iv["exclusive"][iv["region"] == 3][0]) < int(iv["inclusive"][iv["region"] == 3][0]) - (1 << 33)


def test_bounded_wait_for_a_hand_over_runs_out_and_the_call_returns():
    """A block of the tiled kernel that has no stream left polls for hand-overs of long streams, and gives up after a
    bounded number of polls. With the limit set to almost nothing the wait runs out while the long stream's block is
    still busy: the call returns, the status says ARGUS_ERR_TIMEOUT, nothing hangs, and with the default limit the same
    buffers give the oracle's result."""
    lib = argus.load_library()
    rng = np.random.default_rng(36)
    evs = [random_wellformed(rng, 600_000, 6, max_height=8), random_wellformed(rng, 40, 6, max_height=3)]
    offs = np.cumsum([0] + [len(e) for e in evs]).astype(np.uint64)
    ev = np.concatenate(evs)
    d_ev, d_off = to_dev(ev, offs)
    lib.argus_testing_set_poll_limit(1)
    try:
        pr = argus.argus_pair_intervals(d_ev, d_off, 6, kernel=KERNEL_TILED)
        st = pr.fetch_status()
    finally:
        lib.argus_testing_set_poll_limit(0)
    assert int(st["code"]) == 8  # ARGUS_ERR_TIMEOUT
    assert_pair_matches(ev, offs, 6, KERNEL_TILED)


@pytest.mark.parametrize("idx,ctas,iters", [(3, 1, 40), (4, 2, 3000)])
def test_synthesize_long_streams(idx, ctas, iters):
    """The one-call pipeline on streams of 80 K to 110 K events (several hand-overs each), bit for bit."""
    spec = tg.config(idx).scaled(ctas, iters)
    ev, offs = tg.generate_host(spec)
    assert np.diff(offs).max() > 70_000
    _synthesize_matches(spec, ev, offs)


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_other_tile_shapes_give_the_same_result(variant):
    """The compiled alternatives to the default tile shape (threads x events per thread x CTAs per SM), on a
    malformed trace with streams several tiles long and on the one-call pipeline in every mode."""
    from paper_2609_12299_b200.binding import argus_set_synthesize_mode, argus_set_tile_variant
    spec = tg.config(4).scaled(3, 700)
    ev, offs = tg.generate_host(spec)
    argus_set_tile_variant(variant)
    try:
        assert_pair_matches(ev, offs, spec.num_regions, KERNEL_TILED)
        for mode in (1, 2):
            argus_set_synthesize_mode(mode)
            _synthesize_matches(spec, ev, offs)
    finally:
        argus_set_tile_variant(0)
        argus_set_synthesize_mode(-1)
