"""Parity of PC-to-region mapping (argus_pair_intervals on the marker encoding + argus_map_pc_counts:
bit-exact) and of attribution (argus_attribute: fp64, to rounding) against the CPU oracle, which walks
the abstract mapping-run records directly. Everything here needs a GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from paper_2609_12299_b200.tracegen.mapping import encode_map_events
from test_oracle_map_pins import load_map_example, random_map_trace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def gpu_counts(streams, R, P):
    enc = [encode_map_events(s["kind"], s["id"], s["count"], R)[0] for s in streams]
    offs = np.cumsum([0] + [len(e) for e in enc]).astype(np.uint64)
    ev = np.concatenate(enc) if enc else np.zeros(0, argus.EVENT_DTYPE)
    d_ev = torch.from_numpy(ev.view(np.uint8).reshape(-1).copy()).to(DEV)
    d_off = torch.from_numpy(offs.view(np.int64).copy()).to(DEV)
    pr = argus.argus_pair_intervals(d_ev, d_off, R + 1)
    assert int(pr.fetch_status()["code"]) == 0
    counts, status = argus.argus_map_pc_counts(pr.intervals, pr.interval_offsets, R, P)
    assert int(argus.argus_status_fetch(status)["code"]) == 0
    return counts


def check_attribution(counts_dev, want_counts, metric):
    rc, mhat, ent, alpha = oracle.attribute(want_counts, metric)
    assert rc == 0
    g_mhat, g_ent, g_alpha = argus.argus_attribute(counts_dev, torch.from_numpy(metric).to(DEV))
    g_mhat, g_ent, g_alpha = g_mhat.cpu().numpy(), g_ent.cpu().numpy(), g_alpha.cpu().numpy()
    assert np.array_equal(g_alpha, alpha)                       # one IEEE division per cell
    scale = (alpha * np.abs(metric)).sum(1)                     # sum_p |alpha m| per row
    assert np.all(np.abs(g_mhat - mhat) <= 1e-12 * scale + 1e-300), (g_mhat, mhat)
    assert np.allclose(g_ent, ent, rtol=0, atol=1e-14 * max(1.0, np.log(len(want_counts))))
    # no alpha output: same results
    m2, e2, none = argus.argus_attribute(counts_dev, torch.from_numpy(metric).to(DEV), want_alpha=False)
    assert none is None and np.array_equal(m2.cpu().numpy(), g_mhat) and np.array_equal(e2.cpu().numpy(), g_ent)


def test_hand_worked_example_on_gpu():
    ev, want, metric, want_mhat, want_ent = load_map_example()
    counts = gpu_counts([ev], 2, 3)
    assert np.array_equal(counts.cpu().numpy().view(np.uint64), want)
    mhat, ent, alpha = argus.argus_attribute(counts, torch.from_numpy(metric).to(DEV))
    assert np.allclose(mhat.cpu().numpy(), want_mhat, rtol=0, atol=1e-15)
    assert np.allclose(ent.cpu().numpy(), want_ent, rtol=0, atol=1e-15)


@pytest.mark.parametrize("p_bad,n,S,R,P", [(0.0, 3000, 24, 5, 11), (0.3, 3000, 24, 5, 11), (0.05, 40000, 6, 30, 3000)])
def test_random_mapping_traces(p_bad, n, S, R, P):
    """Well-formed and defective streams (mis-nested and unmatched ends), several tiles long, empty streams."""
    rng = np.random.default_rng(int(p_bad * 100) + n)
    streams = [random_map_trace(rng, int(rng.integers(0, n)) if s % 5 else 0, R, P, p_bad, max_depth=20) for s in range(S)]
    offs = np.cumsum([0] + [len(s) for s in streams]).astype(np.uint64)
    rc, want, st = oracle.map_pc_counts(np.concatenate(streams), offs, R, P)
    assert rc == 0 and int(st["code"]) == 0 and int(want.sum()) > 0
    counts = gpu_counts(streams, R, P)
    got = counts.cpu().numpy().view(np.uint64)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)[0]
        raise AssertionError(f"counts differ at {tuple(bad)}: gpu {got[tuple(bad)]} oracle {want[tuple(bad)]}")
    check_attribution(counts, want, rng.normal(size=P) * 1e3)


def test_attribution_shapes_and_extremes():
    """Column totals of zero, single owners, counts near 2^63, one row, more PCs than one block and a ragged tail."""
    rng = np.random.default_rng(12)
    for rows, P in [(1, 5), (203, 1000), (7, 257), (64, 70_560)]:
        counts = rng.integers(0, 1000, size=(rows, P)).astype(np.uint64)
        counts[:, rng.integers(0, P, size=max(1, P // 10))] = 0
        counts[0, 0] = np.uint64(2**62)
        metric = rng.normal(size=P) * 10.0 ** rng.integers(-3, 6, size=P)
        dev = torch.from_numpy(counts.view(np.int64)).to(DEV)
        check_attribution(dev, counts, metric)


def test_pc_index_out_of_range_is_reported():
    ev = np.array([(0, 0, 0), (2, 9, 1), (1, 0, 0)], dtype=oracle.MAP_EVENT)
    enc = encode_map_events(ev["kind"], ev["id"], ev["count"], 1)[0]
    d_ev = torch.from_numpy(enc.view(np.uint8).reshape(-1).copy()).to(DEV)
    d_off = torch.from_numpy(np.array([0, len(enc)], np.int64)).to(DEV)
    pr = argus.argus_pair_intervals(d_ev, d_off, 2)
    counts, status = argus.argus_map_pc_counts(pr.intervals, pr.interval_offsets, 1, 4)
    assert int(argus.argus_status_fetch(status)["code"]) == 1


def test_decode_shaped_mapping_run():
    """The synthetic mapping run used for measurements (decode-megakernel markers with exec records after every
    begin, 203 region ids, 70,560 PCs, eight helper PCs shared by all regions): counts bit for bit, attribution
    to rounding, and shared PCs do come out ambiguous."""
    from paper_2609_12299_b200 import tracegen as tg
    from paper_2609_12299_b200.tracegen.mapping import decode_mapping_trace, mapping_trace
    spec = tg.config(3).scaled(num_ctas=2, iters=6)
    R, P = spec.num_regions, 70_560
    d_ev, d_off = tg.generate_cuda(spec, DEV)
    m_ev, m_off = mapping_trace(d_ev, d_off, R, P, execs_per_begin=2)
    pr = argus.argus_pair_intervals(m_ev, m_off, R + 1)
    assert int(pr.fetch_status()["code"]) == 0
    counts, status = argus.argus_map_pc_counts(pr.intervals, pr.interval_offsets, R, P)
    assert int(argus.argus_status_fetch(status)["code"]) == 0
    host = m_ev.cpu().numpy().view(argus.EVENT_DTYPE)
    offs = m_off.cpu().numpy().astype(np.int64)
    kind, ident, count, removed_before = decode_mapping_trace(host, R)
    a_offs = (offs - np.concatenate([[0], removed_before])[offs]).astype(np.uint64)
    abstract = np.zeros(len(kind), dtype=oracle.MAP_EVENT)
    abstract["kind"], abstract["id"], abstract["count"] = kind, ident, count
    rc, want, st = oracle.map_pc_counts(abstract, a_offs, R, P)
    assert rc == 0 and int(st["code"]) == 0
    assert np.array_equal(counts.cpu().numpy().view(np.uint64), want)
    metric = np.random.default_rng(2).gamma(2.0, 50.0, size=P)
    check_attribution(counts, want, metric)
    _, _, ent, _ = oracle.attribute(want, metric)
    assert np.all(ent[-8:] > 0.1) and np.count_nonzero(ent[:-8]) == 0
