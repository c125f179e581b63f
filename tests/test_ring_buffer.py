"""Ring-buffer container: oracle pins on CPU (a hand-made example, numpy roll, and what a wrap does to
pairing: leading ends lose their begins), and parity of the CUDA path on a GPU."""
import numpy as np
import pytest

import oracle
from helpers import make_events, random_wellformed


def make_ring(streams, slot_capacity):
    """Writes every stream into its slot the way a tracer would: record i at position i % slot_capacity."""
    S = len(streams)
    ring = np.zeros(S * slot_capacity, dtype=oracle.EVENT)
    ring["ts"] = 0xDEAD                      # stale contents must never be read
    for s, ev in enumerate(streams):
        for i, e in enumerate(ev):
            ring[s * slot_capacity + i % slot_capacity] = e
    return ring, np.array([len(ev) for ev in streams], dtype=np.uint64)


def test_hand_made_ring():
    # slot of 4 records; stream 0 wrote 6 (records 2..5 survive, stored at positions 2 3 0 1), stream 1 wrote 3,
    # stream 2 nothing, stream 3 exactly 4
    ev = lambda base, n: make_events([(base + i, "B", i % 3, i) for i in range(n)])
    streams = [ev(100, 6), ev(200, 3), ev(300, 0), ev(400, 4)]
    ring, written = make_ring(streams, 4)
    rc, out, offs, dropped, st = oracle.ring_linearise(ring, 4, written)
    assert rc == 0 and int(st["code"]) == 0
    assert list(offs) == [0, 4, 7, 7, 11] and list(dropped) == [2, 0, 0, 0]
    assert list(out["ts"]) == [102, 103, 104, 105, 200, 201, 202, 400, 401, 402, 403]
    rc, out, offs, dropped, st = oracle.ring_linearise(ring, 4, written, event_capacity=10)
    assert int(st["code"]) == 4 and int(st["intervals_required"]) == 11


def _random_case(rng, S, slot_capacity):
    streams = [random_wellformed(rng, int(rng.integers(0, 3 * slot_capacity // 2)), 5, max_height=5) for _ in range(S)]
    return streams, make_ring(streams, slot_capacity)


def test_survivors_are_the_tail_of_what_was_written():
    rng = np.random.default_rng(6)
    cap = 64
    streams, (ring, written) = _random_case(rng, 9, cap)
    rc, out, offs, dropped, st = oracle.ring_linearise(ring, cap, written)
    assert rc == 0 and int(st["code"]) == 0 and dropped.sum() > 0
    for s, ev in enumerate(streams):
        tail = ev[max(0, len(ev) - cap):]
        assert out[int(offs[s]):int(offs[s + 1])].tobytes() == tail.tobytes()
        # numpy restatement: rotate the slot so that the oldest survivor comes first
        if len(ev) >= cap:
            slot = ring[s * cap:(s + 1) * cap]
            assert np.roll(slot, -(len(ev) % cap)).tobytes() == tail.tobytes()
    # a wrap cuts begins off: the survivors pair like the un-wrapped stream minus the intervals that lost their begin
    rc, iv, ioffs, am, aoffs, st = oracle.pair(out, offs, 5)
    assert rc == 0 and int(st["code"]) == 0
    wrapped = [s for s, ev in enumerate(streams) if len(ev) > cap]
    assert wrapped
    lost = 0
    for s in wrapped:
        ev = streams[s]
        cut = ev[:len(ev) - cap]
        open_at_cut = int((1 - 2 * (cut["tag"] & 1).astype(np.int64)).sum())   # frames whose begin was overwritten
        kinds = am[int(aoffs[s]):int(aoffs[s + 1])]["kind"]
        assert len(kinds) == open_at_cut and np.all(kinds == 1)   # exactly their ends come out unmatched
        lost += open_at_cut
    assert lost > 0


@pytest.mark.gpu
@pytest.mark.parametrize("S,cap", [(9, 64), (40, 1000), (3, 1), (0, 8)])
def test_gpu_ring_linearise_matches_the_oracle(S, cap):
    import torch
    import paper_2609_12299_b200 as argus
    rng = np.random.default_rng(S * 1000 + cap)
    streams, (ring, written) = _random_case(rng, S, cap)
    rc, want, offs, dropped, st = oracle.ring_linearise(ring, cap, written)
    d_ring = torch.from_numpy(ring.view(np.uint8).reshape(-1).copy()).to("cuda:0")
    d_written = torch.from_numpy(written.view(np.int64).copy()).to("cuda:0")
    ev, d_offs, d_dropped, status = argus.argus_ring_linearise(d_ring, cap, d_written)
    assert int(argus.argus_status_fetch(status)["code"]) == 0
    assert np.array_equal(d_offs.cpu().numpy().view(np.uint64), offs)
    assert np.array_equal(d_dropped.cpu().numpy().view(np.uint64), dropped)
    n = int(offs[-1])
    assert ev.cpu().numpy()[: n * 16].tobytes() == want.tobytes()
    if S:
        # straight into pairing: same intervals and ambiguity records as the oracle gets from its own copy
        pr = argus.argus_pair_intervals(ev[: max(n, 1) * 16] if n else ev[:0], d_offs, 5)
        rc, iv, ioffs, am, aoffs, o_st = oracle.pair(want, offs, 5)
        assert int(pr.fetch_status()["code"]) == 0
        assert pr.intervals_numpy().tobytes() == iv.tobytes() and pr.ambig_numpy().tobytes() == am.tobytes()
        # too small an output buffer is reported, not overrun
        ev2, _, _, status2 = argus.argus_ring_linearise(d_ring, cap, d_written, event_capacity=max(n - 1, 0))
        st2 = argus.argus_status_fetch(status2)
        assert (int(st2["code"]) == 4 and int(st2["intervals_required"]) == n) if n else int(st2["code"]) == 0


@pytest.mark.gpu
@pytest.mark.parametrize("S,cap", [(9, 64), (40, 1000), (3, 1), (0, 8), (6, 5000)])
def test_gpu_pairing_straight_from_the_ring(S, cap):
    """argus_pair_intervals_ring = linearise + pair, without the copy: tiles that straddle the slot's end are fetched
    in two pieces (slot sizes below, around and above the 640-record tile; streams that wrapped and streams that did not)."""
    import torch
    import paper_2609_12299_b200 as argus
    rng = np.random.default_rng(S * 77 + cap)
    streams, (ring, written) = _random_case(rng, S, cap)
    rc, want, offs, dropped, st = oracle.ring_linearise(ring, cap, written)
    rc, iv, ioffs, am, aoffs, o_st = oracle.pair(want, offs, 5)
    d_ring = torch.from_numpy(ring.view(np.uint8).reshape(-1).copy()).to("cuda:0")
    d_written = torch.from_numpy(written.view(np.int64).copy()).to("cuda:0")
    pr, d_offs, d_dropped = argus.argus_pair_intervals_ring(d_ring, cap, d_written, 5)
    assert int(pr.fetch_status()["code"]) == 0
    assert np.array_equal(d_offs.cpu().numpy().view(np.uint64), offs)
    assert np.array_equal(d_dropped.cpu().numpy().view(np.uint64), dropped)
    assert pr.intervals_numpy().tobytes() == iv.tobytes()
    assert pr.ambig_numpy().tobytes() == am.tobytes()
    assert np.array_equal(pr.interval_offsets.cpu().numpy().view(np.uint64), ioffs)
    assert np.array_equal(pr.ambig_offsets.cpu().numpy().view(np.uint64), aoffs)


@pytest.mark.gpu
@pytest.mark.parametrize("mode", [-1, 2, 3])
def test_gpu_synthesize_straight_from_the_ring(mode):
    """argus_synthesize_ring = linearise + argus_synthesize, in the modes that exist for a ring (digests, plain calls,
    pass over the records)."""
    import torch
    import paper_2609_12299_b200 as argus
    from paper_2609_12299_b200.binding import argus_set_synthesize_mode
    rng = np.random.default_rng(99)
    S, cap, R, W, M = 12, 3000, 5, 4, 3
    streams = [random_wellformed(rng, int(rng.integers(0, 2 * cap)), R, max_height=5) for _ in range(S)]
    ring, written = make_ring(streams, cap)
    cta_sm = np.array([0, 2, 1], np.uint32)
    pairs_np = np.array([(0, 1), (2, 2), (4, 3)], np.uint32)
    rc, want, offs, dropped, st = oracle.ring_linearise(ring, cap, written)
    rc, iv, ioffs, am, aoffs, o_st = oracle.pair(want, offs, R)
    _, o_tabs, _ = oracle.aggregate(iv, ioffs, am, aoffs, W, cta_sm, M, R)
    _, o_ov, _ = oracle.overlap(iv, ioffs, W, cta_sm, M, pairs_np)
    d_ring = torch.from_numpy(ring.view(np.uint8).reshape(-1).copy()).to("cuda:0")
    d_written = torch.from_numpy(written.view(np.int64).copy()).to("cuda:0")
    d_cta_sm = torch.from_numpy(cta_sm.view(np.int32)).to("cuda:0")
    d_pairs = torch.from_numpy(pairs_np.view(np.int32)).to("cuda:0")
    argus_set_synthesize_mode(mode)
    try:
        res, d_offs, d_dropped = argus.argus_synthesize_ring(d_ring, cap, d_written, R, W, d_cta_sm, M, d_pairs)
        assert int(res.fetch_status()["code"]) == 0
    finally:
        argus_set_synthesize_mode(-1)
    assert np.array_equal(d_offs.cpu().numpy().view(np.uint64), offs)
    assert np.array_equal(d_dropped.cpu().numpy().view(np.uint64), dropped)
    assert res.pair.intervals_numpy().tobytes() == iv.tobytes()
    assert res.pair.ambig_numpy().tobytes() == am.tobytes()
    for lv in ("warp", "cta", "sm", "kernel"):
        assert res.agg.table_numpy(lv).tobytes() == o_tabs[lv].tobytes(), lv
    assert res.overlap_numpy(M).tobytes() == o_ov.tobytes()
