"""Random trace shapes through the entry points beyond the one-call pipeline: both pairing kernels, scope
selection with a random scope, and pairing straight from a ring container, each against the CPU oracle bit
for bit. (The one-call pipeline runs the same shapes in tests/test_gpu_parity.py.) Needs a GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from paper_2609_12299_b200.binding import KERNEL_THREAD_PER_STREAM, KERNEL_TILED
from test_gpu_parity import _fuzz_case, assert_pair_matches
from test_gpu_scope import _check
from test_ring_buffer import make_ring

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", list(range(100, 112)) + [328])   # 328: a stream that opens a 65th frame
def test_random_shape_through_pairing_scopes_and_ring(seed):
    spec, ev, offs = _fuzz_case(seed)
    rng = np.random.default_rng(seed)
    R, W, M = spec.num_regions, spec.warps_per_cta, spec.num_sms
    rc, iv, ioffs, am, aoffs, o_st = oracle.pair(ev, offs, R)
    if int(o_st["code"]) != 0:   # the random corruption opened more than 64 frames: both kernels report it alike
        from test_gpu_parity import run_pair
        for kernel in (KERNEL_THREAD_PER_STREAM, KERNEL_TILED):
            _, st = run_pair(ev, offs, R, kernel)
            assert (int(st["code"]), int(st["bad_stream"]), int(st["bad_event"])) == \
                   (int(o_st["code"]), int(o_st["bad_stream"]), int(o_st["bad_event"]))
        return
    for kernel in (KERNEL_THREAD_PER_STREAM, KERNEL_TILED):
        assert_pair_matches(ev, offs, R, kernel)
    scope = {}
    if rng.random() < 0.6:
        lo = int(rng.integers(0, 16))
        scope["ctx"] = (lo, lo + int(rng.integers(0, 12)))
    if rng.random() < 0.5:
        scope["warps"] = [int(w) for w in rng.choice(W, size=int(rng.integers(0, W + 1)), replace=False)]
    if rng.random() < 0.5:
        scope["sms"] = [int(m) for m in rng.choice(M, size=int(rng.integers(0, M + 1)), replace=False)]
    if rng.random() < 0.5:
        scope["regions"] = [int(r) for r in rng.choice(R, size=int(rng.integers(0, min(R, 6) + 1)), replace=False)]
    pairs = spec.overlap_pairs if len(spec.overlap_pairs) else None
    _check(iv, ioffs, am, aoffs, W, spec.cta_sm, M, R, pairs, scope, "ctx" in scope)
    # the same streams written into ring slots of a random size: some wrap, some do not
    cap = int(rng.integers(1, 3000))
    streams = [ev[int(offs[s]):int(offs[s + 1])] for s in range(len(offs) - 1)]
    ring, written = make_ring(streams, cap)
    rc, want, roffs, dropped, st = oracle.ring_linearise(ring, cap, written)
    rc, riv, rioffs, ram, raoffs, r_st = oracle.pair(want, roffs, R)
    if int(r_st["code"]) == 0:
        d_ring = torch.from_numpy(ring.view(np.uint8).reshape(-1).copy()).to("cuda:0")
        d_written = torch.from_numpy(written.view(np.int64).copy()).to("cuda:0")
        pr, d_offs, d_dropped = argus.argus_pair_intervals_ring(d_ring, cap, d_written, R)
        assert int(pr.fetch_status()["code"]) == 0
        assert pr.intervals_numpy().tobytes() == riv.tobytes()
        assert pr.ambig_numpy().tobytes() == ram.tobytes()
        assert np.array_equal(d_dropped.cpu().numpy().view(np.uint64), dropped)
