"""Parity of the cross-run join (argus_join_samples) against the CPU oracle, bit for bit. Needs a GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from test_oracle_join_pins import load_join_example, random_runs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).to(DEV)


@pytest.fixture(params=["per-query", "hashed"])
def join_fn(request):
    """The block-per-query join and the one-pass hash join: same results."""
    return argus.argus_join_samples if request.param == "per-query" else argus.argus_join_samples_hashed


def _join(ref, idx, smp, fn=None):
    d_idx = torch.from_numpy(np.ascontiguousarray(idx, dtype=np.uint64).view(np.int64).copy()).to(DEV)
    out, status = (fn or argus.argus_join_samples)(_dev(ref), d_idx, _dev(smp))
    st = argus.argus_status_fetch(status)
    return out.cpu().numpy()[: len(idx) * 64].view(argus.JOIN_DTYPE), st


def test_hand_worked_join_on_gpu(join_fn):
    ref, smp, _ = load_join_example()
    idx = np.arange(len(ref), dtype=np.uint64)
    rc, want, _ = oracle.join_samples(ref, idx, smp)
    got, st = _join(ref, idx, smp, join_fn)
    assert int(st["code"]) == 0 and got.tobytes() == want.tobytes()


@pytest.mark.parametrize("n_ref,n_smp,big", [(60, 5000, False), (300, 200_000, True), (2000, 3000, False)])
def test_random_joins(n_ref, n_smp, big, join_fn):
    rng = np.random.default_rng(n_smp)
    ref, smp = random_runs(rng, n_ref, n_smp, streams=7, regions=6, ctxs=9, big=big)
    idx = rng.integers(0, n_ref, size=min(n_ref, 700)).astype(np.uint64)   # repeated queries are fine
    rc, want, o_st = oracle.join_samples(ref, idx, smp)
    assert rc == 0
    got, st = _join(ref, idx, smp, join_fn)
    assert int(st["code"]) == int(o_st["code"])
    if int(o_st["code"]) == 0:
        assert got.tobytes() == want.tobytes()
    else:  # a query with more samples than are ranked: count and sum stay exact
        assert np.array_equal(got["count"], want["count"]) and np.array_equal(got["sum"], want["sum"])


def test_join_on_paired_runs(join_fn):
    """Reference run and three probe runs of a persistent-GEMM-shaped kernel, all through the CUDA pairing: the
    selected operations (region tma_load of the producer warp, iterations 5 to 20) pick up one sample per run."""
    from paper_2609_12299_b200 import tracegen as tg
    from dataclasses import replace
    spec = tg.config(1).scaled(2, 40)
    runs = []
    for k in range(4):
        d_ev, d_off = tg.generate_cuda(replace(spec, seed=spec.seed + 17 * k), DEV)
        pr = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions)
        assert int(pr.fetch_status()["code"]) == 0
        runs.append(pr.intervals_numpy())
    ref, smp = runs[0], np.concatenate(runs[1:])
    sel = np.nonzero((ref["region"] == 1) & (ref["ctx"] >= 5) & (ref["ctx"] <= 20) & (ref["stream"] % spec.warps_per_cta == 0))[0]
    assert len(sel) == 2 * 16 * 8          # two CTAs, sixteen iterations, eight loads per iteration
    rc, want, o_st = oracle.join_samples(ref, sel.astype(np.uint64), smp)
    got, st = _join(ref, sel, smp, join_fn)
    assert int(st["code"]) == 0 and got.tobytes() == want.tobytes()
    assert np.all(got["count"] == 3 * 8)   # the eight loads of an iteration share their key: 8 samples per run


def test_grouped_join_on_paired_runs():
    """The same selection through argus_join_samples_grouped: the three probe runs' interval arrays one after the other
    with their per-stream offsets, so that a query reads only its stream's intervals of every run."""
    from paper_2609_12299_b200 import tracegen as tg
    from dataclasses import replace
    spec = tg.config(1).scaled(2, 40)
    S = spec.num_streams
    runs, offsets = [], []
    for k in range(4):
        d_ev, d_off = tg.generate_cuda(replace(spec, seed=spec.seed + 17 * k), DEV)
        pr = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions)
        assert int(pr.fetch_status()["code"]) == 0
        runs.append(pr.intervals_numpy())
        offsets.append(pr.interval_offsets.cpu().numpy().view(np.uint64).copy())
    ref, smp = runs[0], np.concatenate(runs[1:])
    base = np.cumsum([0] + [len(r) for r in runs[1:-1]]).astype(np.uint64)
    grouped = np.stack([offsets[1 + r] + base[r] for r in range(3)])            # [3, S + 1], indices into smp
    sel = np.nonzero((ref["region"] == 1) & (ref["ctx"] >= 5) & (ref["ctx"] <= 20))[0].astype(np.uint64)
    rc, want, o_st = oracle.join_samples(ref, sel, smp)
    d_idx = torch.from_numpy(sel.view(np.int64).copy()).to(DEV)
    d_grp = torch.from_numpy(grouped.view(np.int64).copy()).to(DEV)
    out, status = argus.argus_join_samples_grouped(_dev(ref), d_idx, _dev(smp), d_grp, S)
    assert int(argus.argus_status_fetch(status)["code"]) == 0
    assert out.cpu().numpy()[: len(sel) * 64].view(argus.JOIN_DTYPE).tobytes() == want.tobytes()
    # offsets that leave the sample array are reported
    bad = grouped.copy()
    bad[2, S] = len(smp) + 5
    out, status = argus.argus_join_samples_grouped(_dev(ref), d_idx, _dev(smp), torch.from_numpy(bad.view(np.int64).copy()).to(DEV), S)
    st = argus.argus_status_fetch(status)
    assert int(st["code"]) in (0, 7)   # 7 only if a query's stream is the last one
    sel_last = np.nonzero(ref["stream"] == S - 1)[0][:4].astype(np.uint64)
    out, status = argus.argus_join_samples_grouped(_dev(ref), torch.from_numpy(sel_last.view(np.int64).copy()).to(DEV), _dev(smp),
                                                   torch.from_numpy(bad.view(np.int64).copy()).to(DEV), S)
    assert int(argus.argus_status_fetch(status)["code"]) == 7


def test_join_edges_on_gpu(join_fn):
    ref, smp, _ = load_join_example()
    got, st = _join(ref, np.zeros(0, np.uint64), smp, join_fn)
    assert len(got) == 0 and int(st["code"]) == 0
    got, st = _join(ref, np.array([1, 99], np.uint64), smp, join_fn)
    assert int(st["code"]) == 1 and int(got[0]["count"]) == 1 and int(got[1]["count"]) == 0
    many = np.repeat(smp[:1], 5000)
    many["inclusive"] = np.arange(5000)
    got, st = _join(ref, np.array([0], np.uint64), many, join_fn)
    assert int(st["code"]) == 4 and int(got[0]["count"]) == 5000 and int(got[0]["sum"]) == 5000 * 4999 // 2


def test_hashed_join_of_many_queries_on_a_shuffled_run():
    """Two thousand queries against the intervals of a probe run in random order (no per-stream grouping to lean
    on), most samples belonging to no query: one pass over the samples, bit for bit the oracle's result."""
    from paper_2609_12299_b200 import tracegen as tg
    from dataclasses import replace
    spec = tg.config(3).scaled(2, 3)
    rng = np.random.default_rng(2609)
    runs = []
    for k in range(3):
        d_ev, d_off = tg.generate_cuda(replace(spec, seed=spec.seed + 5 * k), DEV)
        pr = argus.argus_pair_intervals(d_ev, d_off, spec.num_regions)
        assert int(pr.fetch_status()["code"]) == 0
        runs.append(pr.intervals_numpy())
    ref = runs[0]
    smp = np.concatenate(runs[1:])
    smp = smp[rng.permutation(len(smp))]
    sel = rng.choice(len(ref), size=2000, replace=False).astype(np.uint64)
    rc, want, o_st = oracle.join_samples(ref, sel, smp)
    assert rc == 0
    got, st = _join(ref, sel, smp, argus.argus_join_samples_hashed)
    assert int(st["code"]) == int(o_st["code"])
    if int(o_st["code"]) == 0:
        assert got.tobytes() == want.tobytes()
    else:
        assert np.array_equal(got["count"], want["count"]) and np.array_equal(got["sum"], want["sum"])
    assert int(got["count"].max()) > 2
