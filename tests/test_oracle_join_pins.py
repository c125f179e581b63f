"""Pins of the oracle's cross-run join: a hand-worked example, numpy sort-and-index on random data,
and the properties the definition implies (order and time independence, monotone percentiles)."""
import os

import numpy as np

import oracle
from helpers import GOLDEN


def load_join_example():
    ref, smp, want = [], [], {}
    with open(os.path.join(GOLDEN, "example_k_join.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] in ("ref", "smp"):
                (ref if tok[0] == "ref" else smp).append(tuple(int(x) for x in tok[1:]))
            elif tok[0] == "query":
                want[int(tok[1])] = tuple(int(x) for x in tok[2:])

    def build(rows):
        a = np.zeros(len(rows), dtype=oracle.INTERVAL)
        for i, (s, r, c, t0, incl) in enumerate(rows):
            a[i]["stream"], a[i]["region"], a[i]["ctx"], a[i]["t_begin"], a[i]["inclusive"] = s, r, c, t0, incl
        return a
    return build(ref), build(smp), want


def as_tuple(o):
    return (int(o["count"]), int(o["sum"])) + tuple(int(x) for x in o["pct"]) + (int(o["max"]),)


def random_runs(rng, n_ref, n_smp, streams=6, regions=5, ctxs=8, big=False):
    def make(n):
        a = np.zeros(n, dtype=oracle.INTERVAL)
        a["stream"] = rng.integers(0, streams, n)
        a["region"] = rng.integers(0, regions, n)
        a["ctx"] = rng.integers(0, ctxs, n)
        a["t_begin"] = rng.integers(0, 1 << 40, n)
        a["inclusive"] = rng.integers(0, 1 << 62, n) if big else rng.integers(0, 500, n)
        return a
    return make(n_ref), make(n_smp)


def test_hand_worked_join():
    ref, smp, want = load_join_example()
    rc, out, st = oracle.join_samples(ref, np.arange(len(ref)), smp)
    assert rc == 0 and int(st["code"]) == 0
    for q, w in want.items():
        assert as_tuple(out[q]) == w, (q, as_tuple(out[q]), w)


def test_join_redone_with_numpy_and_its_properties():
    rng = np.random.default_rng(4)
    for big in (False, True):
        ref, smp = random_runs(rng, 60, 5000, big=big)
        idx = rng.permutation(len(ref))[:40].astype(np.uint64)
        rc, out, st = oracle.join_samples(ref, idx, smp)
        assert rc == 0 and int(st["code"]) == 0
        for q, i in enumerate(idx):
            r = ref[int(i)]
            v = np.sort(smp["inclusive"][(smp["stream"] == r["stream"]) & (smp["region"] == r["region"]) & (smp["ctx"] == r["ctx"])])
            n = len(v)
            assert int(out[q]["count"]) == n and n > 0
            assert int(out[q]["sum"]) == int(v.sum(dtype=np.uint64))
            assert [int(x) for x in out[q]["pct"]] == [int(v[(j * n) // 5]) for j in range(5)]
            assert int(out[q]["max"]) == int(v[-1]) and int(out[q]["pct"][0]) == int(v[0])
            assert np.all(np.diff(out[q]["pct"].astype(object)) >= 0) and int(out[q]["pct"][4]) <= int(out[q]["max"])
        # order of the samples and their timestamps do not matter; the reference's timestamps do not either
        smp2 = smp[rng.permutation(len(smp))].copy()
        smp2["t_begin"] = rng.integers(0, 1 << 50, len(smp2))
        ref2 = ref.copy()
        ref2["t_begin"] += np.uint64(12345)
        ref2["inclusive"] = 0
        rc, out2, _ = oracle.join_samples(ref2, idx, smp2)
        assert out2.tobytes() == out.tobytes()
        # reference intervals with the same key share their samples
        twin = np.concatenate([ref, ref[:1]])
        rc, out3, _ = oracle.join_samples(twin, np.array([0, len(ref)], np.uint64), smp)
        assert out3[0].tobytes() == out3[1].tobytes()


def test_join_edges():
    ref, smp, _ = load_join_example()
    rc, out, st = oracle.join_samples(ref, np.zeros(0, np.uint64), smp)
    assert rc == 0 and len(out) == 0
    rc, out, st = oracle.join_samples(ref, np.array([0], np.uint64), smp[:0])
    assert rc == 0 and as_tuple(out[0]) == (0,) * 8
    rc, out, st = oracle.join_samples(ref, np.array([99], np.uint64), smp)
    assert rc == 1
    many = np.repeat(smp[:1], 5000)
    many["inclusive"] = np.arange(5000)
    rc, out, st = oracle.join_samples(ref, np.array([0], np.uint64), many)
    assert rc == 0 and int(st["code"]) == 4 and int(out[0]["count"]) == 5000 and int(out[0]["sum"]) == 5000 * 4999 // 2
