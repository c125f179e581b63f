"""Pins of the oracle's PC-to-region mapping and attribution: a hand-worked example, a stack walk
redone in Python on small random traces, the pairing oracle on the marker encoding of the same trace
(the two must agree, defects included), and closed forms / invariants of alpha, the lifted metric
and the association entropy."""
import math
import os

import numpy as np
import pytest

import oracle
from helpers import GOLDEN


def load_map_example():
    ev, counts, metric, mhat, ent = [], {}, None, {}, {}
    with open(os.path.join(GOLDEN, "example_j_pc_map.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] == "begin":
                ev.append((0, int(tok[1]), 0))
            elif tok[0] == "end":
                ev.append((1, int(tok[1]), 0))
            elif tok[0] == "exec":
                ev.append((2, int(tok[1]), int(tok[2])))
            elif tok[0] == "counts":
                counts[int(tok[1])] = [int(x) for x in tok[2:]]
            elif tok[0] == "metric":
                metric = [float(x) for x in tok[1:]]
            elif tok[0] == "mhat":
                mhat[int(tok[1])] = float(tok[2])
            elif tok[0] == "entropy":
                ent[int(tok[1])] = float(tok[2])
    events = np.array(ev, dtype=oracle.MAP_EVENT)
    want = np.array([counts[r] for r in sorted(counts)], dtype=np.uint64)
    return events, want, np.array(metric), np.array([mhat[r] for r in sorted(mhat)]), np.array([ent[p] for p in sorted(ent)])


def random_map_trace(rng, n, R, P, p_bad=0.0, max_depth=6):
    """Random mapping-run stream: begins, ends (mostly of the top frame, sometimes of another or of no open
    region), exec records."""
    ev, stack = [], []
    for _ in range(n):
        u = rng.random()
        if u < 0.45:
            ev.append((2, int(rng.integers(0, P)), int(rng.integers(0, 9))))
        elif u < 0.75 and len(stack) < max_depth:
            r = int(rng.integers(0, R))
            stack.append(r)
            ev.append((0, r, 0))
        elif stack:
            if rng.random() < p_bad:
                r = int(rng.integers(0, R))          # possibly mis-nested or unmatched
                ev.append((1, r, 0))
                if r in stack:
                    k = len(stack) - 1 - stack[::-1].index(r)
                    del stack[k:]
            else:
                ev.append((1, stack.pop(), 0))
        elif rng.random() < p_bad:
            ev.append((1, int(rng.integers(0, R)), 0))  # end with nothing open
    return np.array(ev, dtype=oracle.MAP_EVENT)


def python_walk(ev, R, P):
    counts = np.zeros((R + 1, P), dtype=np.uint64)
    stack = []
    for kind, ident, k in ev.tolist():
        if kind == 2:
            counts[stack[-1] if stack else R, ident] += np.uint64(k)
        elif kind == 0:
            stack.append(ident)
        else:
            for j in range(len(stack) - 1, -1, -1):
                if stack[j] == ident:
                    del stack[j:]
                    break
    return counts


def encode_as_markers(ev, R):
    """The marker encoding the C-ABI documents: exec(pc, k) = begin/end of region R with ctx = pc, ts 0 and k."""
    out = []
    for kind, ident, k in ev.tolist():
        if kind == 2:
            out.append((0, R << 1, ident))
            out.append((k, (R << 1) | 1, ident))
        else:
            out.append((7, (ident << 1) | kind, 0))
    return np.array(out, dtype=oracle.EVENT)


def test_hand_worked_example():
    ev, want, metric, want_mhat, want_ent = load_map_example()
    rc, counts, st = oracle.map_pc_counts(ev, [0, len(ev)], 2, 3)
    assert rc == 0 and int(st["code"]) == 0
    assert np.array_equal(counts, want)
    rc, mhat, ent, alpha = oracle.attribute(counts, metric)
    assert rc == 0
    assert np.allclose(mhat, want_mhat, rtol=0, atol=1e-15)
    assert np.allclose(ent, want_ent, rtol=0, atol=1e-15)
    assert alpha[0, 0] == 0.75 and alpha[1, 0] == 0.25 and alpha[1, 1] == 1.0 and alpha[2, 2] == 1.0


@pytest.mark.parametrize("p_bad", [0.0, 0.3])
def test_random_traces_against_a_python_walk_and_the_pairing_oracle(p_bad):
    rng = np.random.default_rng(int(p_bad * 10) + 3)
    R, P = 5, 11
    streams = [random_map_trace(rng, int(rng.integers(0, 400)), R, P, p_bad) for _ in range(12)]
    offs = np.cumsum([0] + [len(s) for s in streams]).astype(np.uint64)
    ev = np.concatenate(streams)
    rc, counts, st = oracle.map_pc_counts(ev, offs, R, P)
    assert rc == 0 and int(st["code"]) == 0
    want = sum(python_walk(s, R, P) for s in streams)
    assert np.array_equal(counts, want)
    assert int(counts.sum()) == int(ev["count"][ev["kind"] == 2].sum())
    # the same trace as markers through the pairing oracle: exec intervals carry their owner as parent_region
    enc = [encode_as_markers(s, R) for s in streams]
    eoffs = np.cumsum([0] + [len(s) for s in enc]).astype(np.uint64)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(np.concatenate(enc), eoffs, R + 1)
    assert rc == 0 and int(st["code"]) == 0
    x = iv[iv["region"] == R]
    owner = np.where(x["parent_region"] < R, x["parent_region"], R)
    via_pairing = np.zeros((R + 1, P), dtype=np.uint64)
    np.add.at(via_pairing, (owner, x["ctx"]), x["inclusive"])
    assert np.array_equal(via_pairing, counts)


def test_attribution_closed_forms_and_invariants():
    rng = np.random.default_rng(8)
    rows, P = 7, 40
    counts = rng.integers(0, 50, size=(rows, P)).astype(np.uint64)
    counts[:, 0] = 0                      # a PC that never executed
    counts[:, 1] = 0; counts[3, 1] = 17   # a single owner
    counts[:, 2] = 0; counts[[0, 2, 5, 6], 2] = 9   # four equal owners
    counts[:, 3] = 2**40                  # all rows equal, large counts
    metric = rng.normal(size=P) * 100
    rc, mhat, ent, alpha = oracle.attribute(counts, metric)
    assert rc == 0
    assert ent[0] == 0 and not alpha[:, 0].any()
    assert ent[1] == 0 and alpha[3, 1] == 1.0
    assert ent[2] == pytest.approx(math.log(4), abs=1e-15) and np.all(alpha[[0, 2, 5, 6], 2] == 0.25)
    assert ent[3] == pytest.approx(math.log(rows), abs=1e-14)
    live = counts.sum(0) > 0
    assert np.allclose(alpha[:, live].sum(0), 1.0, rtol=0, atol=1e-15)
    assert np.all(ent >= 0) and np.all(ent <= math.log(rows) + 1e-14)
    # shared PCs contribute in proportion to their owners, so nothing is lost or invented
    assert mhat.sum() == pytest.approx(metric[live].sum(), rel=1e-13)
    # numpy restatement with library routines
    tot = counts.sum(0).astype(np.float64)
    a = np.divide(counts.astype(np.float64), tot, out=np.zeros((rows, P)), where=tot > 0)
    assert np.array_equal(alpha, a)
    assert np.allclose(mhat, a @ metric, rtol=1e-13, atol=1e-10)
    with np.errstate(divide="ignore", invalid="ignore"):
        h = -np.where(a > 0, a * np.log(a), 0.0).sum(0)
    assert np.allclose(ent, h, rtol=1e-13, atol=1e-15)
    # doubling every count changes nothing; a ratio metric lifts numerator and denominator separately
    rc, mhat2, ent2, alpha2 = oracle.attribute(counts * np.uint64(2), metric)
    assert np.array_equal(alpha2, alpha) and np.array_equal(mhat2, mhat) and np.array_equal(ent2, ent)


def test_depth_limit_and_bad_ids():
    deep = np.array([(0, 0, 0)] * 64 + [(2, 0, 1)], dtype=oracle.MAP_EVENT)
    rc, counts, st = oracle.map_pc_counts(deep, [0, len(deep)], 1, 1)
    assert rc == 0 and int(st["code"]) == 5          # an exec record needs a free stack slot, like a begin
    ok = np.array([(0, 0, 0)] * 63 + [(2, 0, 1)], dtype=oracle.MAP_EVENT)
    rc, counts, st = oracle.map_pc_counts(ok, [0, len(ok)], 1, 1)
    assert rc == 0 and int(st["code"]) == 0 and int(counts[0, 0]) == 1
    bad = np.array([(0, 3, 0)], dtype=oracle.MAP_EVENT)
    rc, counts, st = oracle.map_pc_counts(bad, [0, 1], 2, 1)
    assert int(st["code"]) == 6
    rc, counts, st = oracle.map_pc_counts(np.array([(2, 5, 1)], dtype=oracle.MAP_EVENT), [0, 1], 2, 3)
    assert rc == 1
