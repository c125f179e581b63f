"""Shared test helpers: golden-file parsing, hand-built traces, and independent re-derivations
(brute force, closed forms) used to pin the oracle. Nothing here imports the CUDA binding."""
from __future__ import annotations

import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
EVENT = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4")])
NONE = 0xFFFFFFFF


def make_events(rows):
    """rows: iterable of (ts, 'B'|'E', region, ctx)."""
    ev = np.zeros(len(rows), dtype=EVENT)
    for i, (ts, kind, region, ctx) in enumerate(rows):
        ev[i] = (ts, (region << 1) | (1 if kind == "E" else 0), ctx)
    return ev


def load_example(name):
    """Parses tests/golden/<name>: returns (events, intervals[list of tuples], ambiguity[list of tuples])."""
    events, intervals, ambig = [], [], []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if tok[0] == "event":
                events.append((int(tok[1]), tok[2], int(tok[3]), int(tok[4])))
            elif tok[0] == "interval":
                v = [int(x) for x in tok[1:]]
                v[5] = NONE if v[5] < 0 else v[5]
                intervals.append(tuple(v))
            elif tok[0] == "ambiguity":
                ambig.append(tuple(int(x) for x in tok[1:]))
    return make_events(events), intervals, ambig


def interval_tuples(iv):
    return [(int(r["region"]), int(r["t_begin"]), int(r["inclusive"]), int(r["exclusive"]), int(r["depth"]),
             int(r["parent_region"]), int(r["begin_idx"]), int(r["ctx"]), int(r["flags"])) for r in iv]


def ambig_tuples(am):
    return [(int(r["event_idx"]), int(r["tag"]) >> 1, int(r["kind"]), int(r["depth"])) for r in am]


def single_stream(ev):
    return np.array([0, len(ev)], dtype=np.uint64)


def enumerate_matchings(ev):
    """Brute force: every set of (begin i, end j) pairs with i < j, equal region, each marker used at
    most once and no two pairs crossing. Returns a list of frozensets of pairs. Exponential; tiny inputs only."""
    n = len(ev)
    region = [int(t) >> 1 for t in ev["tag"]]
    is_end = [int(t) & 1 for t in ev["tag"]]
    cands = [(i, j) for i in range(n) for j in range(i + 1, n)
             if not is_end[i] and is_end[j] and region[i] == region[j]]
    out = []

    def crosses(a, b):
        (i, j), (k, l) = a, b
        return (i < k < j < l) or (k < i < l < j)

    def rec(start, chosen, used):
        out.append(frozenset(chosen))
        for c in range(start, len(cands)):
            p = cands[c]
            if p[0] in used or p[1] in used or any(crosses(p, q) for q in chosen):
                continue
            rec(c + 1, chosen + [p], used | {p[0], p[1]})

    rec(0, [], frozenset())
    return out


def random_wellformed(rng, n_pairs, num_regions, max_height=6, t0=1000, self_nest=True):
    """A random well-formed single-stream trace with n_pairs begin/end pairs."""
    rows, stack, t, remaining = [], [], t0, n_pairs
    ctx = 0
    while remaining > 0 or stack:
        t += int(rng.integers(0, 40))
        can_begin = remaining > 0 and len(stack) < max_height
        if can_begin and (not stack or rng.random() < 0.5):
            r = int(rng.integers(0, num_regions))
            if not self_nest:
                while r in stack:
                    r = int(rng.integers(0, num_regions))
            if not stack:
                ctx = int(rng.integers(0, 16))
            stack.append(r)
            rows.append((t, "B", r, ctx))
            remaining -= 1
        else:
            rows.append((t, "E", stack.pop(), ctx))
    return make_events(rows)


def closed_form_wellformed(ev):
    """Independent derivation for a WELL-FORMED single stream using only prefix sums:
    height = running sum of +1/-1; the k-th interval (in end order) has depth = height after its end;
    exclusive(I) = sum of gaps ts[k+1]-ts[k] over events k inside I whose post-event height is depth(I)+1.
    Returns list of (inclusive, exclusive, depth) in end order."""
    ts = ev["ts"].astype(object)
    is_end = (ev["tag"] & 1).astype(np.int64)
    h = np.cumsum(1 - 2 * is_end)  # height after each event
    n = len(ev)
    res = []
    for j in range(n):
        if not is_end[j]:
            continue
        d = int(h[j])
        # matching begin: last index i < j with post-height d+1 reached from d (first time since height <= d)
        i = j - 1
        while not (h[i] == d + 1 and (i == 0 or h[i - 1] == d) and not is_end[i]):
            i -= 1
        incl = ts[j] - ts[i]
        excl = sum(ts[k + 1] - ts[k] for k in range(i, j) if h[k] == d + 1)
        res.append((int(incl), int(excl), d))
    return res
