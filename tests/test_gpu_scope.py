"""Parity of scope selection (argus_aggregate_scoped, argus_overlap_scoped) against the CPU oracle,
bit for bit, through the C-ABI. Everything here needs a GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12299_b200 as argus
from paper_2609_12299_b200 import tracegen as tg
from test_oracle_scope_pins import load_scope_example

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ALL32 = 0xFFFFFFFF


def _dev_bytes(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).to(DEV)


def _dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32).copy()).to(DEV)


def _dev_u64(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint64).view(np.int64).copy()).to(DEV)


def _gpu_scope(scope, num_sms, num_regions):
    if scope is None:
        return None
    lo, hi = scope.get("ctx", (0, ALL32))
    warps = scope.get("warps")
    return argus.ArgusScope(
        ctx_lo=int(lo), ctx_hi=int(hi),
        warp_mask=0xFFFFFFFFFFFFFFFF if warps is None else sum(1 << int(w) for w in set(warps)),
        sm_mask=None if scope.get("sms") is None else argus.ArgusScope.bitmask(scope["sms"], num_sms, DEV),
        region_mask=None if scope.get("regions") is None else argus.ArgusScope.bitmask(scope["regions"], num_regions, DEV))


def _check(iv, ioffs, am, aoffs, W, cta_sm, M, R, pairs, scope, want_iter):
    levels = ("warp", "cta", "sm", "kernel", "role") + (("iter",) if want_iter else ())
    rc, want, st = oracle.aggregate_scoped(iv, ioffs, am, aoffs, W, cta_sm, M, R, scope=scope, levels=levels)
    assert rc == 0 and int(st["code"]) == 0
    d_iv, d_ioffs = _dev_bytes(iv), _dev_u64(ioffs)
    d_am = None if am is None else _dev_bytes(am)
    d_aoffs = None if aoffs is None else _dev_u64(aoffs)
    d_cta_sm = _dev_i32(cta_sm)
    gs = _gpu_scope(scope, M, R)
    res = argus.argus_aggregate_scoped(d_iv, d_ioffs, d_am, d_aoffs, W, d_cta_sm, M, R, gs, levels=levels)
    assert int(argus.argus_status_fetch(res.status)["code"]) == 0
    for lv in levels:
        got = res.table_numpy(lv)
        assert got.shape == want[lv].shape, lv
        if got.tobytes() != want[lv].tobytes():
            bad = np.argwhere(got != want[lv])[0]
            raise AssertionError(f"{lv} table differs at {tuple(bad)}: gpu {got[tuple(bad)]} oracle {want[lv][tuple(bad)]}")
    if pairs is not None:
        rc, o_ov, _ = oracle.overlap_scoped(iv, ioffs, W, cta_sm, M, pairs, scope=scope, num_regions=R)
        assert rc == 0
        out, status = argus.argus_overlap_scoped(d_iv, len(iv), d_ioffs, W, d_cta_sm, M, _dev_i32(pairs), gs)
        assert int(argus.argus_status_fetch(status)["code"]) == 0
        g_ov = out.cpu().numpy().view(argus.OVERLAP_DTYPE).reshape(len(pairs), M)
        assert g_ov.tobytes() == o_ov.tobytes(), f"overlap differs: gpu {g_ov} oracle {o_ov}"
    return want


def test_hand_worked_scopes_on_gpu():
    iv, ioffs, scopes, _, _ = load_scope_example()
    cta_sm = np.array([0, 1], dtype=np.uint32)
    for name, sc in scopes.items():
        want_iter = sc["ctx"][1] - sc["ctx"][0] < 16
        _check(iv, ioffs, None, None, 2, cta_sm, 2, 3, np.array([[0, 1]], np.uint32), sc, want_iter)


@pytest.fixture(scope="module")
def malformed_gemm():
    """GEMM-shaped trace with defects (ambiguity records, flags), 12 warps per CTA, one CTA per SM."""
    spec = tg.config(4).scaled(num_ctas=6, iters=60)
    ev, offs = tg.generate_host(spec)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions)
    assert rc == 0 and int(st["code"]) == 0 and len(am) > 0
    return spec, iv, ioffs, am, aoffs


SCOPES = [
    None,
    {},
    {"ctx": (10, 25)},
    {"warps": [0, 1]},
    {"warps": [2, 5, 11], "ctx": (0, 40)},
    {"sms": [1, 4]},
    {"regions": [1, 2]},
    {"ctx": (7, 7), "warps": [0], "sms": [0, 2, 3], "regions": [0, 1, 4]},
    {"ctx": (1000000, 2000000)},          # selects nothing
    {"warps": []},                        # selects nothing
]


@pytest.mark.parametrize("scope", SCOPES, ids=[str(i) for i in range(len(SCOPES))])
def test_scoped_aggregate_and_overlap_match_the_oracle(malformed_gemm, scope):
    spec, iv, ioffs, am, aoffs = malformed_gemm
    want_iter = scope is not None and "ctx" in scope and scope["ctx"][1] - scope["ctx"][0] < 64
    want = _check(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.num_regions,
                  spec.overlap_pairs, scope, want_iter)
    if scope in (None, {}):
        assert int(want["kernel"]["count"].sum()) == len(iv)


def test_iteration_table_too_large_for_shared_memory(malformed_gemm):
    """A window of 400 iterations x 5 regions x 576 B does not fit a block's shared memory: the global-atomics path."""
    spec, iv, ioffs, am, aoffs = malformed_gemm
    _check(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.num_regions, None,
           {"ctx": (0, 399)}, True)


def test_decode_trace_sixteen_iterations():
    """202 regions, 16 warps per CTA: role table and a 16-iteration window (the per-iteration use of the paper's
    worked example)."""
    spec = tg.config(3).scaled(num_ctas=4, iters=24)
    ev, offs = tg.generate_host(spec)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions)
    assert rc == 0
    _check(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.num_regions, spec.overlap_pairs,
           {"ctx": (4, 19), "warps": [0, 1, 2, 3, 8], "regions": list(range(0, 40))}, True)


def test_argument_errors():
    iv, ioffs, _, _, _ = load_scope_example()
    d_iv, d_ioffs = _dev_bytes(iv), _dev_u64(ioffs)
    cta_sm = _dev_i32(np.array([0, 1], np.uint32))
    with pytest.raises(argus.ArgusError):
        argus.argus_aggregate_scoped(d_iv, d_ioffs, None, None, 2, cta_sm, 2, 3, argus.ArgusScope(ctx_lo=5, ctx_hi=4))
    with pytest.raises(argus.ArgusError):  # iteration table without a scope
        argus.argus_aggregate_scoped(d_iv, d_ioffs, None, None, 2, cta_sm, 2, 3, None, levels=("kernel", "iter"))
    with pytest.raises(argus.ArgusError):
        argus.argus_overlap_scoped(d_iv, len(iv), d_ioffs, 2, cta_sm, 2, _dev_i32(np.array([[0, 1]])),
                                   argus.ArgusScope(ctx_lo=5, ctx_hi=4))
