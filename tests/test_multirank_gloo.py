"""The N > 1 plumbing of bench.py (one process per GPU, weak scaling, max-over-ranks timing) run as two
gloo ranks on CPU: per-rank traces differ but have the same shape, the reduced time is the slowest rank's,
and the whole-job rate counts every rank's events."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    import torch.distributed as dist
    from paper_2609_12299_b200 import tracegen as tg
    from paper_2609_12299_b200.multirank import max_over_ranks, rank_env, rank_spec, whole_job_rate
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert rank_env() == (rank, world, rank)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = rank_spec(tg.config(1).scaled(2, 10), rank)
    ev, offs = tg.generate_host(spec, nthreads=1)
    dist.barrier()
    ms = max_over_ranks(10.0 + 5.0 * rank, world)  # rank 1 is the slow one
    rate = whole_job_rate(len(ev), world, ms)
    out[rank] = (len(ev), int(offs[-1]), float(ev["ts"].astype(np.float64).sum()), ms, rate)
    dist.destroy_process_group()


def test_two_gloo_ranks_weak_scaling_plumbing():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] == r0[1] == r1[1]          # same shape on every rank
    assert r0[2] != r1[2]                            # but different traces (per-rank seed)
    assert r0[3] == r1[3] == 15.0                    # everyone sees the slowest rank's time
    assert r0[4] == r1[4] == r0[0] * 2 / 15e-3       # whole-job rate counts both ranks


def _combine_worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2609_12299_b200 import tracegen as tg
    from paper_2609_12299_b200.multirank import combine_kernel_tables, rank_spec
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = rank_spec(tg.config(4).scaled(2, 30), rank)
    ev, offs = tg.generate_host(spec, nthreads=1)
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions)
    _, tabs, _ = oracle.aggregate(iv, ioffs, am, aoffs, spec.warps_per_cta, spec.cta_sm, spec.num_sms, spec.num_regions,
                                  levels=("kernel",))
    mine = tabs["kernel"].copy()
    if rank == 1:
        mine["max_incl"][0, 0] = np.uint64(2**64 - 2)   # values above 2^63 must survive the signed collectives
        mine["sum_incl"][0, 1] = np.uint64(2**64 - 5)   # and sums wrap like unsigned ones
    t = torch.from_numpy(mine.view(np.uint8).reshape(-1).copy())
    combine_kernel_tables(t, world)
    out[rank] = (mine.tobytes(), t.numpy().tobytes())
    dist.destroy_process_group()


def test_kernel_scope_tables_are_combined_across_ranks():
    import oracle
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_combine_worker, args=(world, port, out), nprocs=world, join=True)
        (a, ca), (b, cb) = out[0], out[1]
    assert ca == cb                                   # every rank ends with the same table
    ta, tb, tc = (np.frombuffer(x, dtype=oracle.AGG).copy() for x in (a, b, ca))
    for f in ("count", "sum_incl", "sum_excl", "n_unmatched_begin", "n_unmatched_end", "n_flagged", "hist"):
        assert np.array_equal(tc[f], ta[f] + tb[f]), f     # uint64 arithmetic wraps, as the table's does
    assert np.array_equal(tc["min_incl"], np.minimum(ta["min_incl"], tb["min_incl"]))
    assert np.array_equal(tc["max_incl"], np.maximum(ta["max_incl"], tb["max_incl"]))
    assert int(tc["max_incl"][0]) == 2**64 - 2 and int(tc["count"].sum()) > 0


def test_single_process_defaults():
    from paper_2609_12299_b200.multirank import max_over_ranks, whole_job_rate
    assert max_over_ranks(3.5, 1) == 3.5
    assert whole_job_rate(1000, 1, 2.0) == 500000.0
