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


def test_single_process_defaults():
    from paper_2609_12299_b200.multirank import max_over_ranks, whole_job_rate
    assert max_over_ranks(3.5, 1) == 3.5
    assert whole_job_rate(1000, 1, 2.0) == 500000.0
