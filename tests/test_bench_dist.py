"""The multi-rank leg of bench.py on CPU: two gloo ranks, replicas only (the path
has no exchange step): barrier, max-over-ranks timing, summed work."""
import os
import sys

import numpy as np
import torch
import torch.distributed as td
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    td.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = bench.Workload("small", seed_shift=rank)          # every rank draws its own replica of the same shape
    td.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, device="cpu")
    out[rank] = (ms, bench.job_value(world, w.total_flops, ms), w.total_flops, float(w.pool.q[0, 0, 0]),
                 w.pool.total_tokens > 0)
    td.destroy_process_group()


def test_two_rank_replica_timing_gloo():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] == 15.0                               # the slowest rank sets the time on every rank
    assert r0[3] != r1[3]                                       # different seeds per replica
    assert np.isclose(r0[1], world * r0[2] / 15e-3 / 1e12)      # whole-job value = all ranks' work / that time


def test_single_process_passthrough():
    import bench
    assert bench.max_over_ranks(3.5, device="cpu") == 3.5
    assert np.isclose(bench.job_value(4, 1e12, 1000.0), 4.0)
