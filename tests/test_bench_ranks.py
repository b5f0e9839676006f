"""The rank plumbing of bench.py (barrier, max and sum over ranks) with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, lr, w = bench.dist_setup("gloo")
    assert (r, lr, w) == (rank, rank, world)
    bench.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)       # slowest replica sets the time
    samples = bench.sum_over_ranks(1000.0 * (rank + 1))  # every replica's samples count
    out[rank] = (ms, samples)
    bench.barrier()
    torch.distributed.destroy_process_group()


def test_two_ranks_agree_on_job_time_and_samples():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: (15.0, 3000.0), 1: (15.0, 3000.0)}


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5 and bench.sum_over_ranks(2.0) == 2.0
    bench.barrier()
