"""The multi-process plumbing of bench.py on CPU (gloo, world size 2): ranks are
independent replicas, the process group only carries the barrier and the
max-over-ranks of the measured time, and the reported value aggregates them."""
import os
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    r, w, local, dist = bench.dist_setup(world, backend="gloo")
    assert (r, w, local) == (rank, world, rank) and dist is not None
    bench.barrier_sync(dist, cuda=False)
    # each rank "measures" a different time; everyone must end up with the slowest
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    out[rank] = (ms, bench.whole_job_value(w, 2.0e12, ms))
    bench.barrier_sync(dist, cuda=False)
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 15.0
    assert value == pytest.approx(2 * 2.0e12 / 15e-3 / 1e12)


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert bench.dist_setup(1, backend="gloo") == (0, 1, 0, None)
    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
