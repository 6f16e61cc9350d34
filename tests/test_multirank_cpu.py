"""The N > 1 path of bench.py on CPU: two gloo ranks, replicas only (no data-path collective): the
job's time is the maximum over ranks and the reported value is the aggregate over all replicas."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each replica "measured" its own time; rank 1 is the slow one
    mine = [0.010 * (rank + 1), 0.020 * (rank + 1)]
    dist.barrier()
    sec, sec_e2e = bench.max_over_ranks(dist, torch, mine, "cpu")
    value = bench.whole_job_value(bench.step_bytes(), 100, world, sec)
    out[rank] = (sec, sec_e2e, value)
    dist.destroy_process_group()


def test_two_replicas_max_time_and_aggregate_value():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    sys.path.insert(0, ROOT)
    import bench
    for r in range(world):
        sec, sec_e2e, value = res[r]
        assert sec == pytest.approx(0.020) and sec_e2e == pytest.approx(0.040)      # the slowest rank's
        assert value == pytest.approx(bench.step_bytes() * 100 * 2 / 0.020 / 1e9)   # bytes of BOTH replicas


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(None, torch, [1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.whole_job_value(10e9, 3, 1, 2.0) == pytest.approx(15.0)
