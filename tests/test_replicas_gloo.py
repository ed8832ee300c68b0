"""The multi-GPU mode is N independent replicas; its only cross-rank logic is the barrier and the
max-over-ranks job time.  Checked here on CPU with two gloo ranks."""
import os
import socket
import sys

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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
    dist.barrier()
    job = bench.job_time_ms(local_ms, dist, torch.device("cpu"))
    out[rank] = (job, bench.job_us_per_layer(job, steps=100, world=world))
    dist.barrier()
    dist.destroy_process_group()


def test_job_time_is_max_over_ranks_and_value_is_job_wide():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    job_ms, us = res[0]
    assert job_ms == 15.0                               # the slowest rank
    assert abs(us - 15.0 * 1e3 / (100 * 2)) < 1e-9      # 200 layers were processed job-wide in 15 ms


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.job_time_ms(3.5) == 3.5
    assert bench.job_us_per_layer(2.0, 10, 1) == 200.0
