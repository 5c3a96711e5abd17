"""The multi-process bookkeeping of bench.py (one replica per rank) with two gloo ranks on the CPU."""

import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2105_09837_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, w, lr = replicas.env_rank_world()
    assert (r, w, lr) == (rank, world, rank)
    assert replicas.device_for(lr, w) == rank
    dist.barrier()
    ms = [40.0, 55.0][rank]                      # rank 1 is slower
    mx = replicas.max_over_ranks(ms, dist)
    out[rank] = (mx, replicas.job_throughput(w, 10, mx))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_throughput():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        mx, val = out[rank]
        assert mx == 55.0
        assert abs(val - 2 * 10 / 0.055) < 1e-9


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_rank_world() == (0, 1, 0)
    assert replicas.device_for(3, 1) == 0
    assert replicas.max_over_ranks(12.5) == 12.5
    assert replicas.job_throughput(1, 20, 100.0) == 200.0
