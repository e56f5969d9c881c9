"""N > 1 is replicas only: two CPU processes over gloo exercise the shared clock logic."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2205_05632_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist = replicas.init("gloo")
    assert dist is not None and dist.get_world_size() == world
    replicas.barrier(dist)
    mine = 2.0 + rank  # rank 1 is the slow replica
    slowest = replicas.max_over_ranks(mine, dist)
    out[rank] = (slowest, replicas.aggregate_throughput(1000.0, world, slowest))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_clock_and_the_summed_work():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slowest, value = res[0]
    assert slowest == 3.0
    assert abs(value - 2 * 1000.0 / 3e-3) < 1e-6


def test_single_process_needs_no_group(monkeypatch):
    monkeypatch.setenv("WORLD_SIZE", "1")
    assert replicas.init("gloo") is None
    assert replicas.max_over_ranks(1.5, None) == 1.5
    assert replicas.rank_world_local()[1] == 1
