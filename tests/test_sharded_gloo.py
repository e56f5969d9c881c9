"""Sharded workers, host side: how worker rows are dealt to ranks and the exchange that completes the
message buffers, run as two CPU processes over gloo (the kernels themselves need a GPU and are
compared, shard against whole, in test_sharded_gpu.py)."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2205_05632_b200 import sharded


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_rows_are_dealt_evenly_in_rank_order():
    assert sharded.shard_rows(16, 4, 0) == (0, 4)
    assert sharded.shard_rows(16, 4, 3) == (12, 4)
    assert sharded.shard_rows(2, 2, 1) == (1, 1)
    assert sharded.shard_rows(5, 1, 0) == (0, 5)
    covered = sorted(r for k in range(8) for r in range(*(lambda f, n: (f, f + n))(*sharded.shard_rows(32, 8, k))))
    assert covered == list(range(32))
    for bad in ((6, 4, 0), (3, 4, 0), (8, 4, 4), (8, 0, 0)):
        with pytest.raises(ValueError):
            sharded.shard_rows(*bad)


def test_exchange_without_a_group_leaves_the_buffers_alone():
    buf = torch.arange(12, dtype=torch.int32).view(4, 3)
    keep = buf.clone()
    sharded.exchange([buf], 0, 4)
    assert torch.equal(buf, keep)


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_total, per = 6, 3
    first, rows = sharded.shard_rows(n_total, world, rank)
    # two message buffers of different width and type, as for Top-k (int32 indices, float32 values);
    # rows of other ranks start as garbage
    idx = torch.full((n_total, 5), -7, dtype=torch.int32)
    val = torch.full((n_total, 5), float("nan"), dtype=torch.float32)
    for r in range(first, first + rows):
        idx[r] = torch.arange(5, dtype=torch.int32) + 100 * r
        val[r] = torch.arange(5, dtype=torch.float32) * 0.5 - r
    sharded.exchange([idx, val], first, rows)
    out[rank] = (idx.tolist(), val.tolist())
    with pytest.raises(ValueError):
        sharded.exchange([torch.zeros(5, 2)], first, rows)  # 5 rows cannot come from 2 ranks of 3
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_complete_each_others_rows():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    idx, val = res[0]
    for r in range(6):
        assert idx[r] == [100 * r + k for k in range(5)]
        assert val[r] == [0.5 * k - r for k in range(5)]
