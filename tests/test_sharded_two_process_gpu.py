"""The sharded step end to end - compress, exchange, apply - as two processes that share one GPU.

Each process is one rank of a gloo group (two NCCL ranks cannot share a device) holding half of the workers;
ShardedCompAMS.step runs the worker side on the local rows, all-gathers the compressed gradients (staged
through host memory, as the group moves host memory only) and runs the server side on every rank. Each rank
compares its replica of theta and of the moments, and its own rows of the error accumulators, with the CPU
oracle run on all workers. No kernel of one rank waits for the other rank: the ranks meet in the host-side
collective only.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-7, 1e-6


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _close(gpu, cpu, what):
    ref = torch.from_numpy(np.ascontiguousarray(cpu)).to(gpu.device)
    bad = (gpu - ref).abs() > ATOL + RTOL * ref.abs()
    assert not bool(bad.any()), "%s differs from the oracle at %d elements" % (what, int(bad.sum()))


def _rank(rank, world, port, comp, ratio, steps):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist

    import oracle
    from paper_2205_05632_b200 import BLOCKSIGN, workloads as W
    from paper_2205_05632_b200.sharded import ShardedCompAMS

    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # ResNet-18 parameter tensors as blocks; every rank draws the gradients of all workers from the same seed
        # and keeps its own rows
        w = W.config2("cuda")
        n_local = 2
        w.n = n_total = world * n_local
        theta = w.start()
        opt = ShardedCompAMS(n_local, w.d, w.block_offsets, comp, ratio)
        opt.opt.record_average(True)
        ref = oracle.Oracle(n_total, w.d, w.block_offsets, comp, ratio)
        if comp == 2:
            opt.opt.set_seed(11)
            ref.set_seed(11)
        theta_ref = theta.cpu().numpy().copy()
        first = rank * n_local
        M = len(w.block_offsets) - 1
        for t in range(steps):
            G = w.grads()
            opt.step(G[first:first + n_local].contiguous(), theta)
            ref.step(G.cpu().numpy(), theta_ref)
            assert opt.opt.check_status() == 0
            _close(theta, theta_ref, "theta (rank %d, step %d)" % (rank, t))
            for name in ("m", "v", "vhat", "gbar"):
                _close(opt.opt.buffer(name), ref.buffer(name), "%s (rank %d, step %d)" % (name, rank, t))
            if t in (1, steps - 1):
                _close(opt.opt.buffer("E"), ref.buffer("E")[first:first + n_local], "E rows of rank %d, step %d" % (rank, t))
        if comp == BLOCKSIGN:
            Wd = int(opt.opt.buffer("sign_bits").shape[1])
            assert opt.total_message_bytes_per_step() == n_total * (4 * Wd + 4 * M)
            assert opt.message_bytes_per_step() == (n_total - n_local) * (4 * Wd + 4 * M)
        else:
            K = int(opt.opt.buffer("topk_idx").shape[1])
            assert K == sum(oracle.kept_per_block(ratio, int(s)) for s in np.diff(w.block_offsets))
            assert opt.total_message_bytes_per_step() == n_total * K * 8
            assert opt.message_bytes_per_step() == (n_total - n_local) * K * 8
        # the replicas are bit-identical: compare a digest of theta across the ranks
        digest = torch.tensor([float(theta.double().sum()), float(theta.double().abs().max())], dtype=torch.float64)
        both = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(both, digest)
        assert torch.equal(both[0], both[1])
        opt.close()
        ref.close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("comp,ratio", [(0, 0.01), (1, 1.0), (2, 0.01)])
def test_two_ranks_on_one_gpu_follow_the_oracle(comp, ratio):
    world = 2
    mp.spawn(_rank, args=(world, _free_port(), comp, ratio, 5), nprocs=world, join=True)
