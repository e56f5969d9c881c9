"""Steps captured into a CUDA graph and replayed.

A step enqueues kernels only (programmatic dependents, one cooperative launch, no allocation, no host
synchronisation), so a caller whose loop is bound by launch latency - small models, many small optimizers - can
capture it. What a captured step bakes in are the handle's host-side switches of that moment (which of the two
Block-Sign scale buffers is current, whether E still holds the last step's x): they repeat with period two once
the first step is done, so an even number of steps captured after a warm-up step replays correctly any number of
times. The gradients are read from the captured buffers: the caller refills them before every replay."""
import pytest
import torch

from paper_2205_05632_b200 import BLOCKSIGN, RANDK, TOPK, CompAMS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.01), (BLOCKSIGN, 1.0), (TOPK, 1.0)])
def test_two_captured_steps_replay_like_eager_steps(comp, ratio):
    n, d = 4, 65536
    offs = [0, 3000, 40000, d]
    gen = torch.Generator(device="cuda").manual_seed(6)
    G = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(9)]
    eager = CompAMS(n, d, offs, comp, ratio, record_average=True)
    theta_eager = torch.zeros(d, device="cuda")
    for g in G:
        eager.step(g, theta_eager)
    torch.cuda.synchronize()

    side = torch.cuda.Stream()
    theta = torch.zeros(d, device="cuda")
    slots = [torch.empty(n, d, device="cuda") for _ in range(2)]
    with torch.cuda.stream(side):
        opt = CompAMS(n, d, offs, comp, ratio, stream=side, record_average=True)
        opt.step(G[0].clone(), theta)          # warm-up: from here on the host-side switches alternate
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        slots[0].copy_(G[1])
        slots[1].copy_(G[2])
        with torch.cuda.graph(graph, stream=side):
            opt.set_stream(torch.cuda.current_stream())
            opt.step(slots[0], theta)
            opt.step(slots[1], theta)
        # capturing enqueues nothing: the captured pair runs at every replay
        for r in range(4):
            slots[0].copy_(G[1 + 2 * r])
            slots[1].copy_(G[2 + 2 * r])
            graph.replay()
        side.synchronize()
    opt.set_stream(side)
    assert opt.check_status() == 0
    assert torch.equal(theta, theta_eager)
    for name in ("m", "v", "vhat", "gbar"):
        assert torch.equal(opt.buffer(name), eager.buffer(name)), name
    with torch.cuda.stream(side):
        assert torch.equal(opt.buffer("E"), eager.buffer("E"))
    side.synchronize()
    opt.close()
    eager.close()
