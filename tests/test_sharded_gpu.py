"""Sharded workers on the GPU: R handles that each hold n_total / R workers, with the exchange of the
message buffers done by hand between them (all on one GPU, one after the other - no handle ever waits
for another), must reproduce the single handle that holds all n_total workers bit for bit: theta, the
moments, the averaged gradient, the messages and every worker's error accumulator. The single handle
is itself compared with the oracle in test_parity_gpu.py; one case here goes to the oracle directly."""
import numpy as np
import pytest
import torch

from paper_2205_05632_b200 import BLOCKSIGN, RANDK, TOPK, CompAMS, CompAMSError

pytestmark = pytest.mark.gpu

OFFS = [0, 10, 74, 1098, 5194, 5195, 13392, 13392 + 3 * 8192 + 1234, 13392 + 3 * 8192 + 1234 + 4097]


def _swap_rows(shards):
    """What an all-gather does: every shard's own rows go to every other shard."""
    bufs = [s.message_buffers() for s in shards]
    for a, sa in enumerate(shards):
        lo, hi = sa.first_worker, sa.first_worker + sa.n
        for b, sb in enumerate(shards):
            if a != b:
                for src, dst in zip(bufs[a], bufs[b]):
                    dst[lo:hi].copy_(src[lo:hi])


def _run(comp, ratio, offs, n_total, R, steps=5, seed=0):
    d = offs[-1]
    gen = torch.Generator(device="cuda").manual_seed(seed)
    whole = CompAMS(n_total, d, offs, comp, ratio, record_average=True)
    per = n_total // R
    shards = [CompAMS(per, d, offs, comp, ratio, n_total=n_total, first_worker=r * per, record_average=True)
              for r in range(R)]
    theta = 0.1 * torch.randn(d, generator=gen, device="cuda")
    thetas = [theta.clone() for _ in range(R)]
    for t in range(steps):
        G = torch.randn(n_total, d, generator=gen, device="cuda")
        whole.step(G, theta)
        for r, s in enumerate(shards):
            s.compress(G[r * per:(r + 1) * per].contiguous())
        _swap_rows(shards)
        for r, s in enumerate(shards):
            s.apply(thetas[r])
        for r, s in enumerate(shards):
            assert torch.equal(thetas[r], theta), "theta of shard %d differs at step %d" % (r, t)
            for name in ("m", "v", "vhat", "gbar"):
                assert torch.equal(s.buffer(name), whole.buffer(name)), (name, r, t)
            if comp == BLOCKSIGN:
                assert torch.equal(s.buffer("sign_bits"), whole.buffer("sign_bits"))
                assert torch.equal(s.buffer("scales"), whole.buffer("scales"))
            else:
                # inside a (worker, block) segment the order of the pairs is unspecified: compare as sets
                iw, order_w = torch.sort(whole.buffer("topk_idx"), dim=1, stable=True)
                is_, order_s = torch.sort(s.buffer("topk_idx"), dim=1, stable=True)
                # indices of different blocks never interleave (segments cover disjoint coordinate ranges)
                assert torch.equal(iw, is_), ("kept index sets", r, t)
                vw = torch.gather(whole.buffer("topk_val"), 1, order_w)
                vs = torch.gather(s.buffer("topk_val"), 1, order_s)
                assert torch.equal(vw.view(torch.int32), vs.view(torch.int32)), ("kept values", r, t)
        if t in (0, steps - 1):  # reading E finishes the deferred residual: do it on some steps only
            Ew = whole.buffer("E")
            for r, s in enumerate(shards):
                assert torch.equal(s.buffer("E"), Ew[r * per:(r + 1) * per]), ("E", r, t)
    for o in [whole] + shards:
        assert o.check_status() == 0
        o.close()


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.01), (TOPK, 0.2), (BLOCKSIGN, 1.0), (RANDK, 0.05)])
@pytest.mark.parametrize("n_total,R", [(4, 2), (6, 3), (4, 4)])
def test_shards_reproduce_the_whole_layerwise(comp, ratio, n_total, R):
    _run(comp, ratio, OFFS, n_total, R)


@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_shards_reproduce_the_whole_one_long_block(comp):
    d = 40 * 8192 + 77  # long candidate lists: the multi-CTA select
    _run(comp, 0.01, [0, d], 8, 2, steps=6, seed=3)


def test_shards_reproduce_the_whole_randk_long_rows():
    # long rows; a shard delivers nothing itself, the exchanged messages are scattered by compams_apply
    d = (1 << 21) + 777
    _run(RANDK, 0.01, [0, 300000, 300007, d], 4, 2, steps=3, seed=4)


def test_sharded_run_matches_the_oracle():
    import oracle
    n_total, R, d = 4, 2, OFFS[-1]
    per = n_total // R
    gen = torch.Generator(device="cuda").manual_seed(5)
    for comp, ratio in ((TOPK, 0.05), (BLOCKSIGN, 1.0)):
        ref = oracle.Oracle(n_total, d, OFFS, comp, ratio)
        shards = [CompAMS(per, d, OFFS, comp, ratio, n_total=n_total, first_worker=r * per) for r in range(R)]
        theta = 0.1 * torch.randn(d, generator=gen, device="cuda")
        thetas = [theta.clone() for _ in range(R)]
        theta_ref = theta.cpu().numpy().copy()
        for t in range(4):
            G = torch.randn(n_total, d, generator=gen, device="cuda")
            ref.step(G.cpu().numpy(), theta_ref)
            for r, s in enumerate(shards):
                s.compress(G[r * per:(r + 1) * per].contiguous())
            _swap_rows(shards)
            for r, s in enumerate(shards):
                s.apply(thetas[r])
            for r, s in enumerate(shards):
                for name, got in (("theta", thetas[r]), ("m", s.buffer("m")), ("vhat", s.buffer("vhat"))):
                    want = theta_ref if name == "theta" else ref.buffer(name)
                    err = np.abs(got.cpu().numpy() - want)
                    assert np.all(err <= 1e-7 + 1e-6 * np.abs(want)), (name, r, t)
                want_e = ref.buffer("E")[r * per:(r + 1) * per]
                err = np.abs(s.buffer("E").cpu().numpy() - want_e)
                assert np.all(err <= 1e-7 + 1e-6 * np.abs(want_e)), ("E", r, t)
        for s in shards:
            assert s.check_status() == 0
            s.close()
        ref.close()


def test_a_sharded_handle_refuses_what_needs_the_exchange():
    d = 5000
    s = CompAMS(2, d, [0, d], TOPK, 0.01, n_total=4, first_worker=2)
    G = torch.zeros(2, d, device="cuda")
    theta = torch.zeros(d, device="cuda")
    with pytest.raises(CompAMSError):
        s.step(G, theta)  # the other workers' messages are missing
    s.close()
    with pytest.raises(CompAMSError):
        CompAMS(2, d, [0, d], TOPK, 1.0, n_total=4, first_worker=0)  # k = d has no message to exchange
    with pytest.raises(CompAMSError):
        CompAMS(2, d, [0, d], BLOCKSIGN, 1.0, n_total=3, first_worker=2)  # rows 2, 3 of 3
