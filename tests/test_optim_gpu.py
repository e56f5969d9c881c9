"""COMP-AMS driving a torch model: real per-worker gradients (n micro-batches of a small residual
convolutional network on synthetic images) instead of synthetic ones. Checks that the wrapper feeds
the library what the oracle is fed (same theta after every step) and that training makes progress."""
import numpy as np
import pytest
import torch
import torch.nn as nn
import torch.nn.functional as F

from paper_2205_05632_b200 import BLOCKSIGN, TOPK
from paper_2205_05632_b200.optim import CompAMSOptimizer

pytestmark = pytest.mark.gpu


class Block(nn.Module):
    def __init__(self, cin, cout, stride):
        super().__init__()
        self.c1 = nn.Conv2d(cin, cout, 3, stride, 1, bias=False)
        self.b1 = nn.BatchNorm2d(cout)
        self.c2 = nn.Conv2d(cout, cout, 3, 1, 1, bias=False)
        self.b2 = nn.BatchNorm2d(cout)
        self.proj = None
        if stride != 1 or cin != cout:
            self.proj = nn.Sequential(nn.Conv2d(cin, cout, 1, stride, bias=False), nn.BatchNorm2d(cout))

    def forward(self, x):
        y = F.relu(self.b1(self.c1(x)))
        y = self.b2(self.c2(y))
        return F.relu(y + (x if self.proj is None else self.proj(x)))


class SmallResNet(nn.Module):
    """Two residual stages: the tensor mix of a ResNet (3x3 and 1x1 convolutions, BatchNorm pairs of 16
    and 32 elements, a linear head) at a size that trains in seconds."""

    def __init__(self, classes=10):
        super().__init__()
        self.stem = nn.Conv2d(3, 16, 3, 1, 1, bias=False)
        self.bn = nn.BatchNorm2d(16)
        self.s1 = Block(16, 16, 1)
        self.s2 = Block(16, 32, 2)
        self.fc = nn.Linear(32, classes)

    def forward(self, x):
        x = F.relu(self.bn(self.stem(x)))
        x = self.s2(self.s1(x))
        return self.fc(F.adaptive_avg_pool2d(x, 1).flatten(1))


def _data(n_workers, per, gen):
    x = torch.randn(n_workers, per, 3, 16, 16, generator=gen, device="cuda")
    y = torch.randint(0, 10, (n_workers, per), generator=gen, device="cuda")
    return x, y


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.05), (BLOCKSIGN, 1.0)])
def test_wrapper_feeds_the_library_what_the_oracle_gets(comp, ratio):
    import oracle
    torch.manual_seed(0)
    gen = torch.Generator(device="cuda").manual_seed(0)
    n = 4
    model = SmallResNet().cuda()
    opt = CompAMSOptimizer(model.parameters(), n, comp, ratio, lr=1e-2)
    ref = oracle.Oracle(n, opt.d, opt.offsets, comp, ratio, 1e-2, 0.9, 0.999, 1e-8)
    theta_ref = opt.theta.cpu().numpy().copy()
    x, y = _data(n, 8, gen)
    for t in range(4):
        for i in range(n):
            F.cross_entropy(model(x[i]), y[i]).backward()
            opt.collect(i)
        assert all(p.grad is None for p in model.parameters())
        ref.step(opt.G.cpu().numpy(), theta_ref)
        opt.step()
        got = opt.theta.cpu().numpy()
        assert np.all(np.abs(got - theta_ref) <= 1e-7 + 1e-6 * np.abs(theta_ref)), t
        # the model's tensors are views of theta: they moved with it
        first = next(model.parameters())
        assert first.data_ptr() == opt.theta.data_ptr()
        # the next forward pass must see the library's theta, not the oracle's rounding: keep them in step
        theta_ref[:] = got
    assert opt.opt.check_status() == 0
    opt.close()
    ref.close()


@pytest.mark.parametrize("comp,ratio,whole", [(TOPK, 0.01, False), (TOPK, 0.01, True), (BLOCKSIGN, 1.0, False)])
def test_training_makes_progress_on_a_fixed_synthetic_batch(comp, ratio, whole):
    torch.manual_seed(1)
    gen = torch.Generator(device="cuda").manual_seed(1)
    n = 4
    model = SmallResNet().cuda()
    opt = CompAMSOptimizer(model.parameters(), n, comp, ratio, whole_vector=whole, lr=1e-2 if comp == TOPK else 2e-3)
    x, y = _data(n, 16, gen)

    def mean_loss():
        model.eval()
        with torch.no_grad():
            out = float(sum(F.cross_entropy(model(x[i]), y[i]) for i in range(n)) / n)
        model.train()
        return out

    before = mean_loss()
    for t in range(80):
        for i in range(n):
            F.cross_entropy(model(x[i]), y[i]).backward()
            opt.collect(i)
        opt.step()
    after = mean_loss()
    assert opt.opt.check_status() == 0
    assert np.isfinite(after) and after < 0.9 * before, (before, after)
    opt.close()
