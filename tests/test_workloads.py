"""Input generators: tensor shapes of the synthetic workloads and reproducibility of the draws."""
import numpy as np
import torch

from paper_2205_05632_b200 import workloads as W


def test_resnet18_shape_table():
    shapes = W.resnet18_cifar_shapes()
    assert len(shapes) == 62
    offs = W.offsets_from_shapes(shapes)
    assert offs[0] == 0 and offs[-1] == 11_173_962
    assert shapes[0] == (64, 3, 3, 3) and shapes[-2:] == [(10, 512), (10,)]
    assert all(int(o) % 4 == 0 for o in offs[:-1])


def test_resnet50_shape_table():
    shapes = W.resnet50_imagenet_shapes()
    assert len(shapes) == 161
    offs = W.offsets_from_shapes(shapes)
    assert offs[-1] == 25_557_032
    sizes = np.diff(offs)
    assert (sizes == 64).sum() == 14 and (sizes == 2359296).sum() == 3 and (sizes == 2048000).sum() == 1


def test_fan_in_rule():
    assert W.fan_in((64, 3, 7, 7)) == 147
    assert W.fan_in((1000, 2048)) == 2048
    assert W.fan_in((512,)) == 512


def test_draws_are_reproducible_and_shaped():
    a, b = W.config1(), W.config1()
    ta, tb = a.start(), b.start()
    assert torch.equal(ta, tb) and ta.dtype == torch.float32 and ta.shape == (65536,)
    ga, gb = a.grads(), b.grads()
    assert torch.equal(ga, gb) and ga.shape == (4, 65536)
    assert not torch.equal(ga, a.grads())  # the next step draws fresh gradients
    assert abs(float(ta.std()) - 0.1) < 0.01


def test_config3_has_exact_zeros():
    w = W.config3(0.01)
    w.n = 1
    w.start()
    g = w.grads()
    frac = float((g == 0).float().mean())
    assert 0.045 < frac < 0.055


def test_windows_over_one_buffer_are_fresh_batches():
    """grads_with_tail: the head is the batch grads() would have drawn, every window is N(0,1) and two windows
    give a coordinate unrelated values; workloads with per-tensor scales or several blocks are refused."""
    a, b = W.config1(), W.config1()
    a.start(), b.start()
    assert W.iid_normal(a) and not W.iid_normal(W.config3(0.01)) and not W.iid_normal(W.config4(W.TOPK))
    extra = 64 * 5
    flat = W.grads_with_tail(a, extra)
    assert flat.shape == (4 * 65536 + extra,)
    assert torch.equal(flat[:4 * 65536].view(4, 65536), b.grads())
    w0 = flat[0:4 * 65536].view(4, 65536)
    w1 = flat[64:64 + 4 * 65536].view(4, 65536)
    assert abs(float(w1.mean())) < 0.01 and abs(float(w1.std()) - 1.0) < 0.01
    assert abs(float((w0 * w1).mean())) < 0.01  # no correlation between what a coordinate sees in two steps
