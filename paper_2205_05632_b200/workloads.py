"""Seeded synthetic workloads: shapes, block partitions and gradient draws.

This module holds input generation only: none of the method's arithmetic (no error feedback,
no compression, no optimizer update) lives here, so both the CUDA library's callers and the
CPU oracle's callers can take their inputs from it. Every tensor is drawn once from a seeded
`torch.Generator` and handed, as the same bytes, to whichever side consumes it.

The paper trains on MNIST, CIFAR-10 and IMDB (Section 5.1); none of those datasets is used
here. The workloads keep only the parameter-tensor shapes of ResNet-18 (the paper's largest
model, Appendix A) and ResNet-50, each tensor being one compressor block (Section 3.1: blocks
are "usually the distinct network layers"), and draw heavy-tailed, sparse or biased values
that stand in for real gradients.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np
import torch

TOPK = 0
BLOCKSIGN = 1
RANDK = 2

Shape = Tuple[int, ...]


def _bn(c: int) -> List[Shape]:
    return [(c,), (c,)]


def resnet18_cifar_shapes(num_classes: int = 10) -> List[Shape]:
    """Parameter tensors of a ResNet-18 for 32x32 inputs (3x3 stem, no max-pool), definition order."""
    shapes: List[Shape] = [(64, 3, 3, 3)] + _bn(64)
    in_c = 64
    for stage, width in enumerate((64, 128, 256, 512)):
        for blk in range(2):
            shapes += [(width, in_c, 3, 3)] + _bn(width) + [(width, width, 3, 3)] + _bn(width)
            if blk == 0 and stage > 0:
                shapes += [(width, in_c, 1, 1)] + _bn(width)
            in_c = width
    shapes += [(num_classes, 512), (num_classes,)]
    return shapes


def resnet50_imagenet_shapes(num_classes: int = 1000) -> List[Shape]:
    """Parameter tensors of a ResNet-50 for 224x224 inputs, definition order."""
    shapes: List[Shape] = [(64, 3, 7, 7)] + _bn(64)
    in_c = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for blk in range(blocks):
            out_c = 4 * width
            shapes += [(width, in_c, 1, 1)] + _bn(width)
            shapes += [(width, width, 3, 3)] + _bn(width)
            shapes += [(out_c, width, 1, 1)] + _bn(out_c)
            if blk == 0:
                shapes += [(out_c, in_c, 1, 1)] + _bn(out_c)
            in_c = out_c
    shapes += [(num_classes, 2048), (num_classes,)]
    return shapes


def numel(shape: Shape) -> int:
    return int(math.prod(shape))


def fan_in(shape: Shape) -> int:
    """Product of all dims but the first; for 1-D tensors the number of elements."""
    return numel(shape[1:]) if len(shape) > 1 else numel(shape)


def offsets_from_shapes(shapes: Sequence[Shape]) -> np.ndarray:
    sizes = np.array([numel(s) for s in shapes], dtype=np.int64)
    return np.concatenate([np.zeros(1, dtype=np.int64), np.cumsum(sizes)])


def per_coordinate_scale(shapes: Sequence[Shape], device) -> torch.Tensor:
    """[d] fp32 vector holding fan_in^(-1/2) of the tensor each coordinate belongs to."""
    vals = torch.tensor([1.0 / math.sqrt(fan_in(s)) for s in shapes], dtype=torch.float32)
    reps = torch.tensor([numel(s) for s in shapes], dtype=torch.int64)
    return torch.repeat_interleave(vals, reps).to(device)


def student_t3(gen: torch.Generator, d: int, device) -> torch.Tensor:
    """Student-t with 3 degrees of freedom from four normal draws: z0 / sqrt((z1^2+z2^2+z3^2)/3)."""
    z = torch.randn(4, d, generator=gen, device=device, dtype=torch.float32)
    return z[0] / torch.sqrt((z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0)


@dataclass
class Workload:
    """One benchmark / parity configuration. `grads(step)` returns that step's [n, d] fp32 tensor."""
    name: str
    n: int
    d: int
    block_offsets: np.ndarray
    compressor: int
    k_ratio: float = 1.0
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    steps: int = 10
    seed: int = 0
    device: str = "cpu"
    _row: Optional[Callable[[torch.Generator], torch.Tensor]] = None
    _gen: Optional[torch.Generator] = field(default=None, repr=False)
    _extra: dict = field(default_factory=dict, repr=False)

    def start(self) -> torch.Tensor:
        """Seed the generator and draw theta_1 ~ N(0, 0.01) (sigma = 0.1); call before grads()."""
        self._gen = torch.Generator(device=self.device)
        self._gen.manual_seed(self.seed)
        theta = 0.1 * torch.randn(self.d, generator=self._gen, device=self.device, dtype=torch.float32)
        if "bias_sigma" in self._extra:
            self._extra["bias"] = self._extra["bias_sigma"] * torch.randn(
                self.d, generator=self._gen, device=self.device, dtype=torch.float32)
        return theta

    def grads(self) -> torch.Tensor:
        """The next step's gradients: rows drawn worker by worker from the running generator."""
        assert self._gen is not None, "call start() first"
        G = torch.empty(self.n, self.d, device=self.device, dtype=torch.float32)
        for i in range(self.n):
            G[i] = self._row(self)
        return G


def iid_normal(w: Workload) -> bool:
    """True when every coordinate of every row is an independent N(0,1) draw (one block, no per-tensor scale)."""
    return w._row is _row_normal and len(w.block_offsets) == 2


def grads_with_tail(w: Workload, extra: int) -> torch.Tensor:
    """For iid_normal workloads: one flat tensor of n*d + extra draws. Every window [o, o + n*d) of it, viewed as
    [n, d], is a gradient batch of the workload's distribution, and windows at different offsets give a coordinate
    independent values: a fresh batch per step out of one buffer."""
    assert iid_normal(w) and w._gen is not None
    flat = torch.empty(w.n * w.d + extra, device=w.device, dtype=torch.float32)
    for i in range(w.n):
        flat[i * w.d:(i + 1) * w.d] = _row_normal(w)
    flat[w.n * w.d:] = torch.randn(extra, generator=w._gen, device=w.device, dtype=torch.float32)
    return flat


def _row_normal(w: Workload) -> torch.Tensor:
    return torch.randn(w.d, generator=w._gen, device=w.device, dtype=torch.float32)


def _row_t3_scaled(w: Workload) -> torch.Tensor:
    return student_t3(w._gen, w.d, w.device) * w._extra["scale"]


def _row_t3_scaled_zeros(w: Workload) -> torch.Tensor:
    g = student_t3(w._gen, w.d, w.device) * w._extra["scale"]
    mask = torch.rand(w.d, generator=w._gen, device=w.device, dtype=torch.float32) < 0.05
    g[mask] = 0.0
    return g


def _row_normal_scaled_biased(w: Workload) -> torch.Tensor:
    return _row_normal(w) * w._extra["scale"] + w._extra["bias"]


def config1(device="cpu") -> Workload:
    """n=4, d=65,536, one block, Top-k 1% (k=655), gradients N(0,1)."""
    d = 65536
    return Workload("C1", 4, d, np.array([0, d], dtype=np.int64), TOPK, 0.01, device=device, _row=_row_normal)


def config2(device="cpu") -> Workload:
    """n=16, ResNet-18 tensors as 62 blocks, Block-Sign, Student-t(3) scaled by fan_in^(-1/2)."""
    shapes = resnet18_cifar_shapes()
    offs = offsets_from_shapes(shapes)
    w = Workload("C2", 16, int(offs[-1]), offs, BLOCKSIGN, 1.0, device=device, _row=_row_t3_scaled)
    w._extra["scale"] = per_coordinate_scale(shapes, device)
    return w


def config3(k_ratio: float, device="cpu") -> Workload:
    """Config 2's values with 5% exact zeros, one block, whole-vector Top-k at the given ratio."""
    shapes = resnet18_cifar_shapes()
    d = int(offsets_from_shapes(shapes)[-1])
    w = Workload("C3[k=%g]" % k_ratio, 16, d, np.array([0, d], dtype=np.int64), TOPK, k_ratio, device=device,
                 _row=_row_t3_scaled_zeros)
    w._extra["scale"] = per_coordinate_scale(shapes, device)
    return w


def config4(compressor: int, device="cpu", n: int = 32) -> Workload:
    """n=32, ResNet-50 tensors as 161 blocks; layer-wise Top-k 1% or Block-Sign.
    Gradients N(0, 1/fan_in) plus a persistent per-coordinate bias N(0, 1e-3)."""
    shapes = resnet50_imagenet_shapes()
    offs = offsets_from_shapes(shapes)
    name = "C4[topk]" if compressor == TOPK else "C4[sign]"
    w = Workload(name, n, int(offs[-1]), offs, compressor, 0.01 if compressor == TOPK else 1.0, device=device,
                 _row=_row_normal_scaled_biased)
    w._extra["scale"] = per_coordinate_scale(shapes, device)
    w._extra["bias_sigma"] = math.sqrt(1e-3)
    return w


def sweep_point(d: int, n: int, mode: str, device="cpu") -> Workload:
    """Scaling sweep: one block, gradients N(0,1); mode in {"topk", "sign", "dense", "randk"} (dense: k = d)."""
    comp = BLOCKSIGN if mode == "sign" else RANDK if mode == "randk" else TOPK
    ratio = {"topk": 0.01, "sign": 1.0, "dense": 1.0, "randk": 0.01}[mode]
    return Workload("C5[%s,d=%d,n=%d]" % (mode, d, n), n, d, np.array([0, d], dtype=np.int64), comp, ratio,
                    device=device, _row=_row_normal)
