"""COMP-AMS as the optimizer of a torch model: n workers = n micro-batches whose gradients are kept
apart, compressed separately with error feedback and averaged by the server (Algorithm 2).

The model's parameters are re-pointed at slices of one flat fp32 tensor theta, the vector Algorithm 2
updates; every parameter tensor is one block of the compressor ("the blocks are usually the layers",
Section 3.1) unless whole_vector is set. Per step:

    for i in range(n_workers):
        loss_i = ...            # forward / backward of worker i's micro-batch
        loss_i.backward()
        opt.collect(i)          # row i of G <- the gradients, which are then cleared
    opt.step()                  # one COMP-AMS iteration; the model's parameters move with theta

torch is used for the model and its autograd; the optimizer step itself runs in the CUDA library.
"""
from __future__ import annotations

from typing import Iterable, List

import numpy as np
import torch

from .binding import RANDK, TOPK, CompAMS, CompAMSError


class CompAMSOptimizer:
    def __init__(self, params: Iterable[torch.nn.Parameter], n_workers: int, compressor: int = TOPK,
                 k_ratio: float = 0.01, whole_vector: bool = False, lr: float = 1e-3, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, seed: int = 0):
        self.params: List[torch.nn.Parameter] = [p for p in params if p.requires_grad]
        if not self.params:
            raise CompAMSError("no trainable parameters")
        dev = self.params[0].device
        if dev.type != "cuda" or any(p.device != dev or p.dtype != torch.float32 for p in self.params):
            raise CompAMSError("all parameters must be float32 tensors on one CUDA device")
        sizes = [p.numel() for p in self.params]
        self.offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
        self.d = int(self.offsets[-1])
        self.n = int(n_workers)
        # theta: the flat parameter vector; the model's tensors become views of it
        self.theta = torch.empty(self.d, dtype=torch.float32, device=dev)
        for p, lo, hi in zip(self.params, self.offsets[:-1], self.offsets[1:]):
            self.theta[lo:hi].copy_(p.data.reshape(-1))
            p.data = self.theta[lo:hi].view(p.shape)
        self.G = torch.zeros(self.n, self.d, dtype=torch.float32, device=dev)
        blocks = np.array([0, self.d], dtype=np.int64) if whole_vector else self.offsets
        with torch.cuda.device(dev):
            self.opt = CompAMS(self.n, self.d, blocks, compressor, k_ratio, lr, beta1, beta2, eps)
            if compressor == RANDK:
                self.opt.set_seed(seed)  # Random-k: the seed of the index sets

    def collect(self, worker: int) -> None:
        """Row `worker` of G <- the gradients accumulated since the last collect(); they are cleared."""
        if not 0 <= worker < self.n:
            raise CompAMSError("worker %d outside [0, %d)" % (worker, self.n))
        row = self.G[worker]
        for p, lo, hi in zip(self.params, self.offsets[:-1], self.offsets[1:]):
            if p.grad is None:
                row[lo:hi].zero_()
            else:
                row[lo:hi].copy_(p.grad.reshape(-1))
                p.grad = None

    def step(self) -> None:
        self.opt.step(self.G, self.theta)

    def set_lr(self, lr: float) -> None:
        self.opt.set_lr(lr)

    def close(self) -> None:
        self.opt.close()
