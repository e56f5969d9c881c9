"""Side-by-side runs of the CUDA library (through its C ABI) and the CPU oracle on the same inputs.

The bar, per step and with each side chained on its own state: Top-k index sets and Block-Sign
sign bits bit-exact; every float buffer (gbar, e, m, v, vhat, theta, kept values, scales) within
|gpu - cpu| <= 1e-7 + 1e-6 |cpu|.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2205_05632_b200 import BLOCKSIGN, RANDK, TOPK, CompAMS

ATOL, RTOL = 1e-7, 1e-6


_CHUNK = 1 << 28  # elements compared at a time: bounds the temporaries at the largest sizes


def close(gpu: torch.Tensor, cpu: np.ndarray, what: str, step: int) -> int:
    """Asserts the tolerance elementwise (on the GPU, the arrays can be large). Returns the number of
    elements that are not bit-identical, for reporting."""
    cpu = np.ascontiguousarray(cpu)
    assert tuple(cpu.shape) == tuple(gpu.shape), (what, cpu.shape, tuple(gpu.shape))
    g_flat, c_flat = gpu.reshape(-1), cpu.reshape(-1)
    inexact = 0
    for lo in range(0, g_flat.numel(), _CHUNK):
        hi = min(lo + _CHUNK, g_flat.numel())
        g = g_flat[lo:hi]
        ref = torch.from_numpy(c_flat[lo:hi]).to(gpu.device)
        bad = (g - ref).abs() > (ATOL + RTOL * ref.abs())
        nbad = int(bad.sum())
        if nbad:
            j = int(torch.nonzero(bad)[0])
            raise AssertionError("step %d: %s differs at %d element(s) of a chunk; first at flat index %d: gpu=%r cpu=%r" % (
                step, what, nbad, lo + j, float(g[j]), float(ref[j])))
        inexact += int((g.view(torch.int32) != ref.view(torch.int32)).sum())
        del ref, bad
    return inexact


def unpack_sign_bits(bits: np.ndarray, word_off: np.ndarray, block_offsets: np.ndarray) -> np.ndarray:
    """[n, W] words (each block starting at its own word, LSB first) -> [n, d] booleans."""
    n = bits.shape[0]
    d = int(block_offsets[-1])
    out = np.zeros((n, d), dtype=bool)
    u8 = np.ascontiguousarray(bits).view(np.uint8).reshape(n, -1)
    for b in range(len(block_offsets) - 1):
        lo, hi = int(block_offsets[b]), int(block_offsets[b + 1])
        w0, w1 = int(word_off[b]), int(word_off[b + 1])
        blk = np.unpackbits(u8[:, 4 * w0:4 * w1], axis=1, bitorder="little")
        out[:, lo:hi] = blk[:, :hi - lo].astype(bool)
        assert not blk[:, hi - lo:].any(), "padding bits of block %d are not zero" % b
    return out


class Pair:
    """A CUDA optimizer and an oracle built from the same arguments."""

    def __init__(self, n, d, block_offsets, compressor, k_ratio=1.0, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                 seed=None):
        self.n, self.d = n, d
        self.offsets = np.asarray(block_offsets, dtype=np.int64)
        self.compressor = compressor
        hp = dict(lr=lr, beta1=beta1, beta2=beta2, eps=eps)
        self.gpu = CompAMS(n, d, self.offsets, compressor, k_ratio, record_average=True, **hp)
        self.cpu = oracle.Oracle(n, d, self.offsets, compressor, k_ratio, **hp)
        sizes = np.diff(self.offsets)
        if seed is not None:  # Random-k: the same seed for the index sets on both sides
            self.gpu.set_seed(seed)
            self.cpu.set_seed(seed)
        self.identity = compressor in (TOPK, RANDK) and all(oracle.kept_per_block(k_ratio, int(s)) == int(s) for s in sizes)
        self.step_no = 0
        self.inexact = {}

    def start(self, theta0: torch.Tensor):
        self.theta_gpu = theta0.detach().to("cuda").clone()
        self.theta_cpu = theta0.detach().cpu().numpy().copy()

    def step(self, G: torch.Tensor, check_e: bool = True):
        """One step on both sides from the same gradient tensor, then the full comparison."""
        self.step_no += 1
        s = self.step_no
        Gd = G.to("cuda")
        self.gpu.step(Gd, self.theta_gpu)
        # bfloat16 gradients: the oracle is fed the fp32 numbers with the same values (widening is exact)
        self.cpu.step(np.ascontiguousarray(G.detach().float().cpu().numpy()), self.theta_cpu)
        assert self.gpu.check_status() == 0
        cnt = self.inexact
        if self.compressor in (TOPK, RANDK) and not self.identity:
            idx = self.gpu.buffer("topk_idx").cpu().numpy()
            val = self.gpu.buffer("topk_val")
            order = np.argsort(idx, axis=1, kind="stable")
            idx_sorted = np.take_along_axis(idx, order, axis=1)
            want = self.cpu.buffer("kept_idx")
            # segments of successive blocks hold increasing coordinate ranges, so sorting a worker's
            # row sorts every segment in place: the sets must agree entry by entry
            if not np.array_equal(idx_sorted, want):
                i, p = np.argwhere(idx_sorted != want)[0]
                raise AssertionError("step %d: Top-k index sets differ (worker %d, entry %d: gpu %d, oracle %d)" % (
                    s, i, p, idx_sorted[i, p], want[i, p]))
            seg = self.gpu.buffer("topk_seg_offsets").cpu().numpy()
            assert np.array_equal(seg, self.cpu.buffer("seg_off"))
            # each message entry sits in the segment of the block that owns its coordinate
            blk_of = np.searchsorted(self.offsets, idx, side="right") - 1
            pos = np.broadcast_to(np.arange(idx.shape[1]), idx.shape)
            assert np.all((pos >= seg[blk_of]) & (pos < seg[blk_of + 1])), "an entry is outside its block's segment"
            C = self.cpu.buffer("C")
            want_val = np.take_along_axis(C, idx.astype(np.int64), axis=1)
            nb = int((val.view(torch.int32).cpu().numpy() != want_val.view(np.int32)).sum())
            assert nb == 0, "step %d: %d kept values are not bit-identical to x" % (s, nb)
        elif self.compressor == BLOCKSIGN:
            bits = self.gpu.buffer("sign_bits").cpu().numpy()
            woff = self.gpu.buffer("sign_word_offsets").cpu().numpy()
            got = unpack_sign_bits(bits, woff, self.offsets)
            want = np.signbit(self.cpu.buffer("C"))
            if not np.array_equal(got, want):
                i, j = np.argwhere(got != want)[0]
                raise AssertionError("step %d: %d sign bits differ; first at worker %d coordinate %d" % (
                    s, int((got != want).sum()), i, j))
            cnt["scales"] = cnt.get("scales", 0) + close(self.gpu.buffer("scales"), self.cpu.buffer("scales"),
                                                         "scales", s)
        for name in ("gbar", "m", "v", "vhat"):
            cnt[name] = cnt.get(name, 0) + close(self.gpu.buffer(name), self.cpu.buffer(name), name, s)
        cnt["theta"] = cnt.get("theta", 0) + close(self.theta_gpu, self.theta_cpu, "theta", s)
        if check_e:
            cnt["E"] = cnt.get("E", 0) + close(self.gpu.buffer("E"), self.cpu.buffer("E"), "E", s)

    def set_lr(self, lr: float):
        """eta_t of the following steps, on both sides (Algorithm 2 lets the learning rate vary with t)."""
        self.gpu.set_lr(lr)
        self.cpu.set_lr(lr)

    def close(self):
        self.gpu.close()
        self.cpu.close()


def run_workload(w, steps=None, check_e_every=1):
    """Chained parity over a workloads.Workload; returns the per-buffer counts of non-bit-identical floats."""
    p = Pair(w.n, w.d, w.block_offsets, w.compressor, w.k_ratio, w.lr, w.beta1, w.beta2, w.eps)
    try:
        p.start(w.start())
        T = steps if steps is not None else w.steps
        for t in range(T):
            p.step(w.grads(), check_e=(t % check_e_every == 0) or t == T - 1)
        return p.inexact
    finally:
        p.close()
