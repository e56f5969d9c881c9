"""Scaling sweep of the COMP-AMS step on one GPU: `python -m paper_2205_05632_b200.sweep [--out FILE]`.

One block of d coordinates, n workers, gradients i.i.d. N(0,1); Top-k (1 %), Block-Sign and the
uncompressed step (k = d) at every (d, n). Per point: step time from CUDA events over `--steps`
steps after `--warmup` steps (the Top-k threshold prediction needs a few steps to settle), gradient
elements per second, and the step's compulsory HBM bytes - g and e read, e written, m, v, v-hat,
theta read and written - over the measured time, as a fraction of a peak bandwidth.

Points whose [n, d] buffers fit the L2 cache are marked: there the step is not HBM-bound and the
fraction says nothing about the kernels.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

from . import CompAMS
from . import workloads as W

L2_BYTES = 126 * 1024 * 1024


def min_bytes(mode: str, n: int, d: int) -> int:
    return (4 * n + 32) * d if mode == "dense" else (12 * n + 32) * d


def peak_gbs(path: str | None):
    if path and os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured copy rate"
    return 6650.0, "fallback copy rate"


def time_point(d: int, n: int, mode: str, steps: int, warmup: int) -> float:
    """Milliseconds per step."""
    w = W.sweep_point(d, n, mode, "cuda")
    theta = w.start()
    ring = [w.grads(), w.grads()]
    opt = CompAMS(w.n, w.d, w.block_offsets, w.compressor, w.k_ratio)
    try:
        for t in range(warmup):
            opt.step(ring[t % 2], theta)
        if opt.check_status() != 0:
            raise RuntimeError("device status word is not clean")
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s.record()
        for t in range(steps):
            opt.step(ring[t % 2], theta)
        e.record()
        torch.cuda.synchronize()
        if opt.check_status() != 0:
            raise RuntimeError("device status word is not clean")
        return s.elapsed_time(e) / steps
    finally:
        opt.close()
        del ring, theta
        torch.cuda.empty_cache()


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--log2d", type=int, nargs="+", default=[20, 22, 24, 26, 27])
    ap.add_argument("--n", type=int, nargs="+", default=[1, 8, 32])
    ap.add_argument("--modes", nargs="+", default=["topk", "sign", "dense"], choices=["topk", "sign", "dense"])
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--peaks", default=os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                                    "MEASURED_PEAKS.json"))
    ap.add_argument("--out", default=None, help="also write the table to this file")
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        print("a CUDA device is required", file=sys.stderr)
        return 2
    peak, kind = peak_gbs(a.peaks)
    lines = ["| mode | d | n | ms/step | elem/s | min GB | GB/s | of %s (%.0f GB/s) | of 8 TB/s | note |" % (kind, peak),
             "|---|---:|---:|---:|---:|---:|---:|---:|---:|---|"]
    for mode in a.modes:
        for lg in a.log2d:
            for n in a.n:
                d = 1 << lg
                ms = time_point(d, n, mode, a.steps, a.warmup)
                mb = min_bytes(mode, n, d)
                gbs = mb / ms / 1e6
                note = "fits L2: not HBM-bound" if 2 * n * d * 4 <= L2_BYTES else ""
                lines.append("| %s | 2^%d | %d | %.4f | %.3e | %.3f | %.0f | %.3f | %.3f | %s |" % (
                    mode, lg, n, ms, n * d / ms * 1e3, mb / 1e9, gbs, gbs / peak, gbs / 8000.0, note))
                print(lines[-1], flush=True)
    text = "\n".join(lines) + "\n"
    if a.out:
        with open(a.out, "w") as f:
            f.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
