#!/usr/bin/env python
"""Benchmark of the COMP-AMS optimizer step on B200.

One benchmark "step" is one optimizer step (Algorithm 2: every worker's x = g + e, compression, residual;
the server's average and AMSGrad update) of ONE compressor on one batch of synthetic gradients. The
headline workload is the largest single-GPU point of the scaling sweep: one block, d = 2^27 parameters,
n = 32 workers, gradients N(0,1), Top-k with k = 1 % of d. The metric is gradient elements consumed per
second (n d per step). Beside the headline the line carries, under "configs", one timed entry per
workload and compressor: C1 (n=4, d=65,536), C2 / C3 (ResNet-18 shapes, n=16: Block-Sign per tensor,
whole-vector Top-k at 0.1 % and 1 %), C4 (ResNet-50 shapes, n=32: layer-wise Top-k and Block-Sign) and the
scaling sweep C5 (d = 2^20 .. 2^27, n = 1, 8, 32, Top-k / Block-Sign / k = d), each with its step time,
its compulsory HBM bytes and the fraction of the HBM roofline that makes.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--only NAME ...]

Prints ONE JSON line. With --gpus N > 1 (under torch.distributed.run) every rank runs an independent
replica of the headline on its own GPU ("replicas only": the path has no inter-GPU exchange) and the line
reports the aggregate over the max time across ranks. --impl reference times the CPU oracle on the host
cores, on a bounded sample of the headline workload, instead of the CUDA library.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2205_05632_b200 import workloads as W

METRIC = "COMP-AMS step: gradient elems/s"
UNIT = "elem/s"
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0  # the nominal HBM3e figure the target fraction is quoted against

# kernels of each mode, the first one the dominant (the pass over [n, d])
KERNELS = {
    "topk": ["topk_sweep", "topk_select", "topk_dense", "topk_scatter", "amsgrad", "topk_small"],
    "sign": ["bs_sweep", "bs_scales", "bs_apply"],
    "dense": ["dense_mean_amsgrad"],
}


def measured_peak_gbs():
    """Measured HBM copy bandwidth (GB/s) from MEASURED_PEAKS.json beside this file, else the fallback figure."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per worker-element of one launch of the dominant
# kernel, from an ncu capture of a smaller case of the same kernel (d = 2^24, n = 8; the traffic of these
# streaming kernels grows in proportion to n d), with a hash of the kernel's source code (comments and white
# space aside) at the time of the capture: once the code changes the figure no longer describes the kernel and
# None is reported. The kernel's code is the stretch of its file between the two markers (the kernel with the
# device functions it alone uses) plus the shared helper header.
TRAFFIC_PER_ELEM = {
    "topk_sweep": (1599850752 / 134217728, "topk.cu", ("constexpr uint32_t kNothingKept", "void predict_next("),
                   "b1b2c4af58fd5755"),
}


def code_hash(paths, between=None):
    """Hash of the concatenated sources with comments removed and white space collapsed; of the first file only
    the stretch from the first marker of `between` up to the second."""
    import hashlib
    import re
    text = ""
    for k, p in enumerate(paths):
        with open(p) as f:
            part = f.read()
        if k == 0 and between is not None:
            a = part.index(between[0])
            part = part[a:part.index(between[1], a)]
        text += part
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    text = re.sub(r"\s+", " ", text)
    return hashlib.sha256(text.encode()).hexdigest()[:16]


def captured_traffic(kernel: str, elems: int):
    if kernel not in TRAFFIC_PER_ELEM:
        return None
    per_elem, src, between, want = TRAFFIC_PER_ELEM[kernel]
    base = os.path.join(ROOT, "paper_2205_05632_b200", "csrc")
    try:
        have = code_hash([os.path.join(base, src), os.path.join(base, "common.cuh")], between)
    except (OSError, ValueError):
        return None
    return int(per_elem * elems) if have == want else None


def min_bytes(mode: str, n: int, d: int, bf16: bool = False) -> int:
    """Compulsory HBM bytes of one optimizer step: g and e read, e written (12 B per worker-element, 10 B
    with bfloat16 gradients), m, v, vhat, theta read and written (32 B per coordinate); k = d never touches e."""
    g = 2 if bf16 else 4
    return (g * n + 32) * d if mode == "dense" else ((g + 8) * n + 32) * d


def algorithmic_bytes(kernel: str, n: int, d: int) -> int:
    """Bytes one launch of a dominant kernel must move: the sweeps read g and e and write x (12 B per
    worker-element, plus one sign bit for Block-Sign); the k = d kernel reads g and updates the state."""
    return {"bs_sweep": 12 * n * d + n * d // 8, "topk_sweep": 12 * n * d, "dense_mean_amsgrad": (4 * n + 32) * d}[kernel]


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------------------
# workloads

def headline_point(device) -> dict:
    """The largest single-GPU point of the scaling sweep that fits the device: d = 2^27, n = 32 needs about
    75 GB (two gradient batches, E, the end-to-end staging buffer); smaller devices take d = 2^26."""
    lg = 27
    if device != "cpu":
        free, _ = torch.cuda.mem_get_info()
        if free < 85 * (1 << 30):
            lg = 26
    return dict(config="C5", mode="topk", n=32, log2d=lg)


def describe(pt) -> str:
    return ("scaling sweep (C5) largest single-GPU point: one block, d = 2^%d, n = %d workers, gradients i.i.d. "
            "N(0,1), Top-k with k = 1%% of d; one optimizer step per benchmark step" % (pt["log2d"], pt["n"]))


def workload_config(pt):
    n, d = pt["n"], 1 << pt["log2d"]
    return {
        "workload": describe(pt), "n_workers": n, "d": d, "compressor": "topk", "k_ratio": 0.01,
        "l2": "inputs larger than L2 (each [n,d] buffer is %.1f GB)" % (n * d * 4 / 1e9),
        "parallelism": "replicas only",
    }


def _as_randk(w):
    """The same workload compressed with Random-k instead of Top-k."""
    w.compressor = W.RANDK
    w.name = w.name.replace("C3", "C3/randk")
    return w


def config_entries():
    """Every timed entry of "configs": (name, builder of the workload on a device, mode, bfloat16 input)."""
    out = [("C1/topk1%", lambda dev: W.config1(dev), "topk", False),
           ("C2/sign", lambda dev: W.config2(dev), "sign", False),
           ("C2/sign/bf16", lambda dev: W.config2(dev), "sign", True),
           ("C3/topk0.1%", lambda dev: W.config3(0.001, dev), "topk", False),
           ("C3/topk1%", lambda dev: W.config3(0.01, dev), "topk", False),
           ("C3/topk1%/bf16", lambda dev: W.config3(0.01, dev), "topk", True),
           ("C4/topk1%/layerwise", lambda dev: W.config4(W.TOPK, dev), "topk", False),
           ("C4/sign", lambda dev: W.config4(W.BLOCKSIGN, dev), "sign", False)]
    out.append(("C3/randk1%", lambda dev: _as_randk(W.config3(0.01, dev)), "randk", False))
    for lg in (20, 22, 24, 26, 27):
        for n in (1, 8, 32):
            for mode in ("topk", "sign", "dense") + (("randk",) if (lg, n) == (27, 32) else ()):
                out.append(("C5/%s/d=2^%d/n=%d" % (mode, lg, n),
                            (lambda dev, lg=lg, n=n, mode=mode: W.sweep_point(1 << lg, n, mode, dev)), mode, False))
    return out


FEED_RING = 8                 # gradient batches kept when they fit the budget below
FEED_RING_BYTES = 48 << 30
FEED_SHIFT = 64               # elements between the windows of consecutive steps: whole 128-byte lines in fp32 and bf16
FEED_PERIOD = 509             # windows before the offsets repeat


class GradientFeed:
    """A different gradient batch for every step, with nothing generated inside the timed region. Under error
    feedback a short cycle of batches is not a stand-in for training: with two alternating batches the
    accumulators settle into a period-two pattern whose selection threshold swings from step to step, which fresh
    gradients never do. So: a ring of FEED_RING batches drawn in advance when that fits FEED_RING_BYTES; for
    larger one-block workloads of independent N(0,1) entries one buffer of n d + tail draws, of which step t takes
    the window at offset FEED_SHIFT (t mod FEED_PERIOD) viewed as [n, d] - every coordinate sees an independent
    draw each step, and the rows keep their alignment; otherwise (no such workload exists among the entries) a
    ring of as many batches as fit, at least two."""

    batches = FEED_RING  # --feed-ring

    def __init__(self, w, bf16=False):
        per = w.n * w.d * 4
        self.n, self.d, self.flat, self.ring = w.n, w.d, None, None
        if GradientFeed.batches * per <= FEED_RING_BYTES or not W.iid_normal(w):
            count = max(2, min(GradientFeed.batches, FEED_RING_BYTES // per))
            self.ring = [w.grads() for _ in range(count)]
            if bf16:
                self.ring = [g.bfloat16() for g in self.ring]
            self.kind = "ring of %d gradient batches" % count
        else:
            self.flat = W.grads_with_tail(w, FEED_SHIFT * (FEED_PERIOD - 1))
            if bf16:
                self.flat = self.flat.bfloat16()
            self.kind = "a window moving by %d elements per step over one buffer of n d + %d draws" % (
                FEED_SHIFT, FEED_SHIFT * (FEED_PERIOD - 1))

    def __call__(self, t):
        if self.ring is not None:
            return self.ring[t % len(self.ring)]
        o = FEED_SHIFT * (t % FEED_PERIOD)
        return self.flat[o:o + self.n * self.d].view(self.n, self.d)


def time_entry(name, build, mode, bf16, steps, warmup, peak, peak_kind, cache):
    """Creates the workload and its optimizer, runs `warmup` + `steps` steps and returns the entry's record."""
    from paper_2205_05632_b200 import CompAMS
    w = build("cuda")
    key = (w.n, w.d, name.split("/")[0], bf16)
    if key in cache:  # the modes of one sweep point consume the same gradients
        theta0, feed = cache[key]
    else:
        cache.clear()
        torch.cuda.empty_cache()
        theta0 = w.start()
        feed = GradientFeed(w, bf16)
        cache[key] = (theta0, feed)
    theta = theta0.clone()
    opt = CompAMS(w.n, w.d, w.block_offsets, w.compressor, w.k_ratio, w.lr, w.beta1, w.beta2, w.eps)
    try:
        for t in range(warmup):
            opt.step(feed(t), theta)
        opt.check_status()
        st0 = opt.buffer("status").cpu().tolist()
        l0 = opt.launch_count()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s.record()
        for t in range(steps):
            opt.step(feed(warmup + t), theta)
        e.record()
        torch.cuda.synchronize()
        opt.check_status()
        ms = s.elapsed_time(e) / steps
        st1 = opt.buffer("status").cpu().tolist()
        launches = (opt.launch_count() - l0) / steps
        graph_ms = None
        if 2 * w.n * w.d * 4 <= L2_BYTES:
            # launch-bound: the same steps again as a CUDA graph of two captured steps (the handle's host-side
            # switches repeat with period two), replayed steps / 2 times
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                opt.set_stream(torch.cuda.current_stream())
                opt.step(feed(0), theta)
                opt.step(feed(1), theta)
            opt.set_stream(torch.cuda.current_stream())
            pairs = max(steps // 2, 1)
            graph.replay()
            torch.cuda.synchronize()
            s.record()
            for _ in range(pairs):
                graph.replay()
            e.record()
            torch.cuda.synchronize()
            opt.check_status()
            graph_ms = s.elapsed_time(e) / (2 * pairs)
            del graph
    finally:
        opt.close()
    mb = min_bytes(mode, w.n, w.d, bf16)
    gbs = mb / ms / 1e6
    fits_l2 = 2 * w.n * w.d * 4 <= L2_BYTES
    rec = {"name": name, "mode": mode, "n": w.n, "d": w.d, "blocks": int(len(w.block_offsets) - 1),
           "ms": ms, "elems_per_s": w.n * w.d / ms * 1e3, "min_bytes": mb, "launches_per_step": launches,
           "gradients": feed.kind}
    if fits_l2:
        rec["note"] = "launch-bound: inputs fit L2, no HBM fraction"
        rec["ms_as_cuda_graph"] = graph_ms
    else:
        rec.update({"hbm_gbs": gbs, "frac_of_%s" % peak_kind: gbs / peak, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS})
    if mode == "topk":
        # selections of the timed steps decided by the dense passes / inside the candidate lists, and why lists
        # were given up (too few, too many, out of range, crowded threshold bin)
        rec["status"] = {"word": st1[0], "dense": st1[1] - st0[1], "candidate": st1[2] - st0[2],
                         "gave_up": [st1[k] - st0[k] for k in (3, 4, 5, 6)]}
    return rec


# ------------------------------------------------------------------------------------------------------
# the oracle on the host cores

def oracle_sample(pt, rows_gpu=None, budget_s=20.0, steps=None, warmup=1):
    """Times the CPU oracle, as it stands, on a bounded sample of the headline workload: the first `ns`
    worker rows over the first `ds` coordinates (one block), shrunk until the run fits its time budget.
    Returns (elements per second, threads, description, seconds per step, steps timed)."""
    import oracle
    cores = oracle.max_threads()
    n, d = pt["n"], 1 << pt["log2d"]
    ns, ds = min(n, max(1, cores), 8), d

    def rows(ns_, ds_):
        if rows_gpu is not None:
            return np.ascontiguousarray(rows_gpu[:ns_, :ds_].cpu().numpy())
        gen = torch.Generator().manual_seed(0)
        return torch.randn(ns_, ds_, generator=gen, dtype=torch.float32).numpy()

    while True:
        G = rows(ns, ds)
        o = oracle.Oracle(ns, ds, [0, ds], oracle.TOPK, 0.01)
        theta = np.zeros(ds, dtype=np.float32)
        t0 = time.perf_counter()
        o.step(G, theta)
        probe = time.perf_counter() - t0
        want_steps = steps if steps is not None else max(2, int(budget_s / max(probe, 1e-6)))
        total = probe * (want_steps + warmup)
        if steps is None or total <= budget_s or (ns == 1 and ds <= (1 << 20)):
            break
        o.close()
        # too slow for the budget: fewer rows first (they run in parallel up to the core count), then fewer coordinates
        if ns > 1:
            ns = 1
        else:
            ds = max(1 << 20, ds // 4)
    if steps is None:
        want_steps = min(want_steps, 20)
    for _ in range(max(0, warmup - 1)):
        o.step(G, theta)
    t0 = time.perf_counter()
    for _ in range(want_steps):
        o.step(G, theta)
    dt = (time.perf_counter() - t0) / want_steps
    o.close()
    what = ("the first %d of %d worker rows%s of the headline workload, Top-k 1%%; %d steps after %d warm-up" % (
        ns, n, "" if ds == d else " over the first %d of %d coordinates" % (ds, d), want_steps, warmup))
    return ns * ds / dt, cores, what, dt, want_steps


def run_reference(args):
    """--impl reference: the oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    pt = dict(config="C5", mode="topk", n=32, log2d=27)
    value, cores, what, dt, _ = oracle_sample(pt, None, budget_s=150.0, steps=args.steps, warmup=max(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(pt),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (rank 0, N=1)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration entries")
    ap.add_argument("--no-headline", action="store_true", help="time only the entries selected with --only")
    ap.add_argument("--only", nargs="*", default=None, help="names (or prefixes) of the 'configs' entries to time")
    ap.add_argument("--config-steps", type=int, default=20)
    ap.add_argument("--config-warmup", type=int, default=40)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--feed-ring", type=int, default=FEED_RING,
                    help="gradient batches prepared per entry (profiler captures of small cases use 2 to hold less memory)")
    args = ap.parse_args()
    GradientFeed.batches = max(2, args.feed_ring)

    if args.impl == "reference":
        run_reference(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the COMP-AMS library has no CPU path")
    from paper_2205_05632_b200 import CompAMS, replicas

    rank, world, local = replicas.rank_world_local()
    torch.cuda.set_device(local)
    dist = replicas.init("nccl", torch.device("cuda", local))
    device = "cuda"
    peak, peak_kind = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    line = {}

    if not args.no_headline:
        pt = headline_point(device)
        n, d = pt["n"], 1 << pt["log2d"]
        w = W.sweep_point(d, n, "topk", device)
        theta = w.start()
        feed = GradientFeed(w)
        opt = CompAMS(w.n, w.d, w.block_offsets, w.compressor, w.k_ratio, w.lr, w.beta1, w.beta2, w.eps, stream=stream)
        # at least three warm-up steps: the first selections run the dense passes, the threshold prediction
        # carries the rest
        for t in range(max(args.warmup, 3)):
            opt.step(feed(t), theta)
        opt.check_status()
        st0 = opt.buffer("status").cpu().tolist()
        opt.set_profiling(["topk_sweep"])
        launches0 = opt.launch_count()

        # ---- timed region: K steps, device time from CUDA events on the launching stream
        replicas.barrier(dist)
        sampler = ClockSampler(local)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for t in range(args.steps):
            opt.step(feed(args.warmup + t), theta)
        stop.record(stream)
        replicas.barrier(dist)
        clocks = sampler.stop()
        elapsed_ms = start.elapsed_time(stop)
        launches = opt.launch_count() - launches0
        opt.check_status()
        st1 = opt.buffer("status").cpu().tolist()
        sweep_ms, sweep_cnt = opt.kernel_time("topk_sweep")

        elapsed_ms = replicas.max_over_ranks(elapsed_ms, dist, device)
        ms_per_step = elapsed_ms / args.steps
        value = replicas.aggregate_throughput(n * d, world, ms_per_step)

        # ---- roofline: the dominant kernel live from the event pairs of the timed region, and the whole step
        # against its compulsory bytes
        alg = algorithmic_bytes("topk_sweep", n, d) * args.steps  # every step sweeps all n rows (in one or more launches)
        achieved = alg / (sweep_ms * 1e-3) / 1e9 if sweep_ms > 0 else None
        mb = min_bytes("topk", n, d)
        step_gbs = mb / (ms_per_step * 1e-3) / 1e9
        roofline = {"kernel": "topk_sweep", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak if achieved else None, "peak_kind": "of " + peak_kind,
                    "traffic": captured_traffic("topk_sweep", n * d),
                    "avg_launch_ms": sweep_ms / max(sweep_cnt, 1), "launches_timed": sweep_cnt,
                    "algorithmic_bytes_per_step": alg // args.steps,
                    "step_min_bytes": mb, "step_gbs": step_gbs, "step_frac": step_gbs / peak,
                    "step_frac_of_8TBs": step_gbs / NOMINAL_HBM_GBS}

        # ---- per-kernel breakdown of the step, from a few extra steps with an event pair around every launch
        opt.set_profiling(KERNELS["topk"])
        for t in range(3):
            opt.step(feed(args.warmup + args.steps + t), theta)  # the gradients go on in step
        per_kernel = {}
        for k in KERNELS["topk"]:
            ms, cnt = opt.kernel_time(k)
            if cnt:
                per_kernel[k] = {"ms_per_step": ms / 3}
        opt.set_profiling([])

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "steps_per_s": 1e3 / ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(pt),
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline, "kernels": per_kernel,
            "gradients": feed.kind,
            "status": {"word": st1[0], "dense": st1[1] - st0[1], "candidate": st1[2] - st0[2],
                       "gave_up": [st1[k] - st0[k] for k in (3, 4, 5, 6)]},
        }

        # ---- end to end through the C ABI with HOST buffers (copies inside the timed region)
        if not args.no_e2e:
            hg = ht = None
            try:  # n d 4 bytes of pinned host memory per rank: every rank must get its own or all skip the leg
                hg = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
                ht = torch.empty(d, dtype=torch.float32, pin_memory=True)
                ok = 1.0
            except RuntimeError:
                ok = 0.0
            if -replicas.max_over_ranks(-ok, dist, device) > 0.5:
                hg.copy_(feed(0))
                ht.copy_(theta)
                opt.step_host(hg, ht)  # allocates the staging buffers outside the timed region
                replicas.barrier(dist)
                t0 = time.perf_counter()
                for t in range(args.e2e_steps):
                    opt.step_host(hg, ht)
                torch.cuda.synchronize()
                dt = (time.perf_counter() - t0) / args.e2e_steps
                dt = replicas.max_over_ranks(dt, dist, device)
                line["e2e"] = {"value": world * n * d / dt, "unit": UNIT, "ms_per_step": dt * 1e3,
                               "h2d_bytes_per_step": n * d * 4 + d * 4, "d2h_bytes_per_step": d * 4,
                               "steps": args.e2e_steps, "call": "compams_step_host (pinned host buffers, synchronous)"}
            else:
                line["e2e"] = {"value": None, "unit": UNIT, "unavailable": "a rank could not pin %.1f GB of host memory" % (n * d * 4 / 1e9)}
            del hg, ht

        # ---- the oracle on the host cores, rank 0 at N = 1 only
        if rank == 0 and world == 1 and not args.no_cpu_baseline:
            v, cores, what, dt, _ = oracle_sample(pt, feed(0), budget_s=20.0)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "ms_per_step": dt * 1e3,
                                    "sample": what}
        opt.close()
        del feed, theta
        torch.cuda.empty_cache()

    # ---- every configuration, one compressor per number (rank 0 at N = 1 only)
    if rank == 0 and world == 1 and not args.no_configs:
        entries, cache = [], {}
        for name, build, mode, bf16 in config_entries():
            if args.only is not None and not any(name.startswith(p) for p in args.only):
                continue
            entries.append(time_entry(name, build, mode, bf16, args.config_steps, args.config_warmup, peak, peak_kind,
                                      cache))
        cache.clear()
        line["configs"] = entries
        line["configs_protocol"] = ("per entry: %d steps between two CUDA events after %d warm-up steps, a different "
                                    "gradient batch every step (each entry's `gradients`); min_bytes = (12 n + 32) d with error feedback ((10 n + 32) d with bfloat16 "
                                    "gradients), (4 n + 32) d for k = d" % (args.config_steps, args.config_warmup))
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
