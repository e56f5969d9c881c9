#!/usr/bin/env python
"""Benchmark of the COMP-AMS optimizer step on B200.

One benchmark "step" is one pass over the whole hot path on one batch of synthetic gradients
shaped like a ResNet-18 (n = 16 workers, d = 11,173,962): one Block-Sign step (62 blocks, one
per tensor), one whole-vector Top-k step (k = 1% of d) and one uncompressed step (k = d), each an
optimizer of its own with its own theta and state. The metric is gradient elements consumed
per second (n*d per optimizer step, three optimizer steps per benchmark step).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line. With --gpus N > 1 (under torch.distributed.run) every rank runs an
independent replica on its own GPU ("replicas only": the path has no inter-GPU exchange) and the
line reports the aggregate over the max time across ranks. --impl reference times the CPU oracle
on the host cores instead of the CUDA library.
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
MODES = ("blocksign", "topk", "dense")


def measured_peak_gbs():
    """HBM copy bandwidth measured on this machine (GB/s) and where the figure comes from."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture summarised in
# profiles/dram_traffic_bench_resnet18_n16.md, with a hash of the kernel's source code (comments and
# white space aside) at the time of the capture: once the code changes the figure no longer describes the
# kernel and None is reported.
TRAFFIC = {
    "bs_sweep": (2117579264, "blocksign.cu", "9447bdcb42baf658"),
    "topk_sweep": (2162749952, "topk.cu", "611f9fcc91e294db"),
    "dense_mean_amsgrad": (1144333312, "dense.cu", "c419baa10259b243"),
}


def code_hash(paths):
    """Hash of the concatenated sources with comments removed and white space collapsed."""
    import hashlib
    import re
    text = ""
    for p in paths:
        with open(p) as f:
            text += f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    text = re.sub(r"\s+", " ", text)
    return hashlib.sha256(text.encode()).hexdigest()[:16]


def captured_traffic(kernel: str):
    if kernel not in TRAFFIC:
        return None
    nbytes, src, want = TRAFFIC[kernel]
    base = os.path.join(ROOT, "paper_2205_05632_b200", "csrc")
    try:
        have = code_hash([os.path.join(base, src), os.path.join(base, "common.cuh")])
    except OSError:
        return None
    return nbytes if have == want else None


def min_bytes(mode: str, n: int, d: int) -> int:
    """Compulsory HBM bytes of one optimizer step: g and e read, e written (12 B per worker-element),
    m, v, vhat, theta read and written (32 B per coordinate); k = d never touches e."""
    return (4 * n + 32) * d if mode == "dense" else (12 * n + 32) * d


def build_workloads(device):
    """The three optimizers' inputs: two pre-generated gradient batches each (a ring), theta_1."""
    out = {}
    specs = {"blocksign": W.config2(device), "topk": W.config3(0.01, device)}
    for mode, w in specs.items():
        theta = w.start()
        out[mode] = dict(w=w, theta=theta, grads=[w.grads(), w.grads()])
    # the uncompressed step consumes the Block-Sign optimizer's gradients (same shapes, k = d)
    wd = W.config3(1.0, device)
    out["dense"] = dict(w=wd, theta=out["blocksign"]["theta"].clone(), grads=out["blocksign"]["grads"])
    return out


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


def time_oracle(wl, steps: int, warmup: int, workers=None):
    """Times the CPU oracle, as it stands, on the same workload (optionally only the first `workers`
    worker rows of it): seconds per benchmark step and the threads it used."""
    import oracle
    cores = oracle.max_threads()
    refs = {}
    for mode in MODES:
        w = wl[mode]["w"]
        ns = w.n if workers is None else min(workers, w.n)
        refs[mode] = dict(o=oracle.Oracle(ns, w.d, w.block_offsets, w.compressor, w.k_ratio, w.lr, w.beta1, w.beta2,
                                          w.eps),
                          theta=wl[mode]["theta"].cpu().numpy().copy(),
                          grads=[np.ascontiguousarray(g[:ns].cpu().numpy()) for g in wl[mode]["grads"]])

    def one(t):
        for mode in MODES:
            r = refs[mode]
            r["o"].step(r["grads"][t % 2], r["theta"])

    for t in range(warmup):
        one(t)
    t0 = time.perf_counter()
    for t in range(steps):
        one(warmup + t)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    for r in refs.values():
        r["o"].close()
    return dt, cores


def run_reference(args):
    """--impl reference: the oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = build_workloads("cpu")
    n, d = wl["topk"]["w"].n, wl["topk"]["w"].d
    # bounded sample: as many of the n worker rows as keep the whole run near two minutes
    probe, _ = time_oracle(wl, 1, 1, workers=1)
    per_step = 120.0 / max(args.steps + args.warmup, 1)
    ns = int(max(1, min(n, per_step / max(probe, 1e-9))))
    dt, cores = time_oracle(wl, args.steps, args.warmup, workers=ns)
    elems = len(MODES) * ns * d
    value = elems / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(n, d),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "the first %d of %d worker rows of the workload, every coordinate; %d steps "
                                   "after %d warm-up" % (ns, n, args.steps, args.warmup)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(n, d):
    return {
        "workload": "ResNet-18-shaped gradients (62 tensors, d=%d), n=%d workers: per step one Block-Sign step "
                    "(one block per tensor; Student-t(3) x fan_in^-1/2), one whole-vector Top-k step (k=1%% of d; "
                    "same values with 5%% exact zeros) and one uncompressed step (k=d)" % (d, n),
        "n_workers": n, "d": d, "optimizer_steps_per_step": len(MODES),
        "l2": "inputs larger than L2 (each [n,d] buffer is %.0f MB; ring of 2 gradient batches)" % (n * d * 4 / 1e6),
        "parallelism": "replicas only",
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (rank 0, N=1)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--e2e-steps", type=int, default=10)
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the COMP-AMS library has no CPU path")
    from paper_2205_05632_b200 import CompAMS

    from paper_2205_05632_b200 import replicas
    rank, world, local = replicas.rank_world_local()
    torch.cuda.set_device(local)
    dist = replicas.init("nccl", torch.device("cuda", local))

    device = "cuda"
    wl = build_workloads(device)
    n, d = wl["topk"]["w"].n, wl["topk"]["w"].d
    stream = torch.cuda.current_stream()
    opts = {}
    for mode in MODES:
        w = wl[mode]["w"]
        opts[mode] = CompAMS(w.n, w.d, w.block_offsets, w.compressor, w.k_ratio, w.lr, w.beta1, w.beta2, w.eps,
                             stream=stream)
    dominant = {"blocksign": "bs_sweep", "topk": "topk_sweep", "dense": "dense_mean_amsgrad"}

    def one_step(t):
        for mode in MODES:
            opts[mode].step(wl[mode]["grads"][t % 2], wl[mode]["theta"])

    def barrier():
        replicas.barrier(dist)

    for t in range(args.warmup):
        one_step(t)
    for mode in MODES:
        opts[mode].check_status()
        opts[mode].set_profiling([dominant[mode]])
    launches0 = sum(o.launch_count() for o in opts.values())

    # ---- timed region: K steps, device time from CUDA events on the launching stream
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(MODES) + 1)]
    mode_ms = {m: 0.0 for m in MODES}
    barrier()
    sampler = ClockSampler(local)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per_step_events = []
    start.record(stream)
    for t in range(args.steps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(MODES) + 1)]
        evs[0].record(stream)
        for k, mode in enumerate(MODES):
            opts[mode].step(wl[mode]["grads"][(args.warmup + t) % 2], wl[mode]["theta"])
            evs[k + 1].record(stream)
        per_step_events.append(evs)
    stop.record(stream)
    barrier()
    clocks = sampler.stop()
    elapsed_ms = start.elapsed_time(stop)
    for evs in per_step_events:
        for k, mode in enumerate(MODES):
            mode_ms[mode] += evs[k].elapsed_time(evs[k + 1])
    launches = sum(o.launch_count() for o in opts.values()) - launches0
    for o in opts.values():
        o.check_status()

    elapsed_ms = replicas.max_over_ranks(elapsed_ms, dist, device)
    ms_per_step = elapsed_ms / args.steps
    elems_per_step = len(MODES) * n * d
    value = replicas.aggregate_throughput(elems_per_step, world, ms_per_step)

    # ---- roofline of the dominant kernel, live from the event pairs recorded in the timed region
    peak, peak_kind = measured_peak_gbs()
    kern = {}
    for mode in MODES:
        ms, cnt = opts[mode].kernel_time(dominant[mode])
        kern[dominant[mode]] = (ms, cnt)
    top = max(kern, key=lambda k: kern[k][0])
    # algorithmic bytes per launch of the sweeps: g and e read, x/e written = 12 B per worker-element
    # (+ n*d/8 sign-bit bytes for Block-Sign); dense: (4n + 36) B per coordinate
    alg = {"bs_sweep": 12 * n * d + n * d // 8, "topk_sweep": 12 * n * d, "dense_mean_amsgrad": (4 * n + 36) * d}
    top_ms = kern[top][0] / max(kern[top][1], 1)
    achieved = alg[top] / (top_ms * 1e-3) / 1e9
    roofline = {"kernel": top, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": "of " + peak_kind, "traffic": captured_traffic(top),
                "avg_launch_ms": top_ms, "launches_timed": kern[top][1],
                "algorithmic_bytes_per_launch": alg[top]}
    per_kernel = {k: {"avg_ms": v[0] / max(v[1], 1), "launches": v[1],
                      "achieved_gbs": alg[k] / (v[0] / max(v[1], 1) * 1e-3) / 1e9 if v[0] > 0 else None}
                  for k, v in kern.items()}

    # ---- whole optimizer steps against their compulsory traffic
    modes_out = {}
    for mode in MODES:
        ms = mode_ms[mode] / args.steps
        bmin = min_bytes(mode, n, d)
        gbs = bmin / (ms * 1e-3) / 1e9
        modes_out[mode] = {"ms": ms, "elems_per_s": n * d / (ms * 1e-3), "steps_per_s": 1e3 / ms,
                           "min_bytes": bmin, "hbm_gbs": gbs, "frac_of_%s_peak" % peak_kind: gbs / peak,
                           "frac_of_8TBs": gbs / 8000.0}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(n, d),
        "clocks": clocks, "gpu_launches": launches, "roofline": roofline, "kernels": per_kernel, "modes": modes_out,
    }

    # ---- end to end through the C ABI with HOST buffers (copies inside the timed region)
    if not args.no_e2e:
        for o in opts.values():
            o.set_profiling([])
        host = {m: dict(g=[g.cpu().pin_memory() for g in wl[m]["grads"]], th=wl[m]["theta"].cpu().pin_memory())
                for m in ("blocksign", "topk")}
        host["dense"] = dict(g=host["blocksign"]["g"], th=wl["dense"]["theta"].cpu().pin_memory())
        for mode in MODES:  # allocate the staging buffers outside the timed region
            opts[mode].step_host(host[mode]["g"][0], host[mode]["th"])
        barrier()
        t0 = time.perf_counter()
        for t in range(args.e2e_steps):
            for mode in MODES:
                opts[mode].step_host(host[mode]["g"][t % 2], host[mode]["th"])
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.e2e_steps
        dt = replicas.max_over_ranks(dt, dist, device)
        line["e2e"] = {"value": world * elems_per_step / dt, "unit": UNIT, "ms_per_step": dt * 1e3,
                       "h2d_bytes_per_step": len(MODES) * (n * d * 4 + d * 4),
                       "d2h_bytes_per_step": len(MODES) * d * 4, "steps": args.e2e_steps,
                       "call": "compams_step_host (pinned host buffers, synchronous)"}

    # ---- the oracle on the host cores, rank 0 at N = 1 only
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt, cores = time_oracle(wl, 20, 1)
        line["cpu_baseline"] = {"value": elems_per_step / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "ms_per_step": dt * 1e3,
                                "sample": "20 steps of the full workload (all %d workers) after 1 warm-up step" % n}
    for o in opts.values():
        o.close()
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
