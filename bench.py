#!/usr/bin/env python
"""Benchmark of the grouped SQuant launch: weights quantized per second.

A step is one pass of the whole path (scale, SQuant-E, SQuant-K, candidate update, SQuant-C, emit)
over the large-layer workload: 8 conv layers [2048, 2048, 3, 3] fp32 (301,989,888 weights, 1.2 GB,
far larger than L2), 4 bit, E+K+C, one grouped kernel launch per step.

  python bench.py [--gpus N] [--steps K] [--warmup W]          the CUDA path (default)
  python bench.py --impl reference [...]                        the CPU checker on host cores

With N > 1 (torchrun, one rank per GPU) every rank quantizes its own copy of the workload
(different seed); there is no data-path collective, only the timing barrier and a MAX reduce.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOAD = "large_layer"
BITS = 4
METRIC = "weights_quantized_per_s"
UNIT = "weights/s"
# algorithmic bytes per weight of a 3x3 layer: 4 (fp32 read once) + 1 (int8 code)
# + 4/9 (kernel error sum) + 8/(N*K) (scale and channel error sum)
def algorithmic_bytes(shapes) -> float:
    total = 0.0
    for m, n, kh, kw in shapes:
        k = kh * kw
        total += m * n * k * 5.0 + m * n * 4.0 + m * 8.0
    return total


def source_digest() -> str:
    h = hashlib.sha256()
    for f in ("squant_device.cuh", "squant_pipe.cuh"):   # the device code; squant.cu is host code only
        with open(os.path.join(ROOT, "paper_2202_07471_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ncu_traffic():
    """DRAM bytes per launch from the committed ncu summary, or None if the kernel changed since."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as fh:
            t = json.load(fh)
        if t.get("source_digest") == source_digest() and t.get("workload") == WORKLOAD:
            return float(t["dram_bytes_per_launch"])
    except Exception:
        pass
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    NAMES = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
             0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
             0x10: "sync_boost", 0x100: "display_clock_setting"}

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else int(
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.NAMES.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                break
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ----------------------------------------------------------------------------- CPU checker arm
def oracle_rate(wl, seed, budget_s, threads=8):
    """Times the checker, as it stands, single-threaded on whole output channels of the workload
    until `budget_s` seconds of checker time are spent (at least one slab).  Returns
    (weights, seconds, description)."""
    import oracle
    from paper_2202_07471_b200 import workloads as W
    done_w, done_t, slabs = 0, 0.0, 0
    slab = 128                                       # output channels per slab
    m_total = wl.shapes[0][0]
    for layer in range(len(wl.shapes)):
        for c0 in range(0, m_total, slab):
            w = W.layer_weights(wl, layer, seed, channels=slice(c0, c0 + slab), threads=threads)
            t0 = time.perf_counter()
            oracle.quantize_layer(w, bits=BITS, mode=oracle.MODE_EKC)
            done_t += time.perf_counter() - t0
            done_w += w.size
            slabs += 1
            if done_t >= budget_s:
                return done_w, done_t, f"{slabs} slabs of {slab} output channels ({done_w} weights) of {wl.name}"
    return done_w, done_t, f"all {done_w} weights of {wl.name}"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2202_07471_b200 import workloads as W
    import oracle
    wl = W.WORKLOADS[WORKLOAD]
    steps, warmup = args.steps, args.warmup
    budget = min(1.0, 120.0 / max(1, steps + warmup))      # seconds of checker time per step
    per_ch = wl.shapes[0][1] * 9
    n_ch = max(1, min(2048, int(budget * 25e6 / per_ch)))  # whole output channels per step
    w = W.layer_weights(wl, 0, 0, channels=slice(0, n_ch), threads=os.cpu_count() or 1)
    for _ in range(warmup):
        oracle.quantize_layer(w, bits=BITS, mode=oracle.MODE_EKC)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.quantize_layer(w, bits=BITS, mode=oracle.MODE_EKC)
    dt = time.perf_counter() - t0
    value = w.size * steps / dt
    sample = f"each step = first {n_ch} output channels of layer 0 ({w.size} weights), 1 thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "bits": BITS, "mode": "E+K+C", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- CUDA arm
def run_cuda(args):
    import torch
    import paper_2202_07471_b200 as sq
    from paper_2202_07471_b200 import workloads as W
    from paper_2202_07471_b200 import dist as D

    rank, world, local = D.init_from_env(args.gpus)
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    sq.load_library()
    wl = W.WORKLOADS[WORKLOAD]
    n_weights = wl.n_weights
    steps, warmup = args.steps, max(3, args.warmup)

    # host inputs (pinned) from the seeded generator; each rank has its own seed
    ncpu = max(1, (os.cpu_count() or 1) // max(1, world))
    host = []
    for i, shp in enumerate(wl.shapes):
        t = torch.empty(shp, dtype=torch.float32, pin_memory=True)
        W.layer_weights(wl, i, seed=rank, threads=ncpu, out=t.numpy())
        host.append(t)
    dev = [sq.alloc_outputs(t.cuda(non_blocking=True)) for t in host]
    torch.cuda.synchronize()
    call = sq.ModelCall(dev, bits=BITS, mode=sq.MODE_EKC)
    stream = torch.cuda.current_stream()

    for _ in range(warmup):
        call.run(stream)
    torch.cuda.synchronize()

    # ---- device-resident timing: K launches, one CUDA event pair per launch on the launching
    # stream (for the kernel's own duration) inside one outer pair (for ms_per_step).
    sampler = ClockSampler(physical_gpu_index(local))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    outer = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    D.barrier()
    torch.cuda.synchronize()
    sampler.start()
    launches0 = sq.squant_launch_count()
    outer[0].record(stream)
    for a, b in ev:
        a.record(stream)
        call.run(stream)
        b.record(stream)
    outer[1].record(stream)
    torch.cuda.synchronize()
    launches = sq.squant_launch_count() - launches0
    D.barrier()
    clocks = sampler.stop()
    total_ms = D.max_over_ranks(outer[0].elapsed_time(outer[1]))
    kernel_ms = D.max_over_ranks(sum(a.elapsed_time(b) for a, b in ev) / steps)
    value = n_weights * world * steps / (total_ms * 1e-3)

    # ---- end to end through the host-buffer entry point: H2D of the weights, the launch, D2H of
    # codes / scales / error sums, every step.
    hb = [sq.alloc_outputs(t, pin=True) for t in host]
    hcall = sq.ModelCall(hb, bits=BITS, mode=sq.MODE_EKC)
    e2e_steps = max(1, min(steps, 10))
    for _ in range(2):
        hcall.run(stream)
    D.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        hcall.run(stream)                       # returns after the stream has drained
    e2e_s = D.max_over_ranks(time.perf_counter() - t0)
    h2d = sum(t.numel() * 4 for t in host)
    d2h = sum(b.codes.numel() + b.scales.numel() * 4 + b.kernel_err.numel() * 4 + b.channel_err.numel() * 4 for b in hb)
    same = all(torch.equal(a.codes.cpu(), b.codes) for a, b in zip(dev[:1], hb[:1]))

    # ---- latency of a whole small model in one launch (ResNet-50-shaped, L2 flushed before each)
    extra = {}
    if world == 1:
        r50 = W.WORKLOADS["resnet50"]
        rb = [sq.alloc_outputs(torch.from_numpy(W.layer_weights(r50, i, 0, threads=ncpu)).cuda()) for i in range(len(r50.shapes))]
        rcall = sq.ModelCall(rb, bits=BITS, mode=sq.MODE_EKC)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        for _ in range(3):
            rcall.run(stream)
        lat = []
        for _ in range(20):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); rcall.run(stream); b.record(stream)
            torch.cuda.synchronize()
            lat.append(a.elapsed_time(b))
        extra = {"resnet50_model_latency_ms": {"median": statistics.median(lat), "min": min(lat),
                                               "weights": r50.n_weights, "layers": len(r50.shapes),
                                               "l2": "flushed before each launch"}}
        del rb, flush

    if rank != 0:
        D.finish()
        return

    peak, peak_kind = measured_peak()
    alg = algorithmic_bytes(wl.shapes)
    achieved = alg / (kernel_ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": total_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": len(wl.shapes), "shape": list(wl.shapes[0]),
                   "weights_per_gpu": n_weights, "bits": BITS, "mode": "E+K+C",
                   "l2": "inputs (1.2 GB per step) larger than L2", "launches_per_step": 1},
        "clocks": clocks,
        "e2e": {"value": n_weights * world * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "matches_device_path": bool(same)},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": ncu_traffic(), "peak_kind": f"of {peak_kind}",
                     "kernel": "squant_pipe_kernel", "kernel_ms": kernel_ms,
                     "algorithmic_bytes_per_launch": alg},
    }
    out.update(extra)
    if world == 1 and not args.no_cpu_baseline:
        w_done, t_done, sample = oracle_rate(wl, 0, budget_s=args.cpu_budget, threads=ncpu)
        out["cpu_baseline"] = {"value": w_done / t_done, "unit": UNIT, "cores": 1, "kind": "oracle",
                               "sample": sample + ", 1 thread"}
    print(json.dumps(out))
    D.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of checker time for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
