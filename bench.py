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

At N = 1 the outputs that were timed are then compared, channel by channel, with the CPU checker
run over the whole workload on all host cores ("parity"), the checker is timed single-threaded on
a sample ("cpu_baseline") and every other configuration is timed and checked in full ("configs").
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
    for f in ("squant_device.cuh", "squant_pipe.cuh", "squant_stream.cuh"):   # the device code; squant.cu is host code only
        with open(os.path.join(ROOT, "paper_2202_07471_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def nominal_peak_gbs() -> float:
    """HBM peak as the profiler states it: DRAM bytes per second of the committed capture divided
    by its own percent-of-peak figure (falls back to the 8 TB/s of the data sheet)."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as fh:
            return float(json.load(fh)["ncu_dram_peak_gbs"])
    except Exception:
        return 8000.0


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

    def __init__(self, index: int, period_s: float = 0.002):
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
def _same_words(a, b) -> bool:
    return np.array_equal(np.ascontiguousarray(a).view(np.uint32), np.ascontiguousarray(b).view(np.uint32))


def oracle_single_thread(host, budget_s):
    """Times the checker, as it stands, on ONE thread over whole output channels of the workload
    (slabs of 128 channels, layer after layer) until `budget_s` seconds are spent.  Returns
    (weights, seconds, description)."""
    import oracle
    done_w, done_t, slabs, slab = 0, 0.0, 0, 128
    for w in host:
        for c0 in range(0, w.shape[0], slab):
            part = w[c0:c0 + slab]
            t0 = time.perf_counter()
            oracle.quantize_layer(part, bits=BITS, mode=oracle.MODE_EKC)
            done_t += time.perf_counter() - t0
            done_w += part.size
            slabs += 1
            if done_t >= budget_s:
                return done_w, done_t, f"{slabs} slabs of {slab} output channels ({done_w} weights), 1 thread"
    return done_w, done_t, f"all {done_w} weights, 1 thread"


def oracle_check_all(host, outs, bits, mode, threads, slab=64):
    """Runs the checker over EVERY output channel of the given layers (numpy weights `host`) on
    `threads` host threads - channels are independent sub-problems, so the split changes nothing -
    and compares each slab with every output set in `outs` (lists of per-layer tuples
    (codes, scales, kernel_err, channel_err) of numpy arrays).  Returns (channels, mismatching
    channels per output set, seconds of wall clock)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    jobs = [(i, c0) for i, w in enumerate(host) for c0 in range(0, w.shape[0], slab)]

    def work(job):
        i, c0 = job
        r = oracle.quantize_layer(host[i][c0:c0 + slab], bits=bits, mode=mode)
        bad = []
        for o in outs:
            codes, scales, kerr, cerr = o[i]
            ok = (np.array_equal(codes[c0:c0 + slab], r.codes) and _same_words(scales[c0:c0 + slab], r.scales)
                  and _same_words(kerr[c0:c0 + slab], r.kernel_err) and _same_words(cerr[c0:c0 + slab], r.channel_err))
            if ok:
                bad.append(0)
            else:   # count the channels of the slab that differ anywhere
                n = r.codes.shape[0]
                d = np.zeros(n, dtype=bool)
                d |= (codes[c0:c0 + slab].reshape(n, -1) != r.codes.reshape(n, -1)).any(1)
                d |= scales[c0:c0 + slab].view(np.uint32) != r.scales.view(np.uint32)
                d |= (kerr[c0:c0 + slab].view(np.uint32) != r.kernel_err.view(np.uint32)).any(1)
                d |= cerr[c0:c0 + slab].view(np.uint32) != r.channel_err.view(np.uint32)
                bad.append(int(d.sum()))
        return bad

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:   # the checker is C code called through ctypes: the GIL is released
        res = list(ex.map(work, jobs))
    dt = time.perf_counter() - t0
    channels = sum(w.shape[0] for w in host)
    return channels, [sum(r[k] for r in res) for k in range(len(outs))], dt


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
def _to_host(bufs):
    return [(b.codes.cpu().numpy(), b.scales.cpu().numpy(), b.kernel_err.cpu().numpy(), b.channel_err.cpu().numpy()) for b in bufs]


def time_model(sq, torch, bufs, bits, mode, stream, flush, reps=15, flags=None):
    """One call over all layers: median milliseconds with L2 flushed before every call, and warm."""
    call = sq.ModelCall(bufs, bits=bits, mode=mode) if flags is None else sq.ModelCall(bufs, bits=bits, mode=mode, flags=flags)
    for _ in range(3):
        call.run(stream)
    out = {}
    for kind in ("cold", "warm"):
        lat = []
        for _ in range(reps):
            if kind == "cold":
                flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); call.run(stream); b.record(stream)
            torch.cuda.synchronize()
            lat.append(a.elapsed_time(b))
        out[kind] = statistics.median(lat)
    return out


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
    # The timed steps last a few milliseconds: too short for the clock sampler (NVML, every 2 ms).  The same
    # launches run untimed for 60 ms right before them, with the sampler on, so that the clocks and throttle
    # reasons reported are those of this workload under load; sampling goes on through the timed steps.
    t_settle = time.perf_counter()
    while time.perf_counter() - t_settle < 0.06:
        for _ in range(8):
            call.run(stream)
        torch.cuda.synchronize()
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
    clocks["window"] = "60 ms of the same launches right before the timed steps, and the timed steps"
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

    extra = {}
    if world == 1:
        # ---- the other configurations: whole model in one call, L2 cold and warm, every element
        # compared with the checker; and the E|C ablation on one large layer (its channel step
        # selects among all N*K elements)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        peak, _ = measured_peak()
        cfgs = {}
        for name, bits in (("single_conv", 4), ("resnet18", 4), ("resnet50", 4), ("resnet50", 6), ("mobilenetv2", 4),
                           ("mixed_kernels", 4)):
            w2 = W.WORKLOADS[name]
            hw = [W.layer_weights(w2, i, 0, threads=ncpu) for i in range(len(w2.shapes))]
            bufs = [sq.alloc_outputs(torch.from_numpy(x).cuda()) for x in hw]
            t = time_model(sq, torch, bufs, bits, sq.MODE_EKC, stream, flush)
            ch, bad, _ = oracle_check_all(hw, [_to_host(bufs)], bits, sq.MODE_EKC, ncpu)
            alg = algorithmic_bytes(w2.shapes)
            cfgs[name + ("" if bits == 4 else f"_{bits}bit")] = {
                "layers": len(w2.shapes), "weights": w2.n_weights, "bits": bits, "ms_cold": t["cold"], "ms_warm": t["warm"],
                "weights_per_s_cold": w2.n_weights / (t["cold"] * 1e-3), "gbs_cold": alg / (t["cold"] * 1e-3) / 1e9,
                "frac_of_measured_cold": alg / (t["cold"] * 1e-3) / 1e9 / peak, "channels": ch, "mismatches": bad[0]}
            del bufs
        one = torch.from_numpy(host[0].numpy()).cuda()
        eb = [sq.alloc_outputs(one)]
        mode_ec = sq.MODE_E | sq.MODE_C
        t = time_model(sq, torch, eb, BITS, mode_ec, stream, flush, reps=7)
        ch, bad, _ = oracle_check_all([host[0].numpy()[:256]], [[tuple(a[:256] for a in _to_host(eb)[0])]], BITS, mode_ec, ncpu)
        cfgs["large_layer_one_layer_E|C"] = {"layers": 1, "weights": one.numel(), "bits": BITS, "ms_cold": t["cold"], "ms_warm": t["warm"],
                                             "weights_per_s_cold": one.numel() / (t["cold"] * 1e-3), "channels": ch, "mismatches": bad[0],
                                             "note": "checker compared on the first 256 output channels"}
        # packed int4 codes on the same layer (4 + 0.5 + 4/9 B per weight): long channels with packed or
        # dequantized outputs take the pipelined kernel
        pk = [sq.alloc_outputs(one, pack_int4=True)]
        pflags = sq.FLAG_NARROW_RANGE | sq.FLAG_PACK_INT4
        t = time_model(sq, torch, pk, BITS, sq.MODE_EKC, stream, flush, reps=7, flags=pflags)
        import oracle
        rp = oracle.quantize_layer(host[0].numpy()[:256], bits=BITS, mode=sq.MODE_EKC, flags=pflags)
        pbad = int((pk[0].codes[:256].cpu().numpy() != rp.codes).any(1).sum()
                   + (pk[0].kernel_err[:256].cpu().numpy().view(np.uint32) != rp.kernel_err.view(np.uint32)).any(1).sum())
        palg = one.numel() * (4 + 0.5 + 4 / 9) + one.shape[0] * 8
        cfgs["large_layer_one_layer_packed_int4"] = {
            "layers": 1, "weights": one.numel(), "bits": BITS, "ms_cold": t["cold"], "ms_warm": t["warm"],
            "weights_per_s_cold": one.numel() / (t["cold"] * 1e-3), "gbs_cold": palg / (t["cold"] * 1e-3) / 1e9,
            "frac_of_measured_cold": palg / (t["cold"] * 1e-3) / 1e9 / peak, "channels": 256, "mismatches": pbad,
            "note": "checker compared on the first 256 output channels"}
        del eb, pk, one, flush
        r50 = cfgs["resnet50"]
        extra = {"configs": cfgs,
                 "resnet50_model_latency_ms": {"median": r50["ms_cold"], "weights": r50["weights"], "layers": r50["layers"],
                                               "l2": "flushed before each launch"}}

    if rank != 0:
        D.finish()
        return

    peak, peak_kind = measured_peak()
    nominal = nominal_peak_gbs()
    alg = algorithmic_bytes(wl.shapes)
    achieved = alg / (kernel_ms * 1e-3) / 1e9
    traffic = ncu_traffic()
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
            "peak_ncu": nominal, "frac_of_ncu_peak": achieved / nominal,
            "kernel": "squant_stream_kernel", "kernel_ms": kernel_ms, "algorithmic_bytes_per_launch": alg}
    if traffic:   # what actually crossed the DRAM interface (part of the output is still in L2 at kernel end)
        roof["achieved_dram"] = traffic / (kernel_ms * 1e-3) / 1e9
        roof["frac_dram_of_measured"] = roof["achieved_dram"] / peak
        roof["frac_dram_of_ncu_peak"] = roof["achieved_dram"] / nominal
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": total_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": len(wl.shapes), "shape": list(wl.shapes[0]),
                   "weights_per_gpu": n_weights, "bits": BITS, "mode": "E+K+C",
                   "l2": "inputs (1.2 GB per step) larger than L2", "launches_per_step": 1},
        "clocks": clocks,
        "e2e": {"value": n_weights * world * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roof,
    }
    out.update(extra)
    if world == 1 and not args.no_cpu_baseline:
        # ---- the checker: one thread on a sample (the reported baseline), then all host cores over
        # EVERY output channel, compared with the outputs of the timed device-resident run and of
        # the host-buffer run
        hnp = [t.numpy() for t in host]
        w_done, t_done, sample = oracle_single_thread(hnp, budget_s=args.cpu_budget)
        out["cpu_baseline"] = {"value": w_done / t_done, "unit": UNIT, "cores": 1, "kind": "oracle",
                               "sample": sample + f" of {wl.name}"}
        dev_out = _to_host(dev)
        hb_out = [(b.codes.numpy(), b.scales.numpy(), b.kernel_err.numpy(), b.channel_err.numpy()) for b in hb]
        ch, bad, dt = oracle_check_all(hnp, [dev_out, hb_out], BITS, sq.MODE_EKC, ncpu)
        out["cpu_baseline"]["all_cores"] = {"value": n_weights / dt, "unit": UNIT, "cores": ncpu,
                                            "sample": f"all {n_weights} weights of {wl.name}, {ncpu} threads over slabs of output channels"}
        out["parity"] = {"channels": ch, "mismatches": bad[0], "e2e_mismatches": bad[1],
                         "what": "codes, scales, kernel_err, channel_err of every output channel of the timed runs against the CPU checker"}
    print(json.dumps(out))
    D.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=8.0, help="seconds of single-thread checker time for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
