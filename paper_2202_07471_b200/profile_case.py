"""A small, self-terminating case of the large-layer workload for profilers.

  python -m paper_2202_07471_b200.profile_case [--channels M] [--launches L] [--mode 7]
  python -m paper_2202_07471_b200.profile_case --workload resnet50 [--launches L]

Quantizes one [M, 2048, 3, 3] layer (default M = 4096: 302 MB of weights, larger than L2, a few
hundred MB on the device) L times through the C ABI.  Values follow the large-layer recipe
(seeded normal weights with a per-channel log-uniform scale).  With --workload NAME the whole
model of that name (resnet18, resnet50, mobilenetv2, mixed_kernels) is quantized in one call instead.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as sq
from . import workloads as W


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--channels", type=int, default=4096)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--mode", type=int, default=sq.MODE_EKC)
    ap.add_argument("--workload", default="large_layer")
    args = ap.parse_args()
    if args.workload != "large_layer":
        wl = W.WORKLOADS[args.workload]
        ws = [torch.from_numpy(W.layer_weights(wl, i, seed=0, threads=8)).cuda() for i in range(len(wl.shapes))]
        call = sq.ModelCall([sq.alloc_outputs(w) for w in ws], bits=args.bits, mode=args.mode)
        for _ in range(args.launches):
            call.run()
        sq.squant_device_status()
        print(f"ok: {args.launches} launches of {args.workload}, {sum(w.numel() for w in ws)} weights each")
        return
    wl = W.WORKLOADS["large_layer"]
    m = min(args.channels, 2048)
    reps = (args.channels + m - 1) // m
    parts = [W.layer_weights(wl, i % len(wl.shapes), seed=0, channels=slice(0, m), threads=8) for i in range(reps)]
    w = torch.from_numpy(np.concatenate(parts)[:args.channels]).cuda()
    bufs = sq.alloc_outputs(w)
    call = sq.ModelCall([bufs], bits=args.bits, mode=args.mode)
    for _ in range(args.launches):
        call.run()
    sq.squant_device_status()
    print(f"ok: {args.launches} launches of [{args.channels}, 2048, 3, 3], {w.numel()} weights each")


if __name__ == "__main__":
    main()
