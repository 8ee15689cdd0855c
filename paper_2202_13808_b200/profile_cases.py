"""Run one entry point on one named workload a few times, for use under a profiler.

  python -m paper_2202_13808_b200.profile_cases compress vitb_fc2 --reps 3
  python -m paper_2202_13808_b200.profile_cases weight_grad vitb_fc1 --reps 3
  python -m paper_2202_13808_b200.profile_cases conv_weight_grad r50_conv3x3 --reps 2

Prints the CUDA-event time of every repetition (L2 is flushed between repetitions); with --queued, the mean
time of back-to-back calls over three rotating input sets and the algorithmic rate.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import dropit_inputs as di  # noqa: E402
import paper_2202_13808_b200 as dropit  # noqa: E402

CASES = {c.name: c for c in (di.SINGLE_LINEAR_F32, di.VITB_FC1, di.VITB_FC2, di.R50_CONV1X1, di.R50_CONV3X3,
                             di.VITDET_QKV, di.VITDET_FC1, di.VITDET_FC2)}


def _algorithmic(case, op):
    """(bytes, flops) the call moves / computes by the method's definition (Sec. 3.2, Eq. 4-6)."""
    n = case.n
    es = 2 if case.dtype == "bf16" else 4
    k = dropit.dropit_keep_count(n, case.gamma)
    if op == "compress_random":   # ranks written once and read twice (2 bytes each), retained x gathered, outputs
        return 3 * n * 2 + n / 8 + 2 * k * es + 4 * ((n + 127) // 128), 0.0
    if op == "compress":
        passes = 2 if es == 2 else 3
        return passes * n * es + n / 8 + k * es + 4 * ((n + 127) // 128), 0.0
    if op == "decompress":
        return n * es + n / 8 + k * es + 4 * ((n + 127) // 128), 0.0
    if isinstance(case, di.LinearCase):
        return 0.0, 2.0 * case.M * case.Ca * case.Cz
    return 0.0, 2.0 * case.B * case.Ho * case.Wo * case.Cz * case.Ca * case.R * case.S


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["compress", "compress_random", "decompress", "weight_grad", "conv_weight_grad"])
    ap.add_argument("case", choices=sorted(CASES))
    ap.add_argument("--gamma", type=float, default=None)
    ap.add_argument("--format", default="bitmask", choices=["bitmask", "index32"])
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--queued", action="store_true",
                    help="time all repetitions as one region over 3 rotating input sets (no host sync between "
                         "calls), the way a training step issues them; default: one flushed, synchronised call per line")
    args = ap.parse_args()
    case = CASES[args.case]
    if args.gamma is not None:
        case = di.with_gamma(case, args.gamma)
    gamma = case.gamma
    dev = torch.device("cuda:0")
    need_dy = args.op in ("weight_grad", "conv_weight_grad")
    nsets = 3 if args.queued else 1
    xs = [di.make_x(case, b).to(dev) for b in range(nsets)]
    dys = [di.make_dy(case, b).to(dev) for b in range(nsets)] if need_dy else None
    caches = [dropit.dropit_compress(x, gamma, args.format) for x in xs]

    def call(i):
        b = i % nsets
        if args.op == "compress":
            caches[b] = dropit.dropit_compress(xs[b], gamma, args.format)
        elif args.op == "compress_random":
            caches[b] = dropit.dropit_compress_random(xs[b], gamma, i, args.format)
        elif args.op == "decompress":
            dropit.dropit_decompress(caches[b])
        elif args.op == "weight_grad":
            dropit.dropit_weight_grad(dys[b], caches[b])
        else:
            dropit.dropit_conv_weight_grad(dys[b], caches[b], (case.R, case.S), case.stride, case.pad)

    if args.queued:
        for i in range(3):
            call(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.reps):
            call(i)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / args.reps * 1e3
        by, fl = _algorithmic(case, args.op)
        rate = "%.0f GB/s algorithmic" % (by / us / 1e3) if by else "%.0f TFLOP/s" % (fl / us / 1e6)
        print("%s %s gamma=%g %s: %.1f us per call over %d queued calls, %s"
              % (args.op, case.name, gamma, args.format, us, args.reps, rate))
    else:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        for r in range(args.reps):
            flush.zero_()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            call(r)
            e1.record()
            torch.cuda.synchronize()
            print("%s %s gamma=%g rep %d: %.4f ms" % (args.op, case.name, gamma, r, e0.elapsed_time(e1)))
    dropit.check_device_status(dev)


if __name__ == "__main__":
    main()
