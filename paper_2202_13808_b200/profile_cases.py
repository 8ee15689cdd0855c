"""Run one entry point on one named workload a few times, for use under a profiler.

  python -m paper_2202_13808_b200.profile_cases compress vitb_fc2 --reps 3
  python -m paper_2202_13808_b200.profile_cases weight_grad vitb_fc1 --reps 3
  python -m paper_2202_13808_b200.profile_cases conv_weight_grad r50_conv3x3 --reps 2

Prints the CUDA-event time of every repetition (L2 is flushed between repetitions).
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["compress", "decompress", "weight_grad", "conv_weight_grad"])
    ap.add_argument("case", choices=sorted(CASES))
    ap.add_argument("--gamma", type=float, default=None)
    ap.add_argument("--format", default="bitmask", choices=["bitmask", "index32"])
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    case = CASES[args.case]
    gamma = case.gamma if args.gamma is None else args.gamma
    dev = torch.device("cuda:0")
    x = di.make_x(case).to(dev)
    dy = di.make_dy(case).to(dev) if args.op in ("weight_grad", "conv_weight_grad") else None
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    cache = dropit.dropit_compress(x, gamma, args.format)
    for r in range(args.reps):
        flush.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if args.op == "compress":
            cache = dropit.dropit_compress(x, gamma, args.format)
        elif args.op == "decompress":
            dropit.dropit_decompress(cache)
        elif args.op == "weight_grad":
            dropit.dropit_weight_grad(dy, cache)
        else:
            dropit.dropit_conv_weight_grad(dy, cache, (case.R, case.S), case.stride, case.pad)
        e1.record()
        torch.cuda.synchronize()
        print("%s %s gamma=%g rep %d: %.4f ms" % (args.op, case.name, gamma, r, e0.elapsed_time(e1)))
    dropit.check_device_status(dev)


if __name__ == "__main__":
    main()
