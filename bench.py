#!/usr/bin/env python
"""Benchmark of the DropIT layer path on B200.

A step is one pass of the whole path over one synthetic ViT-B/16 MLP batch (64 images x 197
tokens, gamma = 0.9): min-k compression of the fc1 and fc2 inputs, then both weight gradients
from the compressed caches.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; the path has no exchange step,
so ranks are independent replicas (weak scaling) and NCCL only carries the barrier and the
max-over-ranks of the device time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import dropit_inputs as di  # noqa: E402

BATCH_IMAGES = 64
LAYERS = (di.VITB_FC1, di.VITB_FC2)
WORKLOAD = "vitb16_mlp_fc1_fc2_batch64_gamma0.9"
METRIC = "step samples/s (DropIT hot path: min-k compress + sparse-cache dW)"
N_INPUT_SETS = 3   # distinct input batches rotated between steps; one batch is 194 MB (> 126 MB of L2)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------
# clocks sampled during the timed region
# ------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.1] or [l for (_, l) in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [c.strip() for c in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# the product arm
# ------------------------------------------------------------------------------------------
def algorithmic_bytes_compress(case) -> float:
    """Radix select sees the tensor before and after the threshold is known: 2 reads of X, one write of
    the mask, the retained values and the seek table."""
    import paper_2202_13808_b200 as dropit
    n = case.n
    k = dropit.dropit_keep_count(n, case.gamma)
    return 2 * n * 2 + n / 8 + k * 2 + 4 * ((n + 127) // 128)


def compulsory_bytes_compress(case) -> float:
    """One read of X plus the outputs: what any method has to move."""
    return algorithmic_bytes_compress(case) - case.n * 2


def dense_flops(case) -> float:
    return 2.0 * case.M * case.Ca * case.Cz


def max_over_ranks(ms: float, world: int, device) -> float:
    """A multi-rank time is the slowest rank's device time."""
    if world > 1:
        t = torch.tensor([ms], device=device)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        ms = float(t.item())
    return ms


def whole_job_value(world: int, steps: int, ms: float) -> float:
    """Samples per second of all ranks together (every rank runs the same step on its own batch: weak scaling)."""
    return world * BATCH_IMAGES * steps / (ms / 1e3)


def run_ours(args, rank, world, device):
    import paper_2202_13808_b200 as dropit

    sets = []
    for b in range(N_INPUT_SETS):
        sets.append([(di.make_x(c, b).to(device), di.make_dy(c, b).to(device)) for c in LAYERS])
    dws = [torch.empty((c.Cz, c.Ca), dtype=torch.float32, device=device) for c in LAYERS]
    ws_c = [torch.empty(dropit.dropit_cache_sizes(c.n, c.gamma, dropit.BF16, dropit.FMT_BITMASK)[3], dtype=torch.uint8,
                        device=device) for c in LAYERS]
    ws_g = [torch.empty(dropit.dropit_weight_grad_workspace(c.M, c.Ca, c.Cz, dropit.BF16, dropit.FMT_BITMASK),
                        dtype=torch.uint8, device=device) for c in LAYERS]
    stream = torch.cuda.current_stream(device)

    def step(i, ev=None):
        batch = sets[i % N_INPUT_SETS]
        for li, c in enumerate(LAYERS):
            x, dy = batch[li]
            if ev is not None:
                ev[li][0].record(stream)
            cache = dropit.dropit_compress(x, c.gamma, "bitmask", workspace=ws_c[li])
            if ev is not None:
                ev[li][1].record(stream)
            dropit.dropit_weight_grad(dy, cache, out=dws[li], workspace=ws_g[li])
            if ev is not None:
                ev[li][2].record(stream)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize(device)
    dropit.check_device_status(device)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(device)

    # per-call events: [layer][0..2] per step
    evs = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in LAYERS] for _ in range(args.steps)]
    sampler = ClockSampler(device.index or 0)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    launches0 = dropit.dropit_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i, evs[i])
    e1.record(stream)
    barrier()
    t1 = time.time()
    launches = dropit.dropit_launch_count() - launches0
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    dropit.check_device_status(device)
    ms = max_over_ranks(e0.elapsed_time(e1), world, device)

    comp_ms = [statistics.mean(evs[i][li][0].elapsed_time(evs[i][li][1]) for i in range(args.steps)) for li in range(2)]
    dw_ms = [statistics.mean(evs[i][li][1].elapsed_time(evs[i][li][2]) for i in range(args.steps)) for li in range(2)]

    # ---- the decompress launch of a dW call on its own (same caches, rotating), to split the call's time ----
    caches = [[dropit.dropit_compress(sets[b][li][0], c.gamma, "bitmask", workspace=ws_c[li]) for li, c in enumerate(LAYERS)]
              for b in range(N_INPUT_SETS)]
    dense = [torch.empty(c.n, dtype=torch.bfloat16, device=device) for c in LAYERS]
    dec_ms = []
    for li in range(len(LAYERS)):
        for i in range(6):
            dropit.dropit_decompress(caches[i % N_INPUT_SETS][li], out=dense[li])
        barrier()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 30
        d0.record(stream)
        for i in range(reps):
            dropit.dropit_decompress(caches[i % N_INPUT_SETS][li], out=dense[li])
        d1.record(stream)
        barrier()
        dec_ms.append(d0.elapsed_time(d1) / reps)
    del caches, dense

    # ---- end to end through the public API with host buffers ----
    host_in = [(di.make_x(c, 0).pin_memory(), di.make_dy(c, 0).pin_memory()) for c in LAYERS]
    host_out = [torch.empty((c.Cz, c.Ca), dtype=torch.float32).pin_memory() for c in LAYERS]
    dev_in = [(torch.empty_like(x, device=device), torch.empty_like(dy, device=device)) for (x, dy) in host_in]
    h2d = sum(x.numel() * x.element_size() + dy.numel() * dy.element_size() for (x, dy) in host_in)
    d2h = sum(o.numel() * 4 for o in host_out)

    def e2e_step():
        for li, c in enumerate(LAYERS):
            dev_in[li][0].copy_(host_in[li][0], non_blocking=True)
            dev_in[li][1].copy_(host_in[li][1], non_blocking=True)
            cache = dropit.dropit_compress(dev_in[li][0], c.gamma, "bitmask", workspace=ws_c[li])
            dropit.dropit_weight_grad(dev_in[li][1], cache, out=dws[li], workspace=ws_g[li])
            host_out[li].copy_(dws[li], non_blocking=True)

    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        e2e_step()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    f1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(f0.elapsed_time(f1), world, device)

    if rank != 0:
        return None
    peaks = measured_peaks()
    ms_per_step = ms / args.steps
    value = whole_job_value(world, args.steps, ms)
    # dominant kernel: the fc weight-gradient GEMM (both layers have the same flop count)
    F = dense_flops(LAYERS[0])
    dw_avg_ms = statistics.mean(dw_ms)
    tfl = F / (dw_avg_ms * 1e-3) / 1e12
    comp_bytes = [algorithmic_bytes_compress(c) for c in LAYERS]
    comp_gbs = [b / (t * 1e-3) / 1e9 for b, t in zip(comp_bytes, comp_ms)]
    out = {
        "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": [c.name for c in LAYERS], "tokens": LAYERS[0].M, "gamma": 0.9,
                   "format": "bitmask", "l2": "inputs rotate over %d batches of 194 MB each (> L2)" % N_INPUT_SETS,
                   "parallelism": "replicas x%d" % world},
        "roofline": {"kernel": "dropit_weight_grad (tcgen05 GEMM incl. its decompress)", "bound": "tensor",
                     "achieved": tfl, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tfl / peaks["bf16_tflops"],
                     "traffic": NCU_TRAFFIC["wg_tc_kernel"], "traffic_note": NCU_TRAFFIC["note_dw"],
                     "peak_source": peaks["source"] + " burst", "flops_per_launch": F, "avg_ms": dw_avg_ms},
        "roofline_compress": {"kernel": "dropit_compress (histogram + compaction)", "bound": "hbm",
                              "achieved": comp_gbs[1], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": comp_gbs[1] / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC["fused_compress_kernel_fc2"],
                              "peak_source": peaks["source"], "bytes_per_call": comp_bytes[1], "avg_ms": comp_ms[1],
                              "compulsory_gbs": compulsory_bytes_compress(LAYERS[1]) / (comp_ms[1] * 1e-3) / 1e9,
                              "dram_gbs": (NCU_TRAFFIC["fused_compress_kernel_fc2"] / (comp_ms[1] * 1e-3) / 1e9
                                           if NCU_TRAFFIC["fused_compress_kernel_fc2"] else None),
                              "layer": LAYERS[1].name,
                              "other_layer": {"layer": LAYERS[0].name, "achieved": comp_gbs[0],
                                              "frac": comp_gbs[0] / peaks["hbm_gbs"], "avg_ms": comp_ms[0]}},
        "roofline_gemm_kernel": {"kernel": "wg_tc_kernel alone, estimated on fc2: the dW call minus its decompress launch, which "
                                           "was timed separately on the same caches (the two launches overlap by the GEMM's "
                                           "set-up; fc1's decompress is too short to time from the host; the launch-list "
                                           "shares under profiles/ agree with the estimate)",
                                 "bound": "tensor", "unit": "TFLOP/s", "peak": peaks["bf16_tflops"],
                                 "achieved": F / ((dw_ms[1] - dec_ms[1]) * 1e-3) / 1e12,
                                 "frac": F / ((dw_ms[1] - dec_ms[1]) * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                 "decompress_ms": {"fc1_host_bound": dec_ms[0], "fc2": dec_ms[1]}},
        "per_call_ms": {"compress_fc1": comp_ms[0], "compress_fc2": comp_ms[1], "dw_fc1": dw_ms[0], "dw_fc2": dw_ms[1]},
        "dw_tflops": {"fc1": F / (dw_ms[0] * 1e-3) / 1e12, "fc2": F / (dw_ms[1] * 1e-3) / 1e12},
        "e2e": {"value": whole_job_value(world, e2e_steps, e2e_ms), "unit": "samples/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1:
        out["cpu_baseline"] = cpu_baseline_sample()
    return out


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (weight_grad_gemm_wg_tc_kernel_vitb_fc1/fc2.txt, compress_fused_vitb_fc2.txt).  Set an entry to None
# when its kernel changes, until the counters have been taken again.
NCU_TRAFFIC = {
    "wg_tc_kernel": 0.5 * ((96.877056e6 + 4.115456e6) + (96.871424e6 + 4.160256e6)),
    "note_dw": "wg_tc_kernel alone (mean of fc1, fc2): dY 77.5 MB + dense scratch 19.4 MB read once; the decompress kernel "
               "before it moves another 32.2 MB through DRAM on fc2 (13.8 read, 18.4 written, the rest of its 77.5 MB "
               "output stays in L2 for the GEMM)",
    "fused_compress_kernel_fc2": 78.998016e6 + 3.350784e6,
}


# ------------------------------------------------------------------------------------------
# the oracle on the host cores (reported baseline; also the --impl reference arm)
# ------------------------------------------------------------------------------------------
def oracle_step(images: int, batch: int = 0) -> float:
    """One pass of the path over `images` images of the workload through the CPU oracle; seconds."""
    import oracle

    tokens = images * 197
    secs = 0.0
    for c in LAYERS:
        x = di.make_x(c, batch)[:tokens].contiguous()
        dy = di.make_dy(c, batch)[:tokens].contiguous()
        xb, dt = oracle.to_bits(x)
        dyb, _ = oracle.to_bits(dy)
        t0 = time.perf_counter()
        keep, k = oracle.min_k(xb, c.gamma, dt)
        oracle.encode_bitmask(keep)
        oracle.pack_values(xb, keep, dt)
        oracle.fc_weight_grad(dyb, xb, keep, tokens, c.Ca, c.Cz, dt)
        secs += time.perf_counter() - t0
    return secs


def cpu_baseline_sample(images: int = 48):
    import oracle

    oracle.build()
    secs = oracle_step(images)
    return {"value": images / secs, "unit": "samples/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d of %d images (%d tokens) through the oracle's min_k + encoders + fc_weight_grad for fc1 and "
                      "fc2, %.1f s" % (images, BATCH_IMAGES, images * 197, secs)}


def run_reference(args, rank):
    if rank != 0:
        return None
    import oracle

    oracle.build()
    images = 2
    for _ in range(min(args.warmup, 1)):
        oracle_step(images)
    steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for i in range(steps):
        oracle_step(images, i)
    secs = time.perf_counter() - t0
    value = images * steps / secs
    sample = "%d of %d images per step, %d steps, CPU oracle" % (images, BATCH_IMAGES, steps)
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": secs / steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        out = run_reference(args, rank)
        if out is not None:
            print(json.dumps(out), flush=True)
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)
    try:
        out = run_ours(args, rank, world, device)
        if out is not None:
            print(json.dumps(out), flush=True)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
