#!/usr/bin/env python
"""Benchmark of the spherical neighborhood attention hot path on B200.

A step is one forward pass (out + lse) followed by one backward pass (dq, dk, dv) over one batch of seeded
synthetic fields, through the C ABI.  The default workload is the headline configuration "c3"
(k/v on an equiangular 256x512 grid, q/out on 128x256, B=2, H=8, C=32, theta_cutoff = 3*pi/127).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl reference]

Prints ONE JSON line on rank 0.  `value` is neighbor-pair-channels per second over forward+backward with all
inputs resident in HBM; `e2e` is the same metric with the host->device copy of q, k, v, dout from pinned
memory and the device->host copy of out, dq, dk, dv inside the timed region.  The path does not shard
(one GPU per problem), so with N > 1 every rank runs an independent replica ("replicas only").

`--impl reference` times the fp64 CPU oracle, as it stands, on this machine's host cores on a bounded sample
of the same workload (one batch*head slice per step).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/mma_kernels_c3_counters.md (bench.py cannot run ncu itself)
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("c3", "forward"): 816768768 + 63346432,
    ("c3", "backward_dq"): 980778752 + 66266112,
    ("c3", "backward_dkdv"): 715740160 + 502913024,
}

METRIC = "fwd+bwd neighbor-pair-channels per second"
UNIT = "pair*ch/s"
FP32_LANES_PER_SM = 128


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    return ap.parse_args()


def workload_config(wl, n_gpus):
    return {"workload": f"{wl.name}: {wl.description}", "grid_in": [wl.nlat_in, wl.nlon_in],
            "grid_out": [wl.nlat_out, wl.nlon_out], "B": wl.B, "H": wl.H, "C": wl.C,
            "theta_cutoff": wl.theta_cutoff, "seed": wl.seed,
            "parallelism": "single GPU" if n_gpus == 1 else f"{n_gpus} independent replicas",
            "l2": "inputs larger than L2 (q+k+v+dout > 126 MB); no flush between iterations"}


# ---------------------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the oracle on host cores
# ---------------------------------------------------------------------------------------------------------

def oracle_sample_step(orc, g, wl, q, k, v, dout, n_slices):
    """Forward + backward of the oracle on the first n_slices batch*head slices; returns seconds."""
    N = wl.N
    sl = lambda a, nlat, nlon: a.reshape(N, nlat, nlon, wl.C)[:n_slices]
    qs, ds = sl(q, wl.nlat_out, wl.nlon_out), sl(dout, wl.nlat_out, wl.nlon_out)
    ks, vs = sl(k, wl.nlat_in, wl.nlon_in), sl(v, wl.nlat_in, wl.nlon_in)
    t0 = time.perf_counter()
    orc.forward(g, qs, ks, vs)
    orc.backward(g, qs, ks, vs, ds)
    return time.perf_counter() - t0


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import sna_oracle as orc
    from paper_2505_11157_b200.synthetic import make_inputs
    g = orc.geometry(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)
    q, k, v, dout = make_inputs(wl)
    n_slices = min(wl.N, 2)
    units = g.nnz * wl.nlon_out * n_slices * wl.C
    for _ in range(args.warmup):
        oracle_sample_step(orc, g, wl, q, k, v, dout, n_slices)
    t = sum(oracle_sample_step(orc, g, wl, q, k, v, dout, n_slices) for _ in range(args.steps))
    value = units * args.steps / t
    sample = (f"{n_slices} of {wl.N} batch*head slices per step (fp64, forward+backward; the forward runs on all threads, "
              "the backward scatter on one thread per slice)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(wl, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)
        sm, smax, reasons = [], None, set()
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax = float(f[1])
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------------------

def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def run_ours(args, wl):
    import torch
    from paper_2505_11157_b200 import sna            # raises if the CUDA library is missing: no fallback
    from paper_2505_11157_b200.synthetic import make_inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    B, H, C = wl.B, wl.H, wl.C
    plan = sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)
    pairs = plan.nnz * wl.nlon_out * wl.N
    units = pairs * C                                   # neighbor-pair-channels per step (forward and backward)
    host = [torch.from_numpy(a).pin_memory() for a in make_inputs(wl)]
    q, k, v, dout = [h.cuda(non_blocking=True) for h in host]
    out, dq = torch.empty_like(q), torch.empty_like(q)
    dk, dv = torch.empty_like(k), torch.empty_like(k)
    lse = torch.empty(q.shape[:-1], dtype=torch.float32, device="cuda")
    Dst = torch.empty_like(lse)
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in (out, dq, dk, dv)]
    stream = torch.cuda.current_stream()

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(marks=None):
        sna.sna_forward_ex(plan.handle, q, k, v, out, lse, B, H, C, stream)
        if marks is not None:
            marks[1].record(stream)
        sna.sna_backward_dq(plan.handle, q, k, v, dout, out, lse, dq, Dst, B, H, C, stream)
        if marks is not None:
            marks[2].record(stream)
        sna.sna_backward_dkdv(plan.handle, q, k, v, dout, lse, Dst, dk, dv, B, H, C, stream)
    launches_per_step = sna.sna_forward_kernel_count(plan.handle, C, True) + 2   # forward (dense + band, or one) + dq + dk/dv

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- device-resident timing, K steps, per-kernel events inside the timed region --------------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    marks = [[ev() for _ in range(4)] for _ in range(args.steps)]
    barrier()
    t_start, t_end = ev(), ev()
    t_start.record(stream)
    for i in range(args.steps):
        marks[i][0].record(stream)
        step(marks[i])
        marks[i][3].record(stream)
    t_end.record(stream)
    barrier()
    ms_total = t_start.elapsed_time(t_end)
    ms_fwd = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    ms_dq = statistics.mean(m[1].elapsed_time(m[2]) for m in marks)
    ms_dkdv = statistics.mean(m[2].elapsed_time(m[3]) for m in marks)

    # ---- end to end: pinned host -> device, compute, device -> pinned host ------------------------------
    def e2e_step():
        for d, h in zip((q, k, v, dout), host):
            d.copy_(h, non_blocking=True)
        step()
        for h, d in zip(host_out, (out, dq, dk, dv)):
            h.copy_(d, non_blocking=True)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_step()
    barrier()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None   # sampled over the device-resident and the end-to-end timed regions
    h2d = sum(h.numel() * 4 for h in host)
    d2h = sum(h.numel() * 4 for h in host_out)

    ms_total_max, ms_e2e_step_max = max_over_ranks([ms_total, ms_e2e / e2e_steps], dist, "cuda")

    if rank == 0:
        props = torch.cuda.get_device_properties(local_rank)
        sm_max_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        peak_tflops = props.multi_processor_count * FP32_LANES_PER_SM * 2 * sm_max_mhz * 1e6 / 1e12
        # algorithmic flops per pair*channel credited to each kernel: forward 4 (s and p.v), dq kernel 6 (s, t, dq),
        # dk/dv kernel 4 (dk, dv; its recomputation of s and t is not credited) -- 14 in total = 4 forward + 10 backward
        kernels = {"forward": (ms_fwd, 4.0), "backward_dq": (ms_dq, 6.0), "backward_dkdv": (ms_dkdv, 4.0)}
        dominant = max(kernels, key=lambda n: kernels[n][0])
        dom_ms, dom_flops_per_unit = kernels[dominant]
        achieved = dom_flops_per_unit * units / (dom_ms * 1e-3) / 1e12
        traffic = NCU_DRAM_BYTES_PER_LAUNCH.get((wl.name, dominant))
        peak_measured = sna.sna_measure_fp32_fma_peak()   # pure-FMA loop on this device, TFLOP/s
        ms_step = ms_total_max / args.steps
        roof_fwd_ms = 4.0 * units / (peak_tflops * 1e12) * 1e3
        roof_bwd_ms = 10.0 * units / (peak_tflops * 1e12) * 1e3
        result = {
            "metric": METRIC, "value": world * units / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, world),
            "ms_forward": ms_fwd, "ms_backward": ms_dq + ms_dkdv, "ms_backward_dq": ms_dq, "ms_backward_dkdv": ms_dkdv,
            "pairs_per_step": pairs,
            "roofline_step": {"bound": "alu", "roofline_ms": roof_fwd_ms + roof_bwd_ms, "frac": (roof_fwd_ms + roof_bwd_ms) / ms_step,
                              "peak_derived_tflops": peak_tflops, "peak_fma_measured_tflops": peak_measured,
                              "frac_of_measured_peak": (roof_fwd_ms + roof_bwd_ms) * (peak_tflops / peak_measured) / ms_step,
                              "note": "algorithmic flops (4C fwd + 10C bwd per pair) at the FP32 FMA peak of measured-max clock"},
            "roofline": {"bound": "alu", "kernel": dominant, "achieved": achieved, "peak": peak_tflops, "unit": "TFLOP/s",
                         "frac": achieved / peak_tflops, "traffic": traffic,
                         "note": f"{dom_flops_per_unit:g} flops per pair*channel credited; peak = SMs x 128 FP32 lanes x 2 x max SM clock "
                                 "(of derived peak; a pure-FMA loop measured 127.7 of 128 FMA/clk/SM); contractions run on tensor cores "
                                 "as 3xTF32 MMAs; traffic = ncu dram bytes read+written per launch (profiles/)"},
            "e2e": {"value": world * units / (ms_e2e_step_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e_step_max},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            from oracle import sna_oracle as orc
            g = orc.geometry(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)
            n_slices = min(wl.N, 4)
            arrays = [h.numpy() for h in host]
            t = oracle_sample_step(orc, g, wl, *arrays, n_slices)
            result["cpu_baseline"] = {"value": g.nnz * wl.nlon_out * n_slices * C / t, "unit": UNIT, "cores": orc.num_threads(),
                                      "kind": "oracle", "seconds": t,
                                      "sample": f"{n_slices} of {wl.N} batch*head slices, forward+backward, fp64"}
        print(json.dumps(result))
    plan.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2505_11157_b200.synthetic import WORKLOADS
    wl = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
