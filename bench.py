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

# Recorded constants: dram__bytes_read.sum + dram__bytes_write.sum per stage (its dense kernel + its band kernel) from an
# ncu capture on workload c3 (bench.py cannot run ncu itself; the value is reported as `roofline.traffic` for that
# workload only).
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("c3", "forward"): (44455936 + 725248) + (790744576 + 63745024),
    ("c3", "backward_dq"): (57742592 + 2146560) + (956322304 + 63501312),
    ("c3", "backward_dkdv"): (49276928 + 6318592) + (760281856 + 504061184),
}
HBM_GBS_FALLBACK = 6650.0          # used only if MEASURED_PEAKS.json is absent
L2_BYTES = 126 * 1024 * 1024

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
    ap.add_argument("--no-extras", action="store_true", help="skip the other configurations and the reduced-precision variant")
    return ap.parse_args()


def input_bytes(wl):
    """Bytes of q, k, v, dout (the tensors a step reads)."""
    return 4 * wl.C * wl.N * (2 * wl.nlat_out * wl.nlon_out + 2 * wl.nlat_in * wl.nlon_in)


def l2_policy(wl):
    if input_bytes(wl) > L2_BYTES:
        return f"inputs larger than L2 (q+k+v+dout = {input_bytes(wl) / 1e6:.0f} MB > 126 MB); no flush between iterations"
    return (f"inputs smaller than L2 (q+k+v+dout = {input_bytes(wl) / 1e6:.1f} MB): a 256 MB buffer is overwritten before every "
            "timed step (outside the timed events) to flush L2")


def workload_config(wl, n_gpus):
    return {"workload": f"{wl.name}: {wl.description}", "grid_in": [wl.nlat_in, wl.nlon_in],
            "grid_out": [wl.nlat_out, wl.nlon_out], "B": wl.B, "H": wl.H, "C": wl.C,
            "theta_cutoff": wl.theta_cutoff, "seed": wl.seed,
            "parallelism": "single GPU" if n_gpus == 1 else f"{n_gpus} independent replicas",
            "l2": l2_policy(wl)}


def hbm_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return HBM_GBS_FALLBACK, "fallback"


def kernel_rooflines(wl, units, peak_tflops):
    """Per kernel: credited flops, compulsory bytes, and the slower of the two times (ms) with its bound."""
    hbm, _ = hbm_peak_gbs()
    o = 4 * wl.C * wl.N * wl.nlat_out * wl.nlon_out      # bytes of one out-grid tensor
    i = 4 * wl.C * wl.N * wl.nlat_in * wl.nlon_in        # bytes of one in-grid tensor
    spec = {"forward": (4.0, 2 * o + 2 * i),             # q, out; k, v
            "backward_dq": (6.0, 4 * o + 2 * i),         # q, dout, out, dq; k, v
            "backward_dkdv": (4.0, 2 * o + 4 * i)}       # q, dout; k, v, dk, dv
    res = {}
    for name, (flops_per_unit, nbytes) in spec.items():
        t_alu = flops_per_unit * units / (peak_tflops * 1e12) * 1e3
        t_hbm = nbytes / (hbm * 1e9) * 1e3
        res[name] = {"flops_per_unit": flops_per_unit, "bytes": nbytes, "t_alu_ms": t_alu, "t_hbm_ms": t_hbm,
                     "bound": "alu" if t_alu >= t_hbm else "hbm", "roofline_ms": max(t_alu, t_hbm)}
    return res


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


class Problem:
    """Device tensors and the plan of one workload, plus one step (forward, dq, dk/dv) through the C ABI."""

    def __init__(self, sna, torch, wl, keep_host=False, global_plan=False):
        from paper_2505_11157_b200.synthetic import make_inputs
        self.sna, self.torch, self.wl = sna, torch, wl
        self.plan = sna.Plan(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff,
                             global_attention=global_plan)
        self.pairs = self.plan.nnz * wl.nlon_out * wl.N
        self.units = self.pairs * wl.C                  # neighbor-pair-channels per step (forward and backward)
        host = [torch.from_numpy(a) for a in make_inputs(wl)]
        self.host = [h.pin_memory() for h in host] if keep_host else host
        self.q, self.k, self.v, self.dout = [h.cuda(non_blocking=True) for h in self.host]
        self.out, self.dq = torch.empty_like(self.q), torch.empty_like(self.q)
        self.dk, self.dv = torch.empty_like(self.k), torch.empty_like(self.k)
        self.lse = torch.empty(self.q.shape[:-1], dtype=torch.float32, device="cuda")
        self.D = torch.empty_like(self.lse)
        self.ws = torch.empty(self.plan.workspace_bytes(wl.B, wl.H, wl.C), dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream()
        if not keep_host:
            self.host = None

    def step(self, marks=None):
        s, wl, h = self.sna, self.wl, self.plan.handle
        s.sna_forward_ex(h, self.q, self.k, self.v, self.out, self.lse, wl.B, wl.H, wl.C, self.stream)
        if marks is not None:
            marks[1].record(self.stream)
        s.sna_backward_dq(h, self.q, self.k, self.v, self.dout, self.out, self.lse, self.dq, self.D, wl.B, wl.H, wl.C, self.stream)
        if marks is not None:
            marks[2].record(self.stream)
        s.sna_backward_dkdv(h, self.q, self.k, self.v, self.dout, self.lse, self.D, self.dk, self.dv, wl.B, wl.H, wl.C, self.stream)

    def step_tf32(self, marks=None):
        s, wl, h = self.sna, self.wl, self.plan.handle
        s.sna_forward_tf32(h, self.q, self.k, self.v, self.out, self.lse, wl.B, wl.H, wl.C, self.stream)
        if marks is not None:
            marks[1].record(self.stream)
            marks[2].record(self.stream)
        s.sna_backward_tf32(h, self.q, self.k, self.v, self.dout, self.out, self.lse, self.dq, self.dk, self.dv, self.ws,
                            self.ws.numel(), wl.B, wl.H, wl.C, self.stream)

    def launches_per_step(self):
        return self.sna.sna_forward_kernel_count(self.plan.handle, self.wl.C, True) + 2   # forward (dense + band, or one) + dq + dk/dv

    def close(self):
        self.plan.close()


def time_steps(torch, prob, steps, warmup, step_fn=None, flush=None):
    """Mean per-kernel and per-step times (ms) over `steps` steps, CUDA events on the launching stream.  With `flush`
    (a device buffer larger than L2) the buffer is overwritten before every step, outside the timed events."""
    step_fn = step_fn or prob.step
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(warmup):
        step_fn()
    torch.cuda.synchronize()
    marks = [[ev() for _ in range(4)] for _ in range(steps)]
    for i in range(steps):
        if flush is not None:
            flush.add_(1.0)
        marks[i][0].record(prob.stream)
        step_fn(marks[i])
        marks[i][3].record(prob.stream)
    torch.cuda.synchronize()
    mean = statistics.mean
    return {"ms_forward": mean(m[0].elapsed_time(m[1]) for m in marks), "ms_backward_dq": mean(m[1].elapsed_time(m[2]) for m in marks),
            "ms_backward_dkdv": mean(m[2].elapsed_time(m[3]) for m in marks), "ms_per_step": mean(m[0].elapsed_time(m[3]) for m in marks)}


def accuracy_against_oracle(orc, g, prob, n_slices):
    """Errors of the GPU results of the first n_slices batch*head slices against the oracle: the gated measure
    max|x-o| / max|o| per tensor, the element-wise relative error with denominator max(|o|, 1e-3 max|o|), and the
    per-point relative error ||x_i - o_i|| / max(||o_i||, 1e-3 max_i ||o_i||) over the channel vectors."""
    wl = prob.wl
    arrays = [h.numpy() for h in prob.host]
    sl = lambda a, nlat, nlon: a.reshape(wl.N, nlat, nlon, wl.C)[:n_slices]
    qs, ds = sl(arrays[0], wl.nlat_out, wl.nlon_out), sl(arrays[3], wl.nlat_out, wl.nlon_out)
    ks, vs = sl(arrays[1], wl.nlat_in, wl.nlon_in), sl(arrays[2], wl.nlat_in, wl.nlon_in)
    t0 = time.perf_counter()
    ref_out = orc.forward(g, qs, ks, vs)
    refs = (ref_out,) + tuple(orc.backward(g, qs, ks, vs, ds))
    seconds = time.perf_counter() - t0
    got = (prob.out, prob.dq, prob.dk, prob.dv)
    acc = {}
    for name, x, r in zip(("out", "dq", "dk", "dv"), got, refs):
        x = x.reshape((wl.N,) + r.shape[1:])[:n_slices].cpu().numpy().astype(np.float64)
        scale = np.max(np.abs(r))
        norms = np.linalg.norm(r, axis=-1)
        acc[name] = {"normalised_max_error": float(np.max(np.abs(x - r)) / scale),
                     "floor_relative_max_error": float(np.max(np.abs(x - r) / np.maximum(np.abs(r), 1e-3 * scale))),
                     "per_point_relative_max_error": float(np.max(np.linalg.norm(x - r, axis=-1) / np.maximum(norms, 1e-3 * norms.max())))}
    return seconds, acc


def run_ours(args, wl):
    import torch
    from paper_2505_11157_b200 import sna            # raises if the CUDA library is missing: no fallback
    from paper_2505_11157_b200.synthetic import WORKLOADS

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

    C = wl.C
    prob = Problem(sna, torch, wl, keep_host=True)
    units, pairs = prob.units, prob.pairs
    q, k, v, dout, out, dq, dk, dv = prob.q, prob.k, prob.v, prob.dout, prob.out, prob.dq, prob.dk, prob.dv
    host = prob.host
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in (out, dq, dk, dv)]
    stream = prob.stream
    step = prob.step
    flush = None if input_bytes(wl) > L2_BYTES else torch.zeros(64 * 1024 * 1024, dtype=torch.float32, device="cuda")
    launches_per_step = prob.launches_per_step()
    ev = lambda: torch.cuda.Event(enable_timing=True)

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
        if flush is not None:
            flush.add_(1.0)
        marks[i][0].record(stream)
        step(marks[i])
        marks[i][3].record(stream)
    t_end.record(stream)
    barrier()
    ms_fwd = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    ms_dq = statistics.mean(m[1].elapsed_time(m[2]) for m in marks)
    ms_dkdv = statistics.mean(m[2].elapsed_time(m[3]) for m in marks)
    # with an L2 flush between steps the flush itself is outside the per-step events; without one the K steps run back to back
    ms_total = t_start.elapsed_time(t_end) if flush is None else sum(m[0].elapsed_time(m[3]) for m in marks)

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
        peak_measured = sna.sna_measure_fp32_fma_peak()   # pure-FMA loop on this device, TFLOP/s
        hbm_gbs, hbm_source = hbm_peak_gbs()
        # algorithmic flops per pair*channel credited to each kernel: forward 4 (s and p.v), dq kernel 6 (s, t, dq),
        # dk/dv kernel 4 (dk, dv; its recomputation of s and t is not credited) -- 14 in total = 4 forward + 10 backward.
        # Every kernel's roofline time is the slower of those flops at the FP32 FMA peak and its compulsory bytes at the
        # measured HBM copy bandwidth.
        roofs = kernel_rooflines(wl, units, peak_tflops)
        times = {"forward": ms_fwd, "backward_dq": ms_dq, "backward_dkdv": ms_dkdv}
        dominant = max(times, key=times.get)
        dom = roofs[dominant]
        if dom["bound"] == "alu":
            achieved, peak, unit = dom["flops_per_unit"] * units / (times[dominant] * 1e-3) / 1e12, peak_tflops, "TFLOP/s"
            peak_note = (f"peak = SMs x 128 FP32 lanes x 2 x max SM clock (derived; the pure-FMA probe measured "
                         f"{peak_measured:.1f} TFLOP/s on this device)")
        else:
            achieved, peak, unit = dom["bytes"] / (times[dominant] * 1e-3) / 1e9, hbm_gbs, "GB/s"
            peak_note = f"peak = copy bandwidth ({hbm_source})"
        ms_step = ms_total_max / args.steps
        roof_ms = sum(r["roofline_ms"] for r in roofs.values())
        result = {
            "metric": METRIC, "value": world * units / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, world),
            "ms_forward": ms_fwd, "ms_backward": ms_dq + ms_dkdv, "ms_backward_dq": ms_dq, "ms_backward_dkdv": ms_dkdv,
            "pairs_per_step": pairs,
            "roofline_step": {"bound": "alu" if all(r["bound"] == "alu" for r in roofs.values()) else "mixed",
                              "roofline_ms": roof_ms, "frac": roof_ms / ms_step,
                              "peak_derived_tflops": peak_tflops, "peak_fma_measured_tflops": peak_measured,
                              "frac_of_measured_peak": roof_ms * (peak_tflops / peak_measured) / ms_step,
                              "hbm_gbs": hbm_gbs, "hbm_source": hbm_source,
                              "note": "per kernel the slower of its algorithmic flops (4C fwd + 10C bwd per pair) at the FP32 FMA "
                                      "peak and its compulsory bytes at the HBM copy bandwidth, summed over the three kernels"},
            "roofline": {"bound": dom["bound"], "kernel": dominant, "achieved": achieved, "peak": peak, "unit": unit,
                         "frac": achieved / peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((wl.name, dominant)),
                         "note": f"{dom['flops_per_unit']:g} flops per pair*channel credited, {dom['bytes'] / 1e6:.0f} MB compulsory; "
                                 f"{peak_note}; the contractions run on tensor cores (TF32 main term + stacked BF16 corrections, "
                                 "tcgen05 for whole-ring and wide windows); traffic = recorded ncu DRAM bytes read+written per "
                                 "stage (dense + band kernel), null when this workload has no capture"},
            "e2e": {"value": world * units / (ms_e2e_step_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e_step_max},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
        }
        if world == 1 and not args.no_extras:
            # reduced-precision variant on the same workload, and the other benchmark configurations (10 steps each)
            step_prec = prob.step       # restore the fp32 results afterwards for the accuracy check
            t = time_steps(torch, prob, 10, 3, prob.step_tf32, flush)
            result["variants"] = {"tf32": {"ms_forward": t["ms_forward"], "ms_backward": t["ms_backward_dkdv"],
                                           "ms_per_step": t["ms_per_step"], "frac": roof_ms / t["ms_per_step"],
                                           "note": "sna_forward_tf32 + sna_backward_tf32: one TF32 product per contraction, "
                                                   "tolerance 5e-3 instead of 1e-5 / 1e-4; not the headline"}}
            # channels-first entry points on the same workload: the layout changes (HBM-bound transposes) run inside the calls
            cf = lambda x: x.permute(0, 1, 4, 2, 3).reshape(x.shape[0], -1, x.shape[2], x.shape[3]).contiguous()
            cf_in = [cf(x) for x in (prob.q, prob.k, prob.v, prob.dout)]
            cf_out = [torch.empty_like(cf_in[0]), torch.empty_like(cf_in[0]), torch.empty_like(cf_in[1]), torch.empty_like(cf_in[1])]
            state = torch.empty(sna.sna_cf_state_bytes(prob.plan.handle, wl.B, wl.H, C), dtype=torch.uint8, device="cuda")
            scratch = torch.empty(sna.sna_cf_scratch_bytes(prob.plan.handle, wl.B, wl.H, C), dtype=torch.uint8, device="cuda")

            def step_cf(marks=None):
                sna.sna_forward_cf(prob.plan.handle, cf_in[0], cf_in[1], cf_in[2], cf_out[0], state, state.numel(), wl.B, wl.H, C, prob.stream)
                if marks is not None:
                    marks[1].record(prob.stream)
                    marks[2].record(prob.stream)
                sna.sna_backward_cf(prob.plan.handle, cf_in[3], state, state.numel(), scratch, scratch.numel(), cf_out[1], cf_out[2],
                                    cf_out[3], wl.B, wl.H, C, prob.stream)

            t = time_steps(torch, prob, 10, 3, step_cf, flush)
            moved = 2 * 4 * sum(x.numel() for x in cf_in + cf_out)
            result["variants"]["channels_first"] = {
                "ms_forward": t["ms_forward"], "ms_backward": t["ms_backward_dkdv"], "ms_per_step": t["ms_per_step"],
                "layout_bytes_per_step": moved, "layout_ms_at_hbm_peak": moved / (hbm_gbs * 1e6),
                "note": "sna_forward_cf + sna_backward_cf on [B, H*C, nlat, nlon] tensors: eight tiled transposes per step around "
                        "the same kernels (each element read once and written once)"}
            del cf_in, cf_out, state, scratch
            torch.cuda.empty_cache()
            step_prec()
            torch.cuda.synchronize()
            result["workloads"] = {wl.name: {"ms_forward": ms_fwd, "ms_backward_dq": ms_dq, "ms_backward_dkdv": ms_dkdv,
                                             "ms_per_step": ms_step, "roofline_ms": roof_ms, "roofline_frac": roof_ms / ms_step,
                                             "l2": l2_policy(wl)}}
            big_flush = torch.zeros(64 * 1024 * 1024, dtype=torch.float32, device="cuda")
            for name in sorted(WORKLOADS):
                if name == wl.name:
                    continue
                other = WORKLOADS[name]
                po = Problem(sna, torch, other)
                t = time_steps(torch, po, 10, 3, None, None if input_bytes(other) > L2_BYTES else big_flush)
                r_ms = sum(r["roofline_ms"] for r in kernel_rooflines(other, po.units, peak_tflops).values())
                t.update({"roofline_ms": r_ms, "roofline_frac": r_ms / t["ms_per_step"], "l2": l2_policy(other)})
                result["workloads"][name] = t
                po.close()
                del po
                torch.cuda.empty_cache()
            # the global limit once more through the plan that never builds per-pair structure (dense kernels only)
            c5 = WORKLOADS["c5"]
            pg = Problem(sna, torch, c5, global_plan=True)
            t = time_steps(torch, pg, 10, 3, None, big_flush)
            r_ms = sum(r["roofline_ms"] for r in kernel_rooflines(c5, pg.units, peak_tflops).values())
            t.update({"roofline_ms": r_ms, "roofline_frac": r_ms / t["ms_per_step"], "l2": l2_policy(c5),
                      "note": "c5 through sna_plan_create_global"})
            result["workloads"]["c5_global_plan"] = t
            pg.close()
            del pg
            torch.cuda.empty_cache()
        if not args.no_cpu_baseline and world == 1:
            from oracle import sna_oracle as orc
            g = orc.geometry(wl.nlat_in, wl.nlon_in, wl.nlat_out, wl.nlon_out, wl.grid_in, wl.grid_out, wl.theta_cutoff)
            n_slices = min(wl.N, 4)
            seconds, acc = accuracy_against_oracle(orc, g, prob, n_slices)
            result["cpu_baseline"] = {"value": g.nnz * wl.nlon_out * n_slices * C / seconds, "unit": UNIT, "cores": orc.num_threads(),
                                      "kind": "oracle", "seconds": seconds,
                                      "sample": f"{n_slices} of {wl.N} batch*head slices, forward+backward, fp64"}
            result["accuracy"] = {"slices": n_slices, "gate": "normalised_max_error <= 1e-5 (out), 1e-4 (dq, dk, dv)", **acc}
        print(json.dumps(result))
    prob.close()
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
