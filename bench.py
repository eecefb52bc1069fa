#!/usr/bin/env python
"""Benchmark of the relay-buffer-free MoE dispatch/combine path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic
routing: moe_plan -> moe_dispatch -> moe_combine (identity experts: combine
reads the dispatched windows in place).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3]
  python bench.py --impl reference ...     # the CPU oracle, timed on the host cores

Multi-GPU: the path does not shard (the R expert-parallel ranks are virtual
segments of one GPU's memory), so N > 1 runs N independent replicas, one
process per GPU, with no data-path collective; value is the sum over replicas
divided by the slowest replica's time ("weak" scaling).
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

import numpy as np
import torch

from paper_2605_06055_b200 import synth

NOMINAL_HBM_GBS = 8000.0          # the metric's nominal denominator ("~8 TB/s")
FALLBACK_HBM_GBS = 6650.0         # earlier measurement on this machine, used only without MEASURED_PEAKS.json
L2_BYTES = 126 << 20

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures summarised under
# profiles/; keyed by (kernel, workload).  None = not captured.
NCU_TRAFFIC_BYTES = {
    # captured at T=8192 (1009.5 MB / 998.4 MB per launch) and scaled by 4: every token moves the same bytes
    ("combine_rows_kernel", "c3_prefill_dsv3"): 4 * 1009.5e6,
    ("dispatch_bulk_kernel", "c3_prefill_dsv3"): 4 * 998.4e6,
    ("combine_rows_kernel", "c3_prefill_dsv3_T8192"): 1009.5e6,
    ("dispatch_bulk_kernel", "c3_prefill_dsv3_T8192"): 998.4e6,
}

WORKLOADS = {
    "c1": lambda: synth.config(1),
    "c2": lambda: synth.config(2),
    "c3": lambda: synth.config(3),
    "c4": lambda: synth.config(4),
    "c5": lambda: synth.config(5, 65536, synth.PREFILL),
    # c3 at a quarter of the tokens: the same kernels and row size, sized for ncu captures (about 1.2 GB resident)
    "c3s": lambda: synth.Workload("c3_prefill_dsv3_T8192", 8192, 7168, 256, 8, 8, synth.PREFILL, "uniform",
                                  "identity", 1003),
}


# ----------------------------------------------------------------------------- algorithmic bytes
def bytes_dispatch(wl) -> int:
    # read each X row once, write it K times; per branch one routing index and one small offset; o table once
    return 2 * wl.H * wl.T * (1 + wl.K) + 8 * wl.T * wl.K + 4 * wl.E * wl.R


def bytes_combine(wl) -> int:
    # read K window rows, write one Y row; per branch index, small offset and weight; o table once
    return 2 * wl.H * wl.T * (wl.K + 1) + 12 * wl.T * wl.K + 4 * wl.E * wl.R


def bytes_plan(wl) -> int:
    # read the routing indexes, write the small offsets, plus the R*E count / offset tables
    return 8 * wl.T * wl.K + 8 * wl.E * wl.R


def describe(wl) -> dict:
    return {"workload": wl.name, "T": wl.T, "H": wl.H, "E": wl.E, "R": wl.R, "K": wl.K,
            "schedule": "prefill" if wl.schedule == synth.PREFILL else "decode", "routing": wl.routing,
            "expert_op": "identity (combine reads the dispatched windows in place)"}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.lines = []
        self.proc = None
        sel = str(device_index)
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            sel = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            pass
        self.cmd = ["nvidia-smi", "-i", sel, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]

    def start(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(wl, frac_den: int):
    """Bounded sample of the workload for the CPU oracle: the first 1/frac_den of every rank's tokens
    (same shape, same routing distribution)."""
    per = wl.T // wl.R
    take = max(1, per // frac_den)
    return synth.Workload(wl.name + f"_sample{frac_den}", take * wl.R, wl.H, wl.E, wl.R, wl.K, wl.schedule,
                          wl.routing, wl.expert_op, wl.seed, wl.zipf_s)


def time_oracle(wl, steps: int, warmup: int, inp=None):
    import oracle
    cores = len(os.sched_getaffinity(0))
    inp = synth.make_inputs(wl) if inp is None else inp
    idx = inp.topk_idx.numpy()
    X = synth.bf16_to_u16(inp.X)
    W = inp.topk_w.numpy()
    p = oracle.plan(idx, wl.E, wl.R)
    C = int(p.n_recv.max())
    win = np.zeros((wl.R * C, wl.H), np.uint16)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        p = oracle.plan(idx, wl.E, wl.R)
        _, slots = oracle.slots(idx, wl.E, wl.R, p, C)
        oracle.dispatch(X, slots, win, cores)
        _, Y = oracle.combine(win, slots, W, wl.H, cores)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    return times, cores


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = oracle_sample(wl, 8)
    times, cores = time_oracle(sample, args.steps, args.warmup)
    sec = sum(times) / len(times)
    nbytes = bytes_plan(sample) + bytes_dispatch(sample) + bytes_combine(sample)
    value = nbytes / sec / 1e9
    what = f"first 1/8 of every rank's tokens of {wl.name} (T={sample.T}) per step"
    line = {
        "impl": "reference", "metric": "moe_plan_dispatch_combine_hbm_gbps", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": describe(wl),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def flush_l2(buf):
    buf.add_(1)


def run_cuda(args, wl):
    from paper_2605_06055_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    inp = synth.make_inputs(wl, pin=True)
    idx_h, w_h = inp.topk_idx.pin_memory(), inp.topk_w.pin_memory()
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)

    # capacity sized from the actual counts (plan -> status -> n_recv), as the prefill schedule allows
    comm.moe_plan(wl.schedule, idx)
    assert comm.moe_status() == 0
    C = int(comm.moe_plan_view()["n_recv"].max().item())
    C = (C + 7) // 8 * 8
    windows = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    b_plan, b_disp, b_comb = bytes_plan(wl), bytes_dispatch(wl), bytes_combine(wl)
    step_bytes = b_plan + b_disp + b_comb
    big = (b_disp > 2 * L2_BYTES)
    scratch = None if big else torch.zeros(256 << 20, dtype=torch.uint8, device=dev)

    def step(events=None):
        if events is not None:
            events[0].record()
        comm.moe_plan(wl.schedule, idx)
        if events is not None:
            events[1].record()
        comm.moe_dispatch(X, windows, C)
        if events is not None:
            events[2].record()
        comm.moe_combine(windows, C, w, Y)
        if events is not None:
            events[3].record()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    assert comm.moe_status() == 0

    # ---- timed region: exactly K steps, CUDA events on the launching stream
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    gaps = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    launches0 = comm.moe_launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        if scratch is not None:         # small workload: flush L2 between steps, outside the per-call events
            gaps[2 * i].record()
            flush_l2(scratch)
            gaps[2 * i + 1].record()
        step(ev[i])
    t_end.record()
    barrier()
    launches = comm.moe_launch_count() - launches0
    total_ms = t_start.elapsed_time(t_end)
    if scratch is not None:
        total_ms -= sum(gaps[2 * i].elapsed_time(gaps[2 * i + 1]) for i in range(args.steps))
    clocks = sampler.stop()
    assert comm.moe_status() == 0
    plan_us = [e[0].elapsed_time(e[1]) * 1e3 for e in ev]
    disp_us = [e[1].elapsed_time(e[2]) * 1e3 for e in ev]
    comb_us = [e[2].elapsed_time(e[3]) * 1e3 for e in ev]
    ms_per_step = total_ms / args.steps
    if dist is not None:
        t = torch.tensor([ms_per_step], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_per_step = float(t.item())

    # ---- end to end through the C ABI from HOST buffers (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(args, wl, comm, inp, idx_h, w_h, X, idx, w, windows, C, Y, barrier, dist, dev, world,
                          step_bytes)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    return finish(args, wl, world, dist, ms_per_step, step_bytes, b_plan, b_disp, b_comb, plan_us, disp_us, comb_us,
                  clocks, launches, e2e, C, big, inp)


def measure_e2e(args, wl, comm, inp, idx_h, w_h, X, idx, w, windows, C, Y, barrier, dist, dev, world, step_bytes):
    y_host = torch.empty((wl.T, wl.H), dtype=torch.bfloat16).pin_memory()
    x_dev2, idx_dev2, w_dev2 = torch.empty_like(X), torch.empty_like(idx), torch.empty_like(w)
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        comm.moe_forward_host(wl.schedule, wl.T, None, inp.X, idx_h, w_h, x_dev2, idx_dev2, w_dev2, windows, C, Y,
                              y_host)
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(e2e_steps):
        comm.moe_forward_host(wl.schedule, wl.T, None, inp.X, idx_h, w_h, x_dev2, idx_dev2, w_dev2, windows, C, Y,
                              y_host)
    t1.record()
    barrier()
    assert comm.moe_status() == 0
    e2e_ms = t0.elapsed_time(t1) / e2e_steps
    if dist is not None:
        t = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    h2d = wl.T * wl.H * 2 + wl.T * wl.K * 8
    d2h = wl.T * wl.H * 2
    return {"value": world * step_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}


def finish(args, wl, world, dist, ms_per_step, step_bytes, b_plan, b_disp, b_comb, plan_us, disp_us, comb_us, clocks,
           launches, e2e, C, big, inp):
    peak, peak_kind = measured_peak()
    med = statistics.median
    kernels = {
        "moe_plan": {"us": med(plan_us), "bytes": b_plan},
        "moe_dispatch": {"us": med(disp_us), "us_min": min(disp_us), "bytes": b_disp,
                         "GBps": b_disp / (sum(disp_us) / len(disp_us)) / 1e3},
        "moe_combine": {"us": med(comb_us), "us_min": min(comb_us), "bytes": b_comb,
                        "GBps": b_comb / (sum(comb_us) / len(comb_us)) / 1e3},
    }
    for k in ("moe_dispatch", "moe_combine"):
        kernels[k]["frac_of_measured_peak"] = kernels[k]["GBps"] / peak
        kernels[k]["frac_of_8TBps"] = kernels[k]["GBps"] / NOMINAL_HBM_GBS
    dom = "moe_dispatch" if sum(disp_us) >= sum(comb_us) else "moe_combine"
    dom_kernel = "dispatch_bulk_kernel" if dom == "moe_dispatch" else "combine_rows_kernel"
    roofline = {"bound": "hbm", "kernel": dom_kernel, "achieved": kernels[dom]["GBps"], "peak": peak,
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": kernels[dom]["GBps"] / peak,
                "traffic": NCU_TRAFFIC_BYTES.get((dom_kernel, wl.name))}

    line = {
        "metric": "moe_plan_dispatch_combine_hbm_gbps", "value": world * step_bytes / (ms_per_step * 1e-3) / 1e9,
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": dict(describe(wl), capacity_rows=C, replicas=world,
                       l2="inputs larger than L2" if big else "256 MB L2 flush between steps (untimed)"),
        "dispatch_plus_combine_us": med(disp_us) + med(comb_us),
        "frac_of_8TBps": (b_disp + b_comb) / ((med(disp_us) + med(comb_us)) * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
        "kernels": kernels, "roofline": roofline, "clocks": clocks, "gpu_launches": launches,
        "e2e": e2e,
    }

    if world == 1 and not args.no_cpu_baseline:
        sample = wl if wl.T * wl.K * wl.H <= 2 * (1 << 30) else oracle_sample(wl, 2)
        times, cores = time_oracle(sample, 1, 1, inp if sample is wl else None)
        sb = bytes_plan(sample) + bytes_dispatch(sample) + bytes_combine(sample)
        line["cpu_baseline"] = {"value": sb / times[0] / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "ms": times[0] * 1e3,
                                "sample": ("whole workload" if sample is wl else
                                           f"first half of every rank's tokens (T={sample.T})") +
                                          ", one timed pass after one warm-up pass, token-parallel over all cores"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]()
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
