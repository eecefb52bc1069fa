#!/usr/bin/env python
"""Benchmark of the relay-buffer-free MoE dispatch/combine path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic
routing: moe_plan -> moe_dispatch -> moe_combine (identity experts: combine
reads the dispatched windows in place).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3]
  python bench.py --impl reference ...     # the CPU oracle, timed on the host cores

Default workload: c3, the DeepSeek-V3-like prefill shape on which the HBM
roofline target is stated; the same line carries the decode-step latency (c2)
under "decode".  Multi-GPU: the path does not shard (the R expert-parallel
ranks are virtual segments of one GPU's memory), so N > 1 runs N independent
replicas, one process per GPU, with no data-path collective; value is the sum
over replicas divided by the slowest replica's time ("weak" scaling).
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

METRIC = "moe_plan_dispatch_combine_hbm_gbps"
NOMINAL_HBM_GBS = 8000.0          # the metric's nominal denominator ("~8 TB/s")
FALLBACK_HBM_GBS = 6650.0         # B200 copy bandwidth assumed when no MEASURED_PEAKS.json is present
L2_BYTES = 126 << 20

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/; keyed by (kernel, workload).  Absent = not captured.
NCU_TRAFFIC_BYTES = {
    # dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture at T=8192 (1049.7 MB / 998.8 MB per launch),
    # scaled by 4 for the full size: every token moves the same bytes
    ("combine_rows_kernel", "c3_prefill_dsv3"): 4 * 1049.7e6,
    ("dispatch_bulk_kernel", "c3_prefill_dsv3"): 4 * 998.8e6,
    ("combine_rows_kernel", "c3_prefill_dsv3_T8192"): 1049.7e6,
    ("dispatch_bulk_kernel", "c3_prefill_dsv3_T8192"): 998.8e6,
    # 201 MB workloads, L2 flushed before the launch: part of what the kernel writes is still dirty in L2 at its end
    ("dispatch_bulk_kernel", "c5_mixtral_T8192_prefill"): 67.3e6 + 76.0e6,
    ("combine_rows_kernel", "c5_mixtral_T8192_prefill"): 134.4e6 + 12.4e6,
    # full size, one launch each (read + write)
    ("dispatch_bulk_kernel", "c5_mixtral_T65536_prefill"): 538.0e6 + 1015.1e6,
    ("combine_rows_kernel", "c5_mixtral_T65536_prefill"): 1074.8e6 + 504.7e6,
}

WORKLOADS = {
    "c1": lambda: synth.config(1),
    "c2": lambda: synth.config(2),
    "c3": lambda: synth.config(3),
    "c4": lambda: synth.config(4),
    "c5": lambda: synth.config(5, 65536, synth.PREFILL),
    # a top-k degree without a specialised kernel (K = 7): exercises the any-K paths
    "k7": lambda: synth.Workload("k7_prefill", 16384, 7168, 256, 8, 7, synth.PREFILL, "uniform", "identity", 1007),
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


def bytes_dispatch_quant(wl, group: int = 0) -> int:
    # read each bf16 row once; per branch write H e4m3 codes and one fp32 scale per row (per `group` elements);
    # same metadata as dispatch
    scales = 1 if group == 0 else wl.H // group
    return 2 * wl.H * wl.T + wl.K * wl.T * (wl.H + 4 * scales) + 8 * wl.T * wl.K + 4 * wl.E * wl.R


def bytes_step(wl) -> int:
    return bytes_plan(wl) + bytes_dispatch(wl) + bytes_combine(wl)


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
    """Samples SM clocks and throttle reasons with nvidia-smi while the device is under load."""
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
        self.cmd = ["nvidia-smi", "-i", sel, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                    "-lms", "50"]

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


def time_oracle(wl, steps: int, warmup: int, inp=None, cores=None):
    import oracle
    cores = len(os.sched_getaffinity(0)) if cores is None else cores
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
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample = oracle_sample(wl, 8)
    times, cores = time_oracle(sample, args.steps, args.warmup)
    sec = sum(times) / len(times)
    value = bytes_step(sample) / sec / 1e9
    what = f"first 1/8 of every rank's tokens of {wl.name} (T={sample.T}) per step, token-parallel over all cores"
    cfg = dict(describe(wl), T=sample.T, T_of_full_workload=wl.T,
               sample="first 1/8 of every rank's tokens: the T given here is the T this arm ran")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": cfg,
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def reduce_max_over_ranks(value: float, dist, dev) -> float:
    """Slowest replica's time (device-timed), as the contract asks for multi-GPU numbers."""
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(step_bytes: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` replicas that each move step_bytes per step."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


class Layer:
    """Device buffers and the library context for one workload."""

    def __init__(self, wl, dev, pin=False, inp=None):
        from paper_2605_06055_b200 import binding
        self.wl, self.dev = wl, dev
        self.inp = synth.make_inputs(wl, pin=pin) if inp is None else inp
        self.X, self.idx, self.w = self.inp.X.to(dev), self.inp.topk_idx.to(dev), self.inp.topk_w.to(dev)
        self.comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
        # capacity sized from the actual counts (plan -> status -> n_recv), as the prefill schedule allows
        self.comm.moe_plan(wl.schedule, self.idx)
        assert self.comm.moe_status() == 0
        C = int(self.comm.moe_plan_view()["n_recv"].max().item())
        self.C = (C + 7) // 8 * 8
        self.windows = torch.zeros((wl.R * self.C, wl.H), dtype=torch.bfloat16, device=dev)
        self.Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
        self.big = bytes_dispatch(wl) > 2 * L2_BYTES

    def step(self, events=None):
        c, wl = self.comm, self.wl
        if events is not None:
            events[0].record()
        c.moe_plan(wl.schedule, self.idx)
        if events is not None:
            events[1].record()
        c.moe_dispatch(self.X, self.windows, self.C)
        if events is not None:
            events[2].record()
        c.moe_combine(self.windows, self.C, self.w, self.Y)
        if events is not None:
            events[3].record()


def verify(layer: Layer, samples: int = 4096) -> dict:
    """Checks the state the timed steps left behind, with properties that hold at any size and need no
    reference implementation: the status word is clear; identity experts and weights summing to one give
    Y == X at every element; and sampled branches (t, j) hold X[t] at the window row moe_slots names."""
    c, wl = layer.comm, layer.wl
    assert c.moe_status() == 0
    assert torch.equal(layer.Y.view(torch.int16), layer.X.view(torch.int16)), "combine(dispatch(X)) != X"
    slots = torch.empty((wl.T, wl.K), dtype=torch.int32, device=layer.dev)
    c.moe_slots(layer.C, slots)
    assert c.moe_status() == 0
    g = torch.Generator().manual_seed(5)
    t = torch.randint(0, wl.T, (samples,), generator=g).to(layer.dev)
    j = torch.randint(0, wl.K, (samples,), generator=g).to(layer.dev)
    rows = layer.windows.index_select(0, slots[t, j].long())
    assert torch.equal(rows.view(torch.int16), layer.X.index_select(0, t).view(torch.int16)), "window row != X[t]"
    return {"Y_equals_X": True, "sampled_window_rows": samples}


def time_steps(layer: Layer, steps: int, warmup: int, barrier, scratch=None):
    """K steps bracketed by CUDA events on the launching stream, plus per-call events inside."""
    for _ in range(max(warmup, 3)):
        layer.step()
    assert layer.comm.moe_status() == 0
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    gaps = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps)]
    barrier()
    launches0 = layer.comm.moe_launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(steps):
        if scratch is not None:         # small workload: flush L2 between steps, outside the per-call events
            gaps[2 * i].record()
            scratch.add_(1)
            gaps[2 * i + 1].record()
        layer.step(ev[i])
    t_end.record()
    barrier()
    assert layer.comm.moe_status() == 0
    total_ms = t_start.elapsed_time(t_end)
    if scratch is not None:
        total_ms -= sum(gaps[2 * i].elapsed_time(gaps[2 * i + 1]) for i in range(steps))
    return {
        "ms_per_step": total_ms / steps,
        "plan_us": [e[0].elapsed_time(e[1]) * 1e3 for e in ev],
        "dispatch_us": [e[1].elapsed_time(e[2]) * 1e3 for e in ev],
        "combine_us": [e[2].elapsed_time(e[3]) * 1e3 for e in ev],
        "launches": layer.comm.moe_launch_count() - launches0,
    }


def time_dispatch_quant(layer: Layer, steps: int, scratch=None, group: int = 0):
    """The quantised variant of dispatch (e4m3 codes + one fp32 scale per row, or per `group` elements), same plan."""
    wl = layer.wl
    wq = torch.zeros((wl.R * layer.C, wl.H), dtype=torch.uint8, device=layer.dev)
    if group == 0:
        sc = torch.zeros((wl.R * layer.C,), dtype=torch.float32, device=layer.dev)
        call = lambda: layer.comm.moe_dispatch_quant(layer.X, wq, sc, layer.C)
    else:
        sc = torch.zeros((wl.R * layer.C, wl.H // group), dtype=torch.float32, device=layer.dev)
        call = lambda: layer.comm.moe_dispatch_quant_group(layer.X, wq, sc, layer.C, group)
    for _ in range(3):
        call()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        if scratch is not None:
            scratch.add_(1)
        a.record()
        call()
        b.record()
    torch.cuda.synchronize()
    assert layer.comm.moe_status() == 0
    return [a.elapsed_time(b) * 1e3 for a, b in ev]


def time_e2e(layer: Layer, steps: int, barrier):
    """Whole layer through the C ABI from pinned HOST buffers: H2D of X, K, W and D2H of Y every step."""
    wl, c = layer.wl, layer.comm
    idx_h, w_h = layer.inp.topk_idx.pin_memory(), layer.inp.topk_w.pin_memory()
    x_h = layer.inp.X if layer.inp.X.is_pinned() else layer.inp.X.pin_memory()
    y_h = torch.empty((wl.T, wl.H), dtype=torch.bfloat16).pin_memory()
    x_d, idx_d, w_d = torch.empty_like(layer.X), torch.empty_like(layer.idx), torch.empty_like(layer.w)

    def one():
        c.moe_forward_host(wl.schedule, wl.T, None, x_h, idx_h, w_h, x_d, idx_d, w_d, layer.windows, layer.C,
                           layer.Y, y_h)
    for _ in range(2):
        one()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        one()
    t1.record()
    barrier()
    assert c.moe_status() == 0
    return t0.elapsed_time(t1) / steps, wl.T * wl.H * 2 + wl.T * wl.K * 8, wl.T * wl.H * 2


def time_repeated(fns, n: int) -> float:
    """Microseconds per repetition of calling every function in `fns` once, n repetitions bracketed by
    ONE pair of CUDA events (CUDA event timestamps have a resolution of about 2 us, too coarse for one ~10 us call)."""
    for _ in range(3):
        for f in fns:
            f()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(n):
        for f in fns:
            f()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / n


def time_graphed(fn, launches: int = 20, replays: int = 10) -> float:
    """Microseconds per call of `fn` with `launches` calls captured in one CUDA graph: for kernels of a few
    microseconds, which back-to-back launches from Python cannot feed fast enough to time."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(3):
            fn()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(launches):
                fn()
        g.replay()
        side.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        side.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    return a.elapsed_time(b) * 1e3 / (launches * replays)


def call_latency(layer: Layer, n: int, flush=None) -> dict:
    """Per-call latency as differences of cumulative call sequences (plan | plan+dispatch | plan+dispatch+combine),
    each timed over n repetitions between one pair of CUDA events; `flush` (an L2-flushing call) precedes every
    repetition and its own time is subtracted."""
    c, wl = layer.comm, layer.wl
    plan = lambda: c.moe_plan(wl.schedule, layer.idx)
    disp = lambda: c.moe_dispatch(layer.X, layer.windows, layer.C)
    comb = lambda: c.moe_combine(layer.windows, layer.C, layer.w, layer.Y)
    fused = lambda: c.moe_plan_dispatch(wl.schedule, layer.idx, layer.X, layer.windows, layer.C)
    pre = [flush] if flush is not None else []
    base = time_repeated(pre, n) if pre else 0.0
    t1 = time_repeated(pre + [plan], n)
    t2 = time_repeated(pre + [plan, disp], n)
    t3 = time_repeated(pre + [plan, disp, comb], n)
    tf = time_repeated(pre + [fused, comb], n)
    assert c.moe_status() == 0
    return {"plan_us": t1 - base, "dispatch_us": t2 - t1, "combine_us": t3 - t2, "step_us": t3 - base,
            "step_us_plan_dispatch_fused": tf - base}


def sweeps(dev, n: int = 20) -> dict:
    """Opt-in (--sweeps): one call each of plan, dispatch, combine, the quantised dispatch and the chained
    moe_plan_dispatch over sweeps of the top-k degree, the row length, the rank count and the shapes of published
    MoE models, in microseconds with the TB/s of algorithmic bytes beside them; small jobs start from a flushed L2.
    Every cell checks Y == X.  A paper-independent health check of the kernels away from the benchmark shapes:
    the generic-K combine, the chained launch behind the planner, the table-addressed combine and the long-row
    group-wise quantisation were each found several times below their neighbours by these tables."""
    from paper_2605_06055_b200 import binding
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)

    def cell(name, T, H, E, R, K, sch, peers=False):
        wl = synth.Workload(name, T, H, E, R, K, sch, "uniform", "identity", 1002)
        l = Layer(wl, dev)
        c = l.comm
        nb = 2 * wl.H * wl.T * (1 + wl.K)
        pre = [lambda: flush_buf.add_(1)] if nb < (400 << 20) else []
        base = min(time_repeated(pre, n) for _ in range(2)) if pre else 0.0
        t = lambda fns: min(time_repeated(pre + fns, n) for _ in range(2)) - base
        plan = lambda: c.moe_plan(wl.schedule, l.idx)
        disp = lambda: c.moe_dispatch(l.X, l.windows, l.C)
        comb = lambda: c.moe_combine(l.windows, l.C, l.w, l.Y)
        out = {"T": T, "H": H, "E": E, "R": R, "K": K, "plan_us": t([plan])}
        out["dispatch_us"] = t([disp])
        out["combine_us"] = t([comb])
        out["plan_then_dispatch_us"] = t([plan, disp])
        out["plan_dispatch_chained_us"] = t([lambda: c.moe_plan_dispatch(wl.schedule, l.idx, l.X, l.windows, l.C)])
        if H % 16 == 0:
            wq = torch.zeros((wl.R * l.C, wl.H), dtype=torch.uint8, device=dev)
            sc = torch.zeros((wl.R * l.C,), dtype=torch.float32, device=dev)
            out["dispatch_quant_us"] = t([lambda: c.moe_dispatch_quant(l.X, wq, sc, l.C)])
            if H % 128 == 0:
                scg = torch.zeros((wl.R * l.C, wl.H // 128), dtype=torch.float32, device=dev)
                out["dispatch_quant_group128_us"] = t([lambda: c.moe_dispatch_quant_group(l.X, wq, scg, l.C)])
                del scg
            del wq, sc
        if peers:   # the same windows addressed through a table of bases (the multi-rank calls on one GPU)
            bases = torch.tensor([l.windows.data_ptr() + d * l.C * wl.H * 2 for d in range(wl.R)], dtype=torch.int64,
                                 device=dev)
            out["dispatch_peers_us"] = t([lambda: c.moe_dispatch_peers(l.X, bases, l.C)])
            out["combine_peers_us"] = t([lambda: c.moe_combine_peers(bases, l.C, l.w, l.Y)])
        c.moe_dispatch(l.X, l.windows, l.C)
        c.moe_combine(l.windows, l.C, l.w, l.Y)
        assert c.moe_status() == 0
        assert torch.equal(l.Y.view(torch.int16), l.X.view(torch.int16)), name
        out["dispatch_TBps"] = nb / out["dispatch_us"] / 1e6
        out["combine_TBps"] = nb / out["combine_us"] / 1e6
        c.close()
        del l
        torch.cuda.empty_cache()
        return out

    P, D = synth.PREFILL, synth.DECODE
    res = {"method": f"{n} repetitions per pair of CUDA events, better of two; 256 MB L2 flush in front of jobs below "
                     "400 MB (its time subtracted)"}
    res["top_k"] = {f"K{K}": cell(f"K{K}", 8192, 4096, 64, 8, K, P) for K in (1, 2, 3, 4, 6, 8, 9, 11, 16, 20, 24, 32)}
    res["row_length"] = {f"H{H}": cell(f"H{H}", 16384 if H <= 8192 else 8192, H, 64, 8, 8, P)
                         for H in (256, 512, 1024, 2048, 2880, 4096, 5120, 7168, 8192, 12288, 16384)}
    res["ranks"] = {f"R{R}": cell(f"R{R}", 2048, 7168, 256, R, 8, D, peers=True) for R in (1, 2, 4, 8, 16, 32, 64)}
    res["tokens"] = {f"T{T}": cell(f"T{T}", T, 7168, 256, 8 if T >= 8192 else 16, 8, P if T >= 8192 else D, peers=True)
                     for T in (512, 1024, 3072, 4096, 8192, 32768)}
    models = {"H4096_E128_K8": (4096, 128, 8, 8), "H2048_E128_K8": (2048, 128, 8, 8), "H2880_E128_K4": (2880, 128, 8, 4),
              "H5120_E128_K1": (5120, 128, 8, 1), "H6144_E8_K2": (6144, 8, 8, 2), "H5120_E160_K6": (5120, 160, 8, 6),
              "H7168_E384_K8": (7168, 384, 16, 8)}
    res["model_shapes_T32768"] = {k: cell(k, 32768, H, E, R, K, P) for k, (H, E, R, K) in models.items()}
    res["model_shapes_T1024"] = {k: cell(k, 1024, H, E, R, K, D) for k, (H, E, R, K) in models.items()}
    # one rank's part of a multi-rank plan (moe_layout) and the offsets from the gathered counts (moe_notify)
    res["layout_notify"] = {}
    for R in (8, 16, 64):
        for per in (128, 4096):
            E, K, H = 256, 8, 7168
            wl = synth.Workload(f"R{R}_per{per}", per * R, H, E, R, K, D if per == 128 else P, "uniform", "identity", 1002)
            idx = synth.make_inputs(wl).topk_idx.to(dev)
            whole = binding.MoeComm(wl.T, H, E, R, K, dev)
            whole.moe_plan(P, idx)
            counts = whole.moe_plan_view()["counts"].clone()
            whole_n_recv = whole.moe_plan_view()["n_recv"].clone()
            whole.close()
            mine = idx[:per].contiguous()
            c = binding.MoeComm(per, H, E, R, K, dev)
            lay = lambda: c.moe_layout(wl.schedule, mine, 0, counts[0])
            noti = lambda: c.moe_notify(counts)
            lay(), noti()
            assert c.moe_status() == 0
            entry = {"layout_us": time_graphed(lay), "notify_us": time_graphed(noti),
                     "both_us": time_graphed(lambda: (lay(), noti())), "note": "back to back inside a CUDA graph"}
            # the same with the counts going through the mailboxes: every window of this one GPU behind the table,
            # the other ranks' rows pushed once beforehand (so the notify finds them and never waits)
            flags = binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_COUNTS
            nbytes = c.moe_window_bytes(8, flags)
            backings = [torch.zeros(nbytes // 2, dtype=torch.bfloat16, device=dev) for _ in range(R)]
            bases = [b.data_ptr() for b in backings]
            others = binding.MoeComm(per, H, E, R, K, dev)
            for r in range(1, R):
                others.moe_peers_set(bases, None, 8, my_rank=r, flags=flags)
                others.moe_layout(wl.schedule, idx[r * per:(r + 1) * per].contiguous(), r, counts[r].clone())
                others.moe_push_counts(1)
            c.moe_peers_set(bases, None, 8, my_rank=0, flags=flags)
            boxed = lambda: (c.moe_layout_push(wl.schedule, mine, 0, 1), c.moe_notify_peers(1))
            boxed()
            assert c.moe_status() == 0 and others.moe_status() == 0
            assert torch.equal(c.moe_plan_view()["n_recv"], whole_n_recv)
            entry["layout_push_then_notify_peers_us"] = time_graphed(boxed)
            entry["push_us"] = time_graphed(lambda: c.moe_push_counts(1))
            entry["notify_peers_us"] = time_graphed(lambda: c.moe_notify_peers(1))
            res["layout_notify"][f"R{R}_{per}_tokens_per_rank"] = entry
            others.close()
            c.close()
            del backings
    return res


def decode_latency(dev, peak, n: int = 200, grid: bool = False) -> dict:
    """Decode-step latency (config 2).  Per-call figures are differences of cumulative sequences
    (flush | flush+plan | flush+plan+dispatch | ...), each timed over n repetitions."""
    dwl = synth.config(2)
    dl = Layer(dwl, dev)
    c = dl.comm
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    flush = lambda: flush_buf.add_(1)
    plan = lambda: c.moe_plan(dwl.schedule, dl.idx)
    disp = lambda: c.moe_dispatch(dl.X, dl.windows, dl.C)
    comb = lambda: c.moe_combine(dl.windows, dl.C, dl.w, dl.Y)
    from paper_2605_06055_b200 import binding
    fused = lambda: c.moe_plan_dispatch(dwl.schedule, dl.idx, dl.X, dl.windows, dl.C)
    # three graphs of one step: separate calls with every kernel serialised, separate calls with the
    # combine allowed to start behind the dispatch, and planning folded into the dispatch call
    c.moe_set_option(binding.MOE_OPT_OVERLAP, 0)
    g_serial = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_serial):
        dl.step()
    c.moe_set_option(binding.MOE_OPT_OVERLAP, 1)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        dl.step()
    g_fused = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_fused):
        fused()
        comb()
    replay = lambda: g.replay()
    replay_serial = lambda: g_serial.replay()
    replay_fused = lambda: g_fused.replay()
    out = {"config": describe(dwl),
           "method": f"cumulative sequences of calls, {n} repetitions per pair of CUDA events; per-call = difference",
           "roofline_us_per_call_at_measured_peak": bytes_dispatch(dwl) / peak / 1e3}
    logits = torch.randn(dwl.T, dwl.E, generator=torch.Generator().manual_seed(7)).to(dev)
    g_idx, g_w = torch.empty_like(dl.idx), torch.empty_like(dl.w)
    gate = lambda: binding.moe_gate_topk(logits, dwl.K, g_idx, g_w)
    gate_plan = lambda: c.moe_gate_plan(dwl.schedule, logits, g_idx, g_w)
    # the whole layer front in one call, then combine with the gate's weights (same capacity: the windows were
    # sized for the synthetic routing, so the gate's routing is given a fifth more room)
    g_C = dl.C + dl.C // 5
    g_win = torch.zeros((dwl.R * g_C, dwl.H), dtype=torch.bfloat16, device=dev)
    gate_step = [lambda: c.moe_gate_plan_dispatch(dwl.schedule, logits, g_idx, g_w, dl.X, g_win, g_C),
                 lambda: c.moe_combine(g_win, g_C, g_w, dl.Y)]
    # context for the per-call figures: a plain device-to-device copy that moves the same total bytes
    half = bytes_dispatch(dwl) // 2
    cp_src = torch.zeros(half, dtype=torch.uint8, device=dev)
    cp_dst = torch.empty_like(cp_src)
    copy = lambda: cp_dst.copy_(cp_src)
    wq = torch.empty((dwl.R * dl.C, dwl.H), dtype=torch.uint8, device=dev)
    wscale = torch.empty((dwl.R * dl.C,), dtype=torch.float32, device=dev)
    quant = lambda: c.moe_dispatch_quant(dl.X, wq, wscale, dl.C)
    quant_fused = lambda: c.moe_plan_dispatch_quant(dwl.schedule, dl.idx, dl.X, wq, wscale, dl.C)
    gscale = torch.empty((dwl.R * dl.C, dwl.H // 128), dtype=torch.float32, device=dev) if dwl.H % 128 == 0 else None
    quant_group = (lambda: c.moe_dispatch_quant_group(dl.X, wq, gscale, dl.C, 128)) if gscale is not None else None
    out["gate_us_in_a_cuda_graph"] = time_graphed(gate)      # a 3 us kernel: launches from Python are slower than it
    for name, pre in (("cold", [flush]), ("warm", [])):
        base = time_repeated(pre, n) if pre else 0.0
        t_copy = time_repeated(pre + [copy], n)
        plan()   # the gate leg below leaves the context planned on other indexes
        t_quant = time_repeated(pre + [quant], n)
        t_quant_fused = time_repeated(pre + [quant_fused], n)
        t_quant_group = time_repeated(pre + [quant_group], n) if quant_group is not None else None
        t1 = time_repeated(pre + [plan], n)
        t2 = time_repeated(pre + [plan, disp], n)
        t3 = time_repeated(pre + [plan, disp, comb], n)
        tg = time_repeated(pre + [replay], n)
        tgs = time_repeated(pre + [replay_serial], n)
        tgf = time_repeated(pre + [replay_fused], n)
        tf = time_repeated(pre + [fused, comb], n)
        t_gate_plan = time_repeated(pre + [gate_plan], n)
        t_gate_step = time_repeated(pre + gate_step, n)
        assert c.moe_status() == 0
        out[name] = {"l2": "256 MB L2 flush before every step (its time subtracted)" if pre else
                     "back-to-back steps, no flush",
                     "plan_us": t1 - base, "dispatch_us": t2 - t1, "combine_us": t3 - t2,
                     "step_us_stream_launches": t3 - base, "step_us_cuda_graph": tg - base,
                     "step_us_cuda_graph_no_overlap": tgs - base,
                     "step_us_plan_dispatch_fused_stream_launches": tf - base,
                     "step_us_plan_dispatch_fused_cuda_graph": tgf - base,
                     "dispatch_GBps": bytes_dispatch(dwl) / (t2 - t1) / 1e3,
                     "combine_GBps": bytes_combine(dwl) / (t3 - t2) / 1e3,
                     "gate_plan_us": t_gate_plan - base,
                     "step_us_gate_plan_dispatch_fused_then_combine": t_gate_step - base,
                     "plain_copy_of_the_same_bytes_us": t_copy - base,
                     "dispatch_quant_us": t_quant - base,
                     "plan_dispatch_quant_fused_us": t_quant_fused - base,
                     "dispatch_quant_GBps": bytes_dispatch_quant(dwl) / (t_quant - base) / 1e3}
        if t_quant_group is not None:
            out[name]["dispatch_quant_group128_us"] = t_quant_group - base
            out[name]["dispatch_quant_group128_GBps"] = bytes_dispatch_quant(dwl, 128) / (t_quant_group - base) / 1e3
    plan()   # leave the context planned on dl.idx again
    assert c.moe_status() == 0
    del dl, wq, wscale, cp_src, cp_dst, logits, g_win, flush_buf
    torch.cuda.empty_cache()

    if not grid:
        return out
    # Opt-in (--decode-grid): the grid of the paper's decode table (Table 2): per-rank batch sizes 16..144,
    # H = 4096 and 7168, plain and row-wise quantised dispatch, combine.  The paper does not state its rank
    # count, expert count or top-k; this sweep takes the decode configuration's (16 ranks, 256 experts, top-8).
    # L2 flushed before every call.
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    flush = lambda: flush_buf.add_(1)
    sweep = []
    for H in (4096, 7168):
        for per_rank in (16, 32, 64, 80, 128, 144):
            swl = synth.Workload(f"decode_b{per_rank}_H{H}", per_rank * dwl.R, H, dwl.E, dwl.R, dwl.K, synth.DECODE,
                                 "uniform", "identity", 1200 + per_rank)
            sl = Layer(swl, dev)
            sq = torch.empty((swl.R * sl.C, swl.H), dtype=torch.uint8, device=dev)
            ss = torch.empty((swl.R * sl.C,), dtype=torch.float32, device=dev)
            sc = sl.comm
            s_plan = lambda: sc.moe_plan(swl.schedule, sl.idx)
            best = lambda seq: min(time_repeated(seq, n), time_repeated(seq, n))   # a hiccup inflates one of the two
            base = best([flush])
            t_d = best([flush, lambda: sc.moe_dispatch(sl.X, sl.windows, sl.C)]) - base
            t_q = best([flush, lambda: sc.moe_dispatch_quant(sl.X, sq, ss, sl.C)]) - base
            sg = torch.empty((swl.R * sl.C, swl.H // 128), dtype=torch.float32, device=dev)
            t_g = best([flush, lambda: sc.moe_dispatch_quant_group(sl.X, sq, sg, sl.C, 128)]) - base
            t_c = best([flush, lambda: sc.moe_combine(sl.windows, sl.C, sl.w, sl.Y)]) - base
            t_p = best([flush, s_plan]) - base
            # the same calls back to back (no flush): what a decode loop sees when the windows fit in L2
            # (captured in CUDA graphs: launches from Python cannot feed calls this short fast enough)
            fused_step = lambda: (sc.moe_plan_dispatch(swl.schedule, sl.idx, sl.X, sl.windows, sl.C),
                                  sc.moe_combine(sl.windows, sl.C, sl.w, sl.Y))
            warm = {"dispatch_us": time_graphed(lambda: sc.moe_dispatch(sl.X, sl.windows, sl.C)),
                    "dispatch_quant_us": time_graphed(lambda: sc.moe_dispatch_quant(sl.X, sq, ss, sl.C)),
                    "dispatch_quant_group128_us": time_graphed(lambda: sc.moe_dispatch_quant_group(sl.X, sq, sg, sl.C, 128)),
                    "combine_us": time_graphed(lambda: sc.moe_combine(sl.windows, sl.C, sl.w, sl.Y)),
                    "plan_us": time_graphed(s_plan),
                    "plan_dispatch_fused_then_combine_us": time_graphed(fused_step)}
            t_step = best([flush, lambda: sc.moe_plan_dispatch(swl.schedule, sl.idx, sl.X, sl.windows, sl.C),
                           lambda: sc.moe_combine(sl.windows, sl.C, sl.w, sl.Y)]) - base
            assert sc.moe_status() == 0
            sweep.append({"tokens_per_rank": per_rank, "H": H, "plan_us": t_p, "dispatch_us": t_d,
                          "dispatch_quant_us": t_q, "dispatch_quant_group128_us": t_g, "combine_us": t_c,
                          "plan_dispatch_fused_then_combine_us": t_step, "back_to_back": warm})
            del sl, sq, ss, sg
    out["batch_sweep"] = {"ranks": dwl.R, "experts": dwl.E, "top_k": dwl.K, "rows": sweep}
    return out


# ----------------------------------------------------------------------------- expert-parallel leg (world > 1)
def _group_reduce(value: float, op, dev, group=None) -> float:
    import torch.distributed as dist
    on_host = dist.get_backend(group) == "gloo"
    t = torch.tensor([value], dtype=torch.float64, device="cpu" if on_host else dev)
    dist.all_reduce(t, op=op, group=group)
    return float(t.item())


def ep_shape(key: str, R: int):
    """The decode and prefill shapes with the ranks mapped to processes: 128 / 4096 tokens per rank."""
    per_rank, sched = (128, synth.DECODE) if key == "decode" else (4096, synth.PREFILL)
    return synth.Workload(f"ep_{key}_dsv3", per_rank * R, 7168, 256, R, 8, sched, "uniform", "identity", 1300 + R)


def ep_leg(dev, steps: int, group=None, shapes=("decode", "prefill"),
           variants=(("cached", "host"), ("handshake", "host"), ("cached", "device"), ("static", "device"),
                     ("static", "device", "device"))) -> dict:
    """The path with rank = process = GPU: every process plans its own tokens, the count rows (and window
    generations) are all-gathered over the process group, every rank's window is mapped into every process
    (moe_window_export / moe_peers_open), dispatch stores rows into the other GPUs' windows and combine loads
    them from there.  Only the library's kernels touch peer memory.  Before anything is timed, every rank checks
    its window against the single-GPU path run on the whole batch with R virtual ranks (the path the parity
    tests compare with the CPU definition) and its output against the identity Y == X.
    Variants: (address mode, phase order).  Address mode "cached" exchanges window addresses only when a rank's
    window generation changes (the generations are read on the host every step), "handshake" before every dispatch,
    "static" once (no validity test; with the device phase order a step has no host synchronisation beyond the count
    exchange itself).  Phase order "host" separates the phases by a
    stream synchronisation and a process-group barrier, "device" by arrival flags in the windows' state regions
    (moe_signal_peers / moe_wait_peers) with no host synchronisation between the phases -- unless ranks share a
    GPU, where a host barrier is placed between signal and wait (a wait kernel must not hold a GPU that the
    signalling rank needs).  A third entry "device" sends the count rows through the mailboxes behind the state
    regions (moe_push_counts / moe_notify_peers) instead of an all-gather of the process group: with static
    addresses and the device phase order a step then contains no collective and no host synchronisation at all.
    Times are device time between CUDA events (idle gaps included), max over ranks."""
    import torch.distributed as dist
    from paper_2605_06055_b200 import binding, ep
    rank, R = dist.get_rank(group), dist.get_world_size(group)
    where = ep.all_gather_bytes(f"{os.uname().nodename}:{torch.cuda.get_device_properties(dev).uuid}".encode()
                                .ljust(96)[:96], dev, group)
    shared_gpu = len({where[96 * r:96 * (r + 1)] for r in range(R)}) < R
    out = {"ranks": R, "ranks_share_a_gpu": shared_gpu,
           "peer_access": "windows mapped through inter-process handles; plain bulk stores and coherent loads"}
    if 256 % R != 0:
        out["unavailable"] = f"256 experts do not divide over {R} ranks"
        return out
    for key in shapes:
        wl = ep_shape(key, R)
        inp = synth.make_inputs(wl)               # every rank draws the same batch from the seed and takes its slice
        lo, hi = rank * (wl.T // R), (rank + 1) * (wl.T // R)
        idx, w, X = (inp.topk_idx[lo:hi].contiguous().to(dev), inp.topk_w[lo:hi].contiguous().to(dev),
                     inp.X[lo:hi].contiguous().to(dev))
        Y = torch.empty_like(X)
        res = {"config": describe(wl), "tokens_per_rank": wl.T // R}
        # reference windows: the single-GPU path on the whole batch, R virtual ranks
        ref = binding.MoeComm(wl.T, wl.H, wl.E, R, wl.K, dev)
        g_idx, g_X = inp.topk_idx.to(dev), inp.X.to(dev)
        ref.moe_plan(wl.schedule, g_idx)
        assert ref.moe_status() == 0
        C = (int(ref.moe_plan_view()["n_recv"].max().item()) + 7) // 8 * 8
        ref_win = torch.zeros((R * C, wl.H), dtype=torch.bfloat16, device=dev)
        ref.moe_dispatch(g_X, ref_win, C)
        assert ref.moe_status() == 0
        mine_ref = ref_win[rank * C:(rank + 1) * C].clone()
        del ref_win
        ref_q = torch.zeros((R * C, wl.H), dtype=torch.uint8, device=dev)
        ref_s = torch.zeros((R * C,), dtype=torch.float32, device=dev)
        ref.moe_dispatch_quant(g_X, ref_q, ref_s, C)
        assert ref.moe_status() == 0
        mine_ref_q, mine_ref_s = ref_q[rank * C:(rank + 1) * C].clone(), ref_s[rank * C:(rank + 1) * C].clone()
        del ref_q, ref_s, g_X, g_idx
        ref.close()
        for variant in variants:
            mode, sync = variant[0], variant[1]
            counts = variant[2] if len(variant) > 2 else "collective"
            name = f"{mode}_addresses__{sync}_phase_order" + ("__counts_through_mailboxes" if counts == "device" else "")
            me = ep.EpRank(wl.T // R, wl.H, wl.E, wl.K, dev, group, mode=mode, sync=sync, host_fence=shared_gpu,
                           counts=counts)
            with_quant = (mode, sync) == ("cached", "host")   # this variant also times the quantised dispatch
            window = me.new_window(C, quant=with_quant)       # rows + zeroed state region (+ codes, scales), attached
            ok, why = 1.0, ""
            try:
                me.plan(wl.schedule, idx)     # (with the mailboxes: exchanges the addresses first, they carry the counts)
                if counts != "device":
                    me.handshake()
            except Exception as exc:      # e.g. no peer access between two of the GPUs
                ok, why = 0.0, repr(exc)
            if _group_reduce(ok, dist.ReduceOp.MIN, dev, group) < 1.0:
                res[name] = {"unavailable": why or "the address handshake failed on another rank"}
                continue
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]

            def step(e=None):
                if e is not None:
                    e[0].record()
                me.plan(wl.schedule, idx)
                if e is not None:
                    e[1].record()
                me.dispatch(X)             # addresses (if stale), rows into every window, then the phase boundary
                if e is not None:
                    e[2].record()
                me.combine(w, Y)           # identity experts: the phase boundary, then rows from every window
                if e is not None:
                    e[3].record()
                if sync == "host":
                    me._host_barrier()     # nobody starts the next dispatch while a rank still reads

            step()
            assert me.status() == 0
            same_window = bool(torch.equal(window.view(torch.int16), mine_ref.view(torch.int16)))
            same_output = bool(torch.equal(Y.view(torch.int16), X.view(torch.int16)))
            agreed = _group_reduce(1.0 if (same_window and same_output) else 0.0, dist.ReduceOp.MIN, dev, group)
            assert agreed == 1.0, f"expert-parallel leg ({key}, {name}): rank {rank} window {same_window}, output {same_output}"
            for _ in range(2):
                step()
            handshakes0 = me.handshakes
            for e in ev:
                step(e)
            assert me.status() == 0
            mean = lambda a, b: sum(e[a].elapsed_time(e[b]) for e in ev) / steps * 1e3
            red = lambda v: _group_reduce(v, dist.ReduceOp.MAX, dev, group)
            res[name] = {"verified": {"window_equals_single_gpu_path": True, "Y_equals_X": True},
                         "step_us": red(mean(0, 3)), "plan_and_count_exchange_us": red(mean(0, 1)),
                         "dispatch_phase_us": red(mean(1, 2)), "combine_phase_us": red(mean(2, 3)),
                         "handshakes_in_timed_steps": me.handshakes - handshakes0, "steps": steps,
                         "dispatch_bytes_per_rank": bytes_dispatch(wl) // R}
            if with_quant:
                # row-wise quantised dispatch through the same address table: codes and scales of this rank against
                # the single-GPU path's, then timed like the dispatch phase above
                me.plan(wl.schedule, idx)
                me.dispatch_quant(X)
                assert me.status() == 0
                codes, scales = me.quant_views()
                same = bool(torch.equal(codes, mine_ref_q)) and bool(torch.equal(scales.view(torch.int32),
                                                                                 mine_ref_s.view(torch.int32)))
                assert _group_reduce(1.0 if same else 0.0, dist.ReduceOp.MIN, dev, group) == 1.0, \
                    f"expert-parallel leg ({key}): quantised dispatch differs on rank {rank}"
                qe = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
                for a, b in qe:
                    me.plan(wl.schedule, idx)
                    a.record()
                    me.dispatch_quant(X)
                    b.record()
                    me._host_barrier()
                res[name]["quantised_dispatch_phase_us"] = red(sum(a.elapsed_time(b) for a, b in qe) / steps * 1e3)
                res[name]["verified"]["quantised_codes_and_scales_equal_single_gpu_path"] = True
            me.close()
            del window
        out[key] = res
        del inp, X, Y, idx, w, mine_ref, mine_ref_q, mine_ref_s
        torch.cuda.empty_cache()
    return out


def spawn_ep_child(cmd, env, timeout_s: float) -> dict:
    """Runs the expert-parallel leg of this rank as a child process (its own process group over MASTER_PORT + 17)
    and returns what its rank 0 printed.  The leg touches other GPUs' memory and waits for other ranks; run apart
    from the replica figures, a failure there -- an address handshake that is refused, a rank that dies, a wait
    that never returns -- ends with the child (killed by exact PID after timeout_s) and an `error` entry, never with
    the loss of the benchmark's line."""
    try:
        done = subprocess.run(cmd, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=timeout_s)
    except subprocess.TimeoutExpired:
        return {"error": f"the expert-parallel leg did not finish within {timeout_s:.0f} s; its process was ended"}
    if done.returncode != 0:
        return {"error": f"the expert-parallel leg exited with code {done.returncode}",
                "stderr_tail": done.stderr[-400:]}
    for ln in reversed(done.stdout.splitlines()):
        if ln.startswith("{"):
            return json.loads(ln)
    return {}


def run_ep_child(args) -> None:
    """`--ep-child`: one rank of the expert-parallel leg; rank 0 prints the leg's JSON object."""
    import torch.distributed as dist
    local = int(os.environ.get("LOCAL_RANK", "0")) if args.ep_device < 0 else args.ep_device
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    if args.ep_backend == "nccl":
        dist.init_process_group("nccl", device_id=dev)
    else:
        dist.init_process_group(args.ep_backend)
    shapes = tuple(args.ep_shapes.split(","))
    out = ep_leg(dev, args.steps or 20, None, shapes=shapes)
    if dist.get_rank() == 0:
        print(json.dumps(out), flush=True)
    dist.barrier()
    dist.destroy_process_group()


def kernel_table(wl, r, peak):
    med = statistics.median
    mean = lambda v: sum(v) / len(v)
    p95 = lambda v: sorted(v)[min(len(v) - 1, int(0.95 * len(v)))]
    k = {
        "moe_plan": {"us": med(r["plan_us"]), "us_mean": mean(r["plan_us"]), "us_p95": p95(r["plan_us"]),
                     "bytes": bytes_plan(wl)},
        "moe_dispatch": {"us": med(r["dispatch_us"]), "us_mean": mean(r["dispatch_us"]),
                         "us_min": min(r["dispatch_us"]), "us_p95": p95(r["dispatch_us"]),
                         "bytes": bytes_dispatch(wl),
                         "GBps": bytes_dispatch(wl) / mean(r["dispatch_us"]) / 1e3},
        "moe_combine": {"us": med(r["combine_us"]), "us_mean": mean(r["combine_us"]),
                        "us_min": min(r["combine_us"]), "us_p95": p95(r["combine_us"]),
                        "bytes": bytes_combine(wl),
                        "GBps": bytes_combine(wl) / mean(r["combine_us"]) / 1e3},
    }
    for name, kernel in (("moe_dispatch", "dispatch_bulk_kernel"), ("moe_combine", "combine_rows_kernel")):
        k[name]["frac_of_measured_peak"] = k[name]["GBps"] / peak
        k[name]["frac_of_8TBps"] = k[name]["GBps"] / NOMINAL_HBM_GBS
        k[name]["kernel"] = kernel
        k[name]["ncu_dram_bytes_per_launch"] = NCU_TRAFFIC_BYTES.get((kernel, wl.name))
    return k


def roofline_of(kernels, name, peak, peak_kind):
    k = kernels[name]
    return {"bound": "hbm", "kernel": k["kernel"], "achieved": k["GBps"], "peak": peak, "peak_kind": f"of {peak_kind}",
            "unit": "GB/s", "frac": k["GBps"] / peak, "traffic": k["ncu_dram_bytes_per_launch"]}


def prefill_sizes(dev, peak, barrier, steps: int) -> dict:
    """The other prefill sizes the >= 70 %-of-roofline target is stated on, next to the main workload: the
    skewed-routing configuration and the Mixtral-like shape at T = 65536 under both schedules.  Same timing as
    the main line (per-call CUDA events inside a run of `steps` steps; every window set is far larger than L2),
    each followed by verify()."""
    out = {}
    shared = None
    for key, wl in (("c4", synth.config(4)), ("c5_T65536_prefill", synth.config(5, 65536, synth.PREFILL)),
                    ("c5_T65536_decode", synth.config(5, 65536, synth.DECODE))):
        reuse = shared if (shared is not None and shared.wl.seed == wl.seed and shared.wl.T == wl.T) else None
        layer = Layer(wl, dev, inp=reuse)
        shared = layer.inp
        r = time_steps(layer, steps, 5, barrier)
        check = verify(layer)
        k = kernel_table(wl, r, peak)
        dc_us = k["moe_dispatch"]["us"] + k["moe_combine"]["us"]
        out[key] = {"config": dict(describe(wl), capacity_rows=layer.C), "steps": steps,
                    "ms_per_step": r["ms_per_step"], "dispatch_plus_combine_us": dc_us,
                    "frac_of_8TBps": (bytes_dispatch(wl) + bytes_combine(wl)) / (dc_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
                    "kernels": k, "verified": check}
        del layer
        torch.cuda.empty_cache()
    return out


def run_cuda(args, wl):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    layer = Layer(wl, dev, pin=not args.no_e2e)
    scratch = None if layer.big else torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    sampler.start()
    r = time_steps(layer, args.steps, args.warmup, barrier, scratch)
    ms_per_step = reduce_max_over_ranks(r["ms_per_step"], dist, dev)
    verified = verify(layer)            # bench steps use identity experts whatever the workload names
    quant_us = quant_group_us = None
    if wl.H % 16 == 0 and not args.no_decode:
        quant_us = time_dispatch_quant(layer, min(args.steps, 50), scratch)
        if wl.H % 128 == 0:
            quant_group_us = time_dispatch_quant(layer, min(args.steps, 50), scratch, 128)
    chained_us = None
    if not args.no_decode:
        # moe_plan_dispatch (the dispatch kernel launched behind the planner) against the two calls it replaces
        c = layer.comm
        pre = [] if scratch is None else [lambda: scratch.add_(1)]   # small workloads start cold
        n = max(3, min(args.steps, 30))
        base = time_repeated(pre, n) if pre else 0.0
        two = time_repeated(pre + [lambda: c.moe_plan(wl.schedule, layer.idx),
                                   lambda: c.moe_dispatch(layer.X, layer.windows, layer.C)], n) - base
        one = time_repeated(pre + [lambda: c.moe_plan_dispatch(wl.schedule, layer.idx, layer.X, layer.windows, layer.C)],
                            n) - base
        chained_us = (one, two)
    gate_us = None
    if not args.no_decode:
        from paper_2605_06055_b200 import binding
        logits = torch.randn(wl.T, wl.E, generator=torch.Generator().manual_seed(7)).to(dev)
        g_idx, g_w = torch.empty_like(layer.idx), torch.empty_like(layer.w)
        gate_us = time_graphed(lambda: binding.moe_gate_topk(logits, wl.K, g_idx, g_w))
        del logits, g_idx, g_w
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 10))
        e2e_ms, h2d, d2h = time_e2e(layer, e2e_steps, barrier)
        e2e_ms = reduce_max_over_ranks(e2e_ms, dist, dev)
        e2e = {"value": aggregate_value(bytes_step(wl), world, e2e_ms), "unit": "GB/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    clocks = sampler.stop()
    ep_result = None
    if world > 1:
        # every rank starts its part of the expert-parallel leg as a child process (see spawn_ep_child)
        # (its own store on another port: the launcher's store holds this process group's keys)
        env = dict(os.environ, MASTER_PORT=str(int(os.environ.get("MASTER_PORT", "29500")) + 17),
                   TORCHELASTIC_USE_AGENT_STORE="False")
        cmd = [sys.executable, os.path.abspath(__file__), "--ep-child", "--steps", str(min(args.steps, 20))]
        ep_result = spawn_ep_child(cmd, env, timeout_s=420.0)
        ep_result.setdefault("ranks", world)
        barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    kernels = kernel_table(wl, r, peak)
    if quant_us is not None:
        gbps = bytes_dispatch_quant(wl) / (sum(quant_us) / len(quant_us)) / 1e3
        kernels["moe_dispatch_quant"] = {"us": statistics.median(quant_us), "us_min": min(quant_us),
                                         "bytes": bytes_dispatch_quant(wl), "GBps": gbps,
                                         "frac_of_measured_peak": gbps / peak, "frac_of_8TBps": gbps / NOMINAL_HBM_GBS,
                                         "note": "row-wise e4m3 + fp32 scale variant of dispatch; not part of the step"}
    if quant_group_us is not None:
        gb = bytes_dispatch_quant(wl, 128)
        gbps = gb / (sum(quant_group_us) / len(quant_group_us)) / 1e3
        kernels["moe_dispatch_quant_group"] = {"us": statistics.median(quant_group_us), "us_min": min(quant_group_us),
                                               "bytes": gb, "GBps": gbps, "frac_of_measured_peak": gbps / peak,
                                               "frac_of_8TBps": gbps / NOMINAL_HBM_GBS,
                                               "note": "e4m3 + one fp32 scale per 128 elements; not part of the step"}
    if chained_us is not None:
        kernels["moe_plan_dispatch"] = {"us": chained_us[0], "moe_plan_then_moe_dispatch_us": chained_us[1],
                                        "note": "planning folded into the dispatch call (Section 5.3), the dispatch "
                                                "kernel launched behind the planner; not part of the step"}
    if gate_us is not None:
        gb = wl.T * wl.E * 4 + wl.T * wl.K * 8
        kernels["moe_gate_topk"] = {"us": gate_us, "bytes": gb, "GBps": gb / gate_us / 1e3,
                                    "note": "top-k + softmax over fp32 router logits [T,E], 20 launches in one CUDA "
                                            "graph (logits fit in L2); not part of the step"}
    dom = "moe_dispatch" if sum(r["dispatch_us"]) >= sum(r["combine_us"]) else "moe_combine"
    other = "moe_combine" if dom == "moe_dispatch" else "moe_dispatch"
    roofline = roofline_of(kernels, dom, peak, peak_kind)               # the dominant kernel of the step
    roofline["second_kernel"] = roofline_of(kernels, other, peak, peak_kind)
    dc_us = kernels["moe_dispatch"]["us"] + kernels["moe_combine"]["us"]
    line = {
        "metric": METRIC, "value": aggregate_value(bytes_step(wl), world, ms_per_step),
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": dict(describe(wl), capacity_rows=layer.C, replicas=world,
                       l2="inputs larger than L2" if layer.big else "256 MB L2 flush between steps (untimed)"),
        "dispatch_plus_combine_us": dc_us,
        "frac_of_8TBps": (bytes_dispatch(wl) + bytes_combine(wl)) / (dc_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
        "kernels": kernels, "roofline": roofline, "clocks": clocks, "gpu_launches": r["launches"], "e2e": e2e,
        "verified": verified,
    }
    if ep_result is not None:
        ep_result["note"] = ("rank = GPU; reported beside the replica figures above, which remain `value`")
        line["ep"] = ep_result

    cpu_inp = layer.inp
    del layer, scratch
    torch.cuda.empty_cache()

    if world == 1 and not args.no_prefill_sizes and args.workload == "c3":
        line["prefill_sizes"] = prefill_sizes(dev, peak, barrier, min(args.steps, 50))
        torch.cuda.empty_cache()

    if world == 1 and not args.no_decode and wl.name != synth.config(2).name:
        line["decode"] = decode_latency(dev, peak, grid=args.decode_grid)
        torch.cuda.empty_cache()
    if world == 1 and args.sweeps:
        line["sweeps"] = sweeps(dev)
        torch.cuda.empty_cache()

    if world == 1 and args.workload == "c5" and not args.no_decode:
        # config 5: both schedules timed at each T of the sweep.  Calls of a few microseconds cannot be timed by
        # one event pair each (the events tick in ~2 us steps), so every figure is a difference of cumulative
        # call sequences; the L2 is flushed before every step while the windows are not far larger than it.
        line["sweep"] = []
        flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
        flush = lambda: flush_buf.add_(1)
        for T in (128, 1024, 8192, 65536):
            for sch in (synth.PREFILL, synth.DECODE):
                swl = synth.config(5, T, sch)
                sl = Layer(swl, dev)
                if T <= 8192:
                    lat = call_latency(sl, 200, flush)
                else:   # calls of hundreds of microseconds: one event pair per call attributes the time best
                    sr = time_steps(sl, 50, 5, barrier)
                    lat = {"plan_us": statistics.median(sr["plan_us"]), "dispatch_us": statistics.median(sr["dispatch_us"]),
                           "combine_us": statistics.median(sr["combine_us"]), "step_us": sr["ms_per_step"] * 1e3}
                line["sweep"].append(dict({"T": T, "schedule": "prefill" if sch == synth.PREFILL else "decode",
                                           "l2": "flushed before every step" if T <= 8192 else "windows far larger than L2",
                                           "dispatch_GBps": bytes_dispatch(swl) / lat["dispatch_us"] / 1e3,
                                           "combine_GBps": bytes_combine(swl) / lat["combine_us"] / 1e3,
                                           "bytes_per_call": bytes_dispatch(swl)}, **lat))
                del sl
        del flush_buf
        torch.cuda.empty_cache()

    if world == 1 and not args.no_cpu_baseline:
        sample = wl if wl.T * wl.K * wl.H <= 2 * (1 << 30) else oracle_sample(wl, 2)
        times, cores = time_oracle(sample, 3, 1, cpu_inp if sample is wl else None)
        best = min(times)
        line["cpu_baseline"] = {"value": bytes_step(sample) / best / 1e9, "unit": "GB/s", "cores": cores,
                                "kind": "oracle", "ms": best * 1e3, "ms_all_passes": [t * 1e3 for t in times],
                                "sample": ("whole workload" if sample is wl else
                                           f"first half of every rank's tokens (T={sample.T})") +
                                          ", best of 3 timed passes after one warm-up pass, token-parallel over all cores"}
        one = oracle_sample(wl, 16) if wl.T // wl.R >= 16 else wl
        t1, _ = time_oracle(one, 3, 1, cores=1)
        t1 = [min(t1)]
        line["cpu_baseline"]["single_thread"] = {"value": bytes_step(one) / t1[0] / 1e9, "unit": "GB/s",
                                                 "ms": t1[0] * 1e3,
                                                 "sample": f"first 1/16 of every rank's tokens (T={one.T})"
                                                           if one is not wl else "whole workload"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default 200 (cuda) / 10 (reference)")
    ap.add_argument("--warmup", type=int, default=None, help="default 10 (cuda) / 2 (reference)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-decode", action="store_true", help="skip the decode-latency leg (profiling runs)")
    ap.add_argument("--no-prefill-sizes", action="store_true",
                    help="skip the other prefill sizes the roofline target is stated on (c4, c5 at T=65536)")
    ap.add_argument("--ep-child", action="store_true", help=argparse.SUPPRESS)      # one rank of the expert-parallel leg
    ap.add_argument("--ep-backend", default="nccl", help=argparse.SUPPRESS)
    ap.add_argument("--ep-device", type=int, default=-1, help=argparse.SUPPRESS)    # tests: every rank on this GPU
    ap.add_argument("--ep-shapes", default="decode,prefill", help=argparse.SUPPRESS)
    ap.add_argument("--sweeps", action="store_true",
                    help="also time single calls over sweeps of top-k, row length, rank count and model shapes")
    ap.add_argument("--decode-grid", action="store_true",
                    help="also time the batch-size x hidden-size grid of the paper's decode table (off by default)")
    args = ap.parse_args()
    if args.ep_child:
        run_ep_child(args)
        return
    wl = WORKLOADS[args.workload]()
    if args.impl == "reference":                 # the oracle takes ~0.3 s per step on its 1/8 sample
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 2 if args.warmup is None else args.warmup
        run_reference(args, wl)
    else:
        args.steps = 200 if args.steps is None else args.steps
        args.warmup = 10 if args.warmup is None else args.warmup
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
