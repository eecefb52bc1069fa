"""Runs one call of the library a few times on a named workload, for profilers.

    python -m paper_2605_06055_b200.cases <call> <workload> [--reps N] [--flush]

  call      gate | plan | dispatch | combine | dispatch_quant | dispatch_quant_group | step
  workload  c1 c2 c3 c4 c3s (config 3 at a quarter of the tokens) c5 (T=65536) c5m (T=8192) k7

Every repetition is preceded by a 256 MB write when --flush is given, so that a workload smaller than the L2
starts cold.  Inputs are the seeded synthetic ones of `synth`; windows are sized from the plan.  Nothing is
timed here: wrap the command in a profiler (one kernel, a few launches) or time it with CUDA events yourself.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, synth

WORKLOADS = {
    "c1": lambda: synth.config(1),
    "c2": lambda: synth.config(2),
    "c3": lambda: synth.config(3),
    "c4": lambda: synth.config(4),
    "c3s": lambda: synth.Workload("c3_prefill_dsv3_T8192", 8192, 7168, 256, 8, 8, synth.PREFILL, "uniform", "identity",
                                  1003),
    "c5": lambda: synth.config(5, 65536, synth.PREFILL),
    "c5m": lambda: synth.config(5, 8192, synth.PREFILL),
    "k7": lambda: synth.Workload("k7_prefill", 16384, 7168, 256, 8, 7, synth.PREFILL, "uniform", "identity", 1007),
}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("call", choices=["gate", "plan", "dispatch", "combine", "dispatch_quant", "dispatch_quant_group", "step"])
    ap.add_argument("workload", choices=sorted(WORKLOADS))
    ap.add_argument("--reps", type=int, default=4)
    ap.add_argument("--flush", action="store_true")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    wl = WORKLOADS[args.workload]()
    inp = synth.make_inputs(wl)
    idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_plan(wl.schedule, idx)
    assert comm.moe_status() == 0
    C = (int(comm.moe_plan_view()["n_recv"].max().item()) + 7) // 8 * 8
    windows = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_dispatch(X, windows, C)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev) if args.flush else None
    if args.call == "gate":
        logits = torch.randn(wl.T, wl.E, generator=torch.Generator().manual_seed(7)).to(dev)
        g_idx, g_w = torch.empty_like(idx), torch.empty_like(w)
        call = lambda: binding.moe_gate_topk(logits, wl.K, g_idx, g_w)
    elif args.call == "plan":
        call = lambda: comm.moe_plan(wl.schedule, idx)
    elif args.call == "dispatch":
        call = lambda: comm.moe_dispatch(X, windows, C)
    elif args.call == "combine":
        call = lambda: comm.moe_combine(windows, C, w, Y)
    elif args.call == "dispatch_quant":
        wq = torch.zeros((wl.R * C, wl.H), dtype=torch.uint8, device=dev)
        sc = torch.zeros((wl.R * C,), dtype=torch.float32, device=dev)
        call = lambda: comm.moe_dispatch_quant(X, wq, sc, C)
    elif args.call == "dispatch_quant_group":
        wq = torch.zeros((wl.R * C, wl.H), dtype=torch.uint8, device=dev)
        sc = torch.zeros((wl.R * C, wl.H // 128), dtype=torch.float32, device=dev)
        call = lambda: comm.moe_dispatch_quant_group(X, wq, sc, C)
    else:
        def call():
            comm.moe_plan(wl.schedule, idx)
            comm.moe_dispatch(X, windows, C)
            comm.moe_combine(windows, C, w, Y)
    for _ in range(args.reps):
        if flush is not None:
            flush.add_(1)
        call()
    torch.cuda.synchronize()
    assert comm.moe_status() == 0
    print(f"{args.call} on {wl.name}: {args.reps} repetitions done")


if __name__ == "__main__":
    main()
