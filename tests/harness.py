"""Test harness: runs one workload through the CUDA library (via the C ABI
binding) and through the CPU oracle on the same seeded inputs.

The harness owns what is not part of the method: device buffers, canary fill,
and the stand-in expert op between dispatch and combine.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

import oracle
from paper_2605_06055_b200 import binding, synth

CANARY = 0x7FC1  # a bf16 NaN pattern: a stray read poisons the sum, a stray write is visible


def bf16_key(a: np.ndarray) -> np.ndarray:
    """Monotone integer view of bf16 bit patterns (difference = distance in ulps)."""
    a = a.astype(np.int32)
    return np.where(a & 0x8000, 0x8000 - (a & 0x7FFF), 0x8000 + a)


def max_ulp_diff(got_u16: np.ndarray, want_u16: np.ndarray) -> int:
    """Largest bf16 ulp distance; NaN matches NaN, +0 matches -0."""
    g, w = got_u16.astype(np.int32), want_u16.astype(np.int32)
    g_nan = ((g & 0x7F80) == 0x7F80) & ((g & 0x7F) != 0)
    w_nan = ((w & 0x7F80) == 0x7F80) & ((w & 0x7F) != 0)
    if not np.array_equal(g_nan, w_nan):
        return 1 << 30
    d = np.abs(bf16_key(g) - bf16_key(w))
    d[g_nan] = 0
    return int(d.max()) if d.size else 0


def gpu_expert_scale(windows: torch.Tensor, topk_idx: torch.Tensor, E: int, R: int, C: int,
                     scale: torch.Tensor, align: int = 1) -> None:
    """Stand-in expert op on the device (harness code, not the library):
    every received row of expert e is multiplied by the bf16 scalar scale[e]; with align > 1 the
    padding rows behind an expert's run get the factor 1 (they stay as they are)."""
    n_exp = torch.bincount(topk_idx.reshape(-1).long(), minlength=E)
    E_r = E // R
    win = windows.view(R, C, -1)
    for d in range(R):
        cnt = n_exp[d * E_r:(d + 1) * E_r]
        pad = (cnt + align - 1) // align * align - cnt
        rows = int((cnt + pad).sum())
        if rows == 0:
            continue
        runs = torch.stack([cnt, pad], 1).reshape(-1)                       # count, padding, count, padding, ...
        factors = torch.stack([scale[d * E_r:(d + 1) * E_r]] * 2, 1).reshape(-1)
        real = torch.repeat_interleave(torch.tensor([True, False] * E_r, device=scale.device), runs)
        row_scale = torch.repeat_interleave(factors, runs)
        win[d, :rows][real] = win[d, :rows][real] * row_scale[real][:, None]   # bf16*bf16: fp32 product, one RNE rounding


@dataclass
class OracleRun:
    plan: oracle.Plan
    slots: np.ndarray
    windows: np.ndarray
    Y: np.ndarray
    windows_zero_init: np.ndarray = None   # the same dispatch into zero-filled windows


def oracle_run(inp: synth.Inputs, C: int, n_threads: int = 4, align: int = 1) -> OracleRun:
    wl = inp.wl
    idx = inp.topk_idx.numpy()
    p = oracle.plan(idx, wl.E, wl.R, inp.rank_tok_start, align=align)
    assert p.status == oracle.OK
    st, slots = oracle.slots(idx, wl.E, wl.R, p, C, inp.rank_tok_start)
    assert st == oracle.OK
    win = np.full((wl.R * C, wl.H), CANARY, np.uint16)
    assert oracle.dispatch(synth.bf16_to_u16(inp.X), slots, win, n_threads) == oracle.OK
    win_after_dispatch = win.copy()
    if wl.expert_op == "scale":
        assert oracle.expert_scale(win, wl.H, wl.E, wl.R, C, p.n_exp, synth.bf16_to_u16(inp.scale),
                                   align=align) == oracle.OK
    st, Y = oracle.combine(win, slots, inp.topk_w.numpy(), wl.H, n_threads)
    assert st == oracle.OK
    used = np.zeros(wl.R * C, bool)
    used[slots.reshape(-1)] = True
    zero_init = win_after_dispatch.copy()
    zero_init[~used] = 0
    return OracleRun(p, slots, win_after_dispatch, Y, zero_init)


@dataclass
class DeviceRun:
    view: dict          # plan tensors copied to host (numpy) after the run
    slots: np.ndarray
    windows: np.ndarray  # after dispatch, before the expert op
    Y: np.ndarray
    statuses: list
    expert_start: np.ndarray = None
    expert_count: np.ndarray = None


def gpu_run(inp: synth.Inputs, C: int, schedule: Optional[int] = None, comm: Optional[binding.MoeComm] = None,
            T_max: Optional[int] = None, dispatch_path: int = binding.MOE_DISPATCH_AUTO, granule: int = 0,
            align: int = 1) -> DeviceRun:
    wl = inp.wl
    dev = torch.device("cuda:0")
    schedule = wl.schedule if schedule is None else schedule
    own = comm is None
    if own:
        comm = binding.MoeComm(T_max or max(wl.T, 1), wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_set_option(binding.MOE_OPT_DISPATCH_PATH, dispatch_path)
    comm.moe_set_option(binding.MOE_OPT_GRANULE, granule)
    comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, align)
    idx = inp.topk_idx.to(dev)
    w = inp.topk_w.to(dev)
    X = inp.X.to(dev)
    rts = None if wl.rank_tokens is None else inp.rank_tok_start
    statuses = []
    comm.moe_plan(schedule, idx, wl.T, rts)
    statuses.append(comm.moe_status())
    slots = torch.full((wl.T, wl.K), -5, dtype=torch.int32, device=dev)
    comm.moe_slots(C, slots)
    e_start = torch.full((wl.E,), -5, dtype=torch.int64, device=dev)
    e_count = torch.full((wl.E,), -5, dtype=torch.int32, device=dev)
    comm.moe_expert_ranges(C, e_start, e_count)
    windows = torch.from_numpy(np.full((wl.R * C, wl.H), CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    comm.moe_dispatch(X, windows, C)
    statuses.append(comm.moe_status())
    view = {k: (v.cpu().numpy().copy() if torch.is_tensor(v) else v) for k, v in comm.moe_plan_view().items()}
    win_host = windows.cpu().view(torch.int16).numpy().view(np.uint16).copy()
    if wl.expert_op == "scale":
        gpu_expert_scale(windows, idx, wl.E, wl.R, C, inp.scale.to(dev), align)
    Y = torch.from_numpy(np.full((wl.T, wl.H), CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    comm.moe_combine(windows, C, w, Y)
    statuses.append(comm.moe_status())
    out = DeviceRun(view, slots.cpu().numpy(), win_host, Y.cpu().view(torch.int16).numpy().view(np.uint16).copy(), statuses,
                 e_start.cpu().numpy(), e_count.cpu().numpy())
    if own:
        comm.close()
    return out


def assert_parity(g: DeviceRun, o: OracleRun, schedule: int, combine_ulp: int = 1, align: int = 1):
    assert g.statuses == [0, 0, 0], g.statuses
    names = {"counts": "M", "c_rank": "c_rank", "small_off": "s", "large_off": "o", "n_exp": "n_exp", "n_recv": "n_recv"}
    for k, on in names.items():
        if g.view[k] is None:
            assert schedule == synth.DECODE and k in ("counts", "c_rank", "n_exp")
            continue
        assert np.array_equal(g.view[k], getattr(o.plan, on)), k          # bit-exact integers
    assert np.array_equal(g.slots.astype(np.int64), o.slots)
    # the rows the whole-batch dispatch recorded for the combine behind it: the same numbers, for the same capacity
    if g.slots.size:
        assert g.view["rows_capacity"] == g.windows.shape[0] // o.plan.o.shape[1]
        assert np.array_equal(g.view["rows"].astype(np.int64), o.slots)
    else:
        assert g.view["rows"] is None and g.view["rows_capacity"] == -1
    E, R = o.plan.o.shape
    st, want_start, want_count = oracle.expert_ranges(E, R, g.windows.shape[0] // R, o.plan.n_exp, align=align)
    assert st == oracle.OK and np.array_equal(g.expert_start, want_start) and np.array_equal(g.expert_count, want_count)
    assert np.array_equal(g.windows, o.windows)                           # bit-exact rows and canaries
    ulp = max_ulp_diff(g.Y, o.Y)
    assert ulp <= combine_ulp, ulp
    return ulp
