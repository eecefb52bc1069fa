"""Full benchmark sizes, in the launch configuration bench.py times, compared with the oracle whole tensor by
whole tensor: every integer the plan produces, every byte of the expert windows after dispatch (padding rows
and their canaries included), and every element of the combined output with a non-trivial expert stand-in
(per-expert scaling) between dispatch and combine.  Covers configs 3 and 4, config 5 at T = 65536 under both
schedules (the large-job combine with two branches), the top-7 shape of the benchmark (the large-job combine of
the any-K family) and the quantised dispatch at config 3, row-wise (the three-stage ring) and with one scale per
128 elements (the register kernel).

The oracle runs token-parallel over all host cores (about half a second per pass at config 3); its windows are
uploaded in chunks and compared on the device.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth

import harness

pytestmark = pytest.mark.gpu

CORES = len(os.sched_getaffinity(0))
CANARY_I16 = int(np.int16(np.uint16(harness.CANARY)))


def as_u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def device_equals_host(dev_rows: torch.Tensor, host_rows: np.ndarray, chunk_rows: int = 1 << 16) -> bool:
    """Element-wise comparison of a device tensor [rows, H] of 16-bit (or 8-bit) patterns with a host array of
    the same shape, uploading the host side in chunks."""
    assert tuple(dev_rows.shape) == host_rows.shape, (dev_rows.shape, host_rows.shape)
    view = {2: torch.int16, 1: torch.uint8, 4: torch.int32}[host_rows.dtype.itemsize]
    np_view = {2: np.int16, 1: np.uint8, 4: np.int32}[host_rows.dtype.itemsize]
    for r0 in range(0, host_rows.shape[0], chunk_rows):
        r1 = min(host_rows.shape[0], r0 + chunk_rows)
        want = torch.from_numpy(host_rows[r0:r1].view(np_view)).to(dev_rows.device)
        if not torch.equal(dev_rows[r0:r1].view(view), want):
            return False
    return True


def full_windows(rows: int, H: int, dev) -> torch.Tensor:
    win = torch.empty((rows, H), dtype=torch.bfloat16, device=dev)
    win.view(torch.int16).fill_(CANARY_I16)
    return win


FULL_CASES = {
    "c3": lambda: (synth.config(3), synth.PREFILL),
    "c4": lambda: (synth.config(4), synth.PREFILL),
    "c5_T65536_prefill": lambda: (synth.config(5, 65536, synth.PREFILL), synth.PREFILL),
    "c5_T65536_decode": lambda: (synth.config(5, 65536, synth.DECODE), synth.DECODE),
    # the benchmark's top-7 workload (no K-specialised dispatch; combine<7> in its large-job form)
    "k7": lambda: (synth.Workload("k7_prefill", 16384, 7168, 256, 8, 7, synth.PREFILL, "uniform", "identity", 1007),
                   synth.PREFILL),
}


@pytest.mark.parametrize("case", sorted(FULL_CASES))
def test_full_size_whole_tensors_against_the_oracle(case):
    dev = torch.device("cuda:0")
    wl, schedule = FULL_CASES[case]()
    inp = synth.make_inputs(wl)
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, wl.E, wl.R)
    assert p.status == oracle.OK
    if case == "c4":
        assert p.n_exp.max() >= 10 * wl.B / wl.E              # the premise of the skewed configuration
    C = (int(p.n_recv.max()) + 7) // 8 * 8                     # as bench.py sizes it
    st, slots = oracle.slots(idx_np, wl.E, wl.R, p, C)
    assert st == oracle.OK
    # per-expert bf16 scale factors of the stand-in expert op (drawn apart from the inputs, so that X, K and W
    # stay the benchmark's own)
    scale = (0.5 + torch.rand(wl.E, generator=torch.Generator().manual_seed(4200 + wl.seed % 1000),
                              dtype=torch.float32)).to(torch.bfloat16)

    # ---- oracle: dispatch into canary-filled windows, scale, combine
    X_u16 = synth.bf16_to_u16(inp.X)
    win_ref = np.full((wl.R * C, wl.H), harness.CANARY, np.uint16)
    assert oracle.dispatch(X_u16, slots, win_ref, CORES) == oracle.OK

    # ---- device
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    windows = full_windows(wl.R * C, wl.H, dev)
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    got_slots = torch.empty((wl.T, wl.K), dtype=torch.int32, device=dev)
    comm.moe_plan(schedule, idx)
    comm.moe_slots(C, got_slots)
    comm.moe_dispatch(X, windows, C)
    assert comm.moe_status() == 0

    # -- integers: everything, bit-exact
    v = comm.moe_plan_view()
    for k, name in {"counts": "M", "c_rank": "c_rank", "small_off": "s", "large_off": "o", "n_exp": "n_exp",
                    "n_recv": "n_recv"}.items():
        if v[k] is None:
            assert schedule == synth.DECODE and k in ("counts", "c_rank", "n_exp")
            continue
        assert np.array_equal(v[k].cpu().numpy(), getattr(p, name)), k
    assert np.array_equal(got_slots.cpu().numpy().astype(np.int64), slots)
    # -- dispatched bytes: the whole window allocation, padding rows (canaries) included
    assert device_equals_host(windows, win_ref)

    # -- planning folded into the dispatch call: the same bytes everywhere
    windows2 = full_windows(wl.R * C, wl.H, dev)
    comm.moe_plan_dispatch(schedule, idx, X, windows2, C)
    assert comm.moe_status() == 0
    assert torch.equal(windows2.view(torch.int16), windows.view(torch.int16))
    del windows2

    # -- combine, identity experts and weights summing to 1: Y == X at every element
    comm.moe_combine(windows, C, w, Y)
    assert comm.moe_status() == 0
    assert torch.equal(Y.view(torch.int16), X.view(torch.int16))

    # -- combine behind the scaling expert op: all of Y against the oracle's, at most 1 bf16 ulp apart
    assert oracle.expert_scale(win_ref, wl.H, wl.E, wl.R, C, p.n_exp, synth.bf16_to_u16(scale)) == oracle.OK
    st, Y_ref = oracle.combine(win_ref, slots, inp.topk_w.numpy(), wl.H, CORES)
    assert st == oracle.OK
    harness.gpu_expert_scale(windows, idx, wl.E, wl.R, C, scale.to(dev))
    assert device_equals_host(windows, win_ref)               # the harness op itself, so Y is compared on equal inputs
    comm.moe_combine(windows, C, w, Y)
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(as_u16(Y), Y_ref) <= 1
    comm.close()


def test_full_size_quantised_dispatch_codes_and_scales():
    """Row-wise quantised dispatch at config 3: every e4m3 code of the code windows and every fp32 scale,
    bit-exact against the oracle (padding rows keep their fill)."""
    dev = torch.device("cuda:0")
    wl = synth.config(3)
    inp = synth.make_inputs(wl)
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, wl.E, wl.R)
    C = (int(p.n_recv.max()) + 7) // 8 * 8
    st, slots = oracle.slots(idx_np, wl.E, wl.R, p, C)
    assert st == oracle.OK
    want_q = np.full((wl.R * C, wl.H), 0xAB, np.uint8)
    want_s = np.full((wl.R * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), slots, want_q, want_s, CORES) == oracle.OK

    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx = inp.X.to(dev), inp.topk_idx.to(dev)
    wq = torch.full((wl.R * C, wl.H), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((wl.R * C,), -1.0, dtype=torch.float32, device=dev)
    comm.moe_plan(wl.schedule, idx)
    comm.moe_dispatch_quant(X, wq, sc, C)
    assert comm.moe_status() == 0
    assert device_equals_host(wq, want_q)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    # the chained form gives the same bytes
    wq2 = torch.full_like(wq, 0xAB)
    sc2 = torch.full_like(sc, -1.0)
    comm.moe_plan_dispatch_quant(wl.schedule, idx, X, wq2, sc2, C)
    assert comm.moe_status() == 0
    assert torch.equal(wq2, wq) and torch.equal(sc2.view(torch.int32), sc.view(torch.int32))
    comm.close()


def test_full_size_group_quantised_dispatch_codes_and_scales():
    """One scale per 128 elements at config 3 (the register kernel with ten warps per SM): every e4m3 code and
    every one of the 56 fp32 scales of every window row, bit-exact against the oracle; padding rows keep their fill."""
    dev = torch.device("cuda:0")
    wl = synth.config(3)
    G = wl.H // 128
    inp = synth.make_inputs(wl)
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, wl.E, wl.R)
    C = (int(p.n_recv.max()) + 7) // 8 * 8
    st, slots = oracle.slots(idx_np, wl.E, wl.R, p, C)
    assert st == oracle.OK
    want_q = np.full((wl.R * C, wl.H), 0xAB, np.uint8)
    want_s = np.full((wl.R * C, G), -1.0, np.float32)
    assert oracle.dispatch_quant_group(synth.bf16_to_u16(inp.X), slots, want_q, want_s, 128, CORES) == oracle.OK

    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx = inp.X.to(dev), inp.topk_idx.to(dev)
    wq = torch.full((wl.R * C, wl.H), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((wl.R * C, G), -1.0, dtype=torch.float32, device=dev)
    comm.moe_plan(wl.schedule, idx)
    comm.moe_dispatch_quant_group(X, wq, sc, C)
    assert comm.moe_status() == 0
    assert device_equals_host(wq, want_q)
    assert device_equals_host(sc.view(torch.int32), want_s.view(np.int32))
    # the chained form gives the same bytes
    wq2 = torch.full_like(wq, 0xAB)
    sc2 = torch.full_like(sc, -1.0)
    comm.moe_plan_dispatch_quant_group(wl.schedule, idx, X, wq2, sc2, C)
    assert comm.moe_status() == 0
    assert torch.equal(wq2, wq) and torch.equal(sc2.view(torch.int32), sc.view(torch.int32))
    comm.close()
