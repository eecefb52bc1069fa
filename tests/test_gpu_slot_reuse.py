"""The window rows a whole-batch dispatch records for the combine behind it (MOE_OPT_SLOT_REUSE): the record equals
the slots of the definition, combine gives the same output with and without it, and a record that does not belong
to the call -- another capacity, a range dispatch, an error in between, words that are no rows at all -- is not used.
Every expected value comes from the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu

SHAPES = [
    Workload("reuse_decode", 512, 1024, 64, 8, 8, DECODE, "uniform", "scale", 9101),            # single-launch planner
    Workload("reuse_prefill_tiles", 6000, 512, 32, 4, 6, PREFILL, "zipf", "scale", 9102),        # tile planner
    Workload("reuse_decode_tiles", 5000, 264, 16, 2, 3, DECODE, "uniform", "scale", 9103),       # finished on the fly
    Workload("reuse_any_k", 300, 2048, 27, 3, 9, PREFILL, "replace", "scale", 9104, rank_tokens=(0, 299, 1)),
]


def u16(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def device_inputs(wl):
    dev = torch.device("cuda:0")
    inp = synth.make_inputs(wl)
    rts = None if wl.rank_tokens is None else inp.rank_tok_start
    return dev, inp, inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev), rts


def capacity(inp, wl, rts, extra=0):
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start)
    assert p.status == oracle.OK
    return int(p.n_recv.max()) + extra


@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
@pytest.mark.parametrize("reuse", [0, 1])
def test_combine_is_the_same_with_and_without_the_record(wl, reuse):
    dev, inp, idx, w, X, rts = device_inputs(wl)
    C = capacity(inp, wl, rts, 3)
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_set_option(binding.MOE_OPT_SLOT_REUSE, reuse)
    g = harness.gpu_run(inp, C, wl.schedule, comm=comm)
    harness.assert_parity(g, o, wl.schedule)
    comm.close()


def test_nothing_is_recorded_before_a_dispatch_nor_by_range_dispatches():
    wl = SHAPES[0]
    dev, inp, idx, w, X, rts = device_inputs(wl)
    C = capacity(inp, wl, rts)
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_plan(wl.schedule, idx)
    v = comm.moe_plan_view()
    assert v["rows"] is None and v["rows_capacity"] == -1
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_dispatch_range(X, win, C, 0, 200)
    comm.moe_dispatch_range(X, win, C, 200, wl.T)
    v = comm.moe_plan_view()
    assert v["rows"] is None and v["rows_capacity"] == -1
    harness.gpu_expert_scale(win, idx, wl.E, wl.R, C, inp.scale.to(dev), 1)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_combine(win, C, w, Y)
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
    # a new plan drops the record of the one before
    comm.moe_dispatch(X, win, C)
    assert comm.moe_plan_view()["rows_capacity"] == C
    comm.moe_plan(wl.schedule, idx)
    assert comm.moe_plan_view()["rows"] is None
    comm.close()


def test_a_record_for_another_capacity_is_not_used():
    wl = SHAPES[1]
    dev, inp, idx, w, X, rts = device_inputs(wl)
    C1 = capacity(inp, wl, rts)
    C2 = C1 + 37
    o2 = harness.oracle_run(inp, C2)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_plan(wl.schedule, idx)
    win1 = torch.zeros((wl.R * C1, wl.H), dtype=torch.bfloat16, device=dev)
    win2 = torch.zeros((wl.R * C2, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_dispatch(X, win2, C2)
    comm.moe_dispatch(X, win1, C1)                      # the record now describes windows of C1 rows
    v = comm.moe_plan_view()
    assert v["rows_capacity"] == C1
    assert np.array_equal(v["rows"].cpu().numpy().astype(np.int64), harness.oracle_run(inp, C1).slots)
    harness.gpu_expert_scale(win2, idx, wl.E, wl.R, C2, inp.scale.to(dev), 1)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_combine(win2, C2, w, Y)                    # resolves every branch from the plan again
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(u16(Y), o2.Y) <= 1
    comm.close()


@pytest.mark.parametrize("call", ["row", "group"])
def test_the_quantised_dispatch_records_the_same_rows(call):
    wl = Workload("reuse_quant", 700, 1024, 32, 4, 4, PREFILL, "uniform", "identity", 9105)
    dev, inp, idx, w, X, rts = device_inputs(wl)
    C = capacity(inp, wl, rts, 1)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_plan(wl.schedule, idx)
    wq = torch.zeros((wl.R * C, wl.H), dtype=torch.uint8, device=dev)
    if call == "row":
        comm.moe_dispatch_quant(X, wq, torch.zeros((wl.R * C,), dtype=torch.float32, device=dev), C)
    else:
        comm.moe_dispatch_quant_group(X, wq, torch.zeros((wl.R * C, wl.H // 128), dtype=torch.float32, device=dev), C)
    assert comm.moe_status() == 0
    v = comm.moe_plan_view()
    assert v["rows_capacity"] == C
    assert np.array_equal(v["rows"].cpu().numpy().astype(np.int64), harness.oracle_run(inp, C).slots)
    comm.close()


def test_words_that_are_no_rows_never_become_addresses():
    """The record is overwritten behind the library's back with values outside the windows: combine skips those
    branches, reports MOE_ERR_NOT_PLANNED and touches nothing outside its buffers; the report drops the record and
    the next combine is right again."""
    wl = SHAPES[0]
    dev, inp, idx, w, X, rts = device_inputs(wl)
    C = capacity(inp, wl, rts)
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_plan(wl.schedule, idx)
    guard = 64
    buf = torch.full(((wl.R * C + 2 * guard) * wl.H,), 0, dtype=torch.int16, device=dev)
    buf.fill_(int(np.int16(np.uint16(harness.CANARY))))
    win = buf[guard * wl.H:(guard + wl.R * C) * wl.H].view(torch.bfloat16).view(wl.R * C, wl.H)
    comm.moe_dispatch(X, win, C)
    assert comm.moe_status() == 0
    rows = comm.moe_plan_view()["rows"]
    junk = torch.tensor([wl.R * C, 2 ** 31 - 1, -1, -(2 ** 31), wl.R * C + 5], dtype=torch.int32, device=dev)
    flat = rows.view(-1)
    n = flat[::7].numel()
    flat[::7] = junk.repeat(n // 5 + 1)[:n]
    harness.gpu_expert_scale(win, idx, wl.E, wl.R, C, inp.scale.to(dev), 1)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    assert comm.moe_combine(win, C, w, Y, check=False) == binding.MOE_OK
    assert comm.moe_status() == binding.MOE_ERR_NOT_PLANNED
    canary = int(np.int16(np.uint16(harness.CANARY)))
    assert bool((buf[:guard * wl.H] == canary).all()) and bool((buf[(guard + wl.R * C) * wl.H:] == canary).all())
    assert comm.moe_plan_view()["rows"] is None
    comm.moe_combine(win, C, w, Y)
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
    comm.close()
