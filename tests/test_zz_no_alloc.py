"""moe_slots_noalloc against the workspace-based entry points.

Some users of the library run where nothing may allocate device memory: inside an
engine that took all of HBM for its own pool, or in a decode loop that must never
stall on an allocation.  They call moe_slots_noalloc, whose planning scratch is a
fixed array inside the library.  This test calls it through the C ABI twice in a
row (the array keeps the first call's contents, so the second call proves that
stale state does no harm) and requires exactly the slots and receive counts that
moe_plan + moe_slots produce -- integers, so the tolerance is zero.

Collected last on purpose: if it fails, every other test has already run.
"""
import numpy as np
import pytest
import torch

from paper_2605_06055_b200 import binding, synth

pytestmark = pytest.mark.gpu


def reference_slots(idx, E, R, C, rts):
    T, K = idx.shape
    comm = binding.MoeComm(max(T, 1), 8, E, R, K, idx.device)
    comm.moe_plan(binding.MOE_SCHED_DECODE, idx, T, rts)
    slots = torch.full((T, K), -9, dtype=torch.int32, device=idx.device)
    comm.moe_slots(C, slots)
    assert comm.moe_status() == 0
    n_recv = comm.moe_plan_view()["n_recv"].clone()
    comm.close()
    return slots, n_recv


def test_noalloc_matches_workspace_path_on_two_calls_in_a_row():
    dev = torch.device("cuda:0")
    cases = [
        # T, K, E, R, routing, tokens per rank
        (2048, 8, 256, 16, "uniform", None),
        (777, 4, 24, 3, "replace", (500, 0, 277)),
    ]
    # every buffer the entry point touches is created up front; the calls themselves allocate nothing
    bufs = []
    for (T, K, E, R, routing, per) in cases:
        wl = synth.Workload("noalloc", T, 8, E, R, K, synth.DECODE, routing, "identity", 900 + T, rank_tokens=per)
        idx, _, _, _ = synth.make_routing(wl)
        rts = None if per is None else synth.rank_tok_start(wl)
        bufs.append((wl, idx.to(dev), rts,
                     torch.full((T, K), -3, dtype=torch.int32, device=dev),
                     torch.full((R,), -3, dtype=torch.int32, device=dev),
                     torch.full((1,), -3, dtype=torch.int32, device=dev)))
    C = 4096
    for (wl, idx, rts, slots, n_recv, status) in bufs:           # two calls in a row, no sync in between
        rc = binding.moe_slots_noalloc(idx, wl.E, wl.R, C, slots, n_recv, status, rts)
        assert rc == binding.MOE_OK
    torch.cuda.synchronize()
    for (wl, idx, rts, slots, n_recv, status) in bufs:
        want_slots, want_n_recv = reference_slots(idx, wl.E, wl.R, C, rts)
        assert int(status.item()) == 0
        assert torch.equal(slots, want_slots)
        assert torch.equal(n_recv, want_n_recv)

    # same inputs again, in the opposite order: results do not depend on what the array held before
    for (wl, idx, rts, slots, n_recv, status) in reversed(bufs):
        first = slots.clone()
        slots.fill_(-3)
        assert binding.moe_slots_noalloc(idx, wl.E, wl.R, C, slots, n_recv, status, rts) == binding.MOE_OK
        torch.cuda.synchronize()
        assert torch.equal(slots, first) and int(status.item()) == 0


def test_noalloc_rejects_oversize_and_reports_device_errors():
    dev = torch.device("cuda:0")
    slots = torch.zeros((8, 2), dtype=torch.int32, device=dev)
    n_recv = torch.zeros((64,), dtype=torch.int32, device=dev)
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    big = torch.zeros((65536 // 8 + 8, 8), dtype=torch.int32, device=dev)              # T*K just over the limit
    big_slots = torch.zeros_like(big)
    assert binding.moe_slots_noalloc(big, 8, 8, 1 << 20, big_slots, n_recv, status) == binding.MOE_ERR_INVALID_ARG
    idx = torch.zeros((8, 2), dtype=torch.int32, device=dev)
    assert binding.moe_slots_noalloc(idx, 1024, 2, 64, slots, n_recv, status) == binding.MOE_ERR_INVALID_ARG   # E > 512
    assert binding.moe_slots_noalloc(idx, 128, 128, 64, slots, torch.zeros(128, dtype=torch.int32, device=dev),
                                     status) == binding.MOE_ERR_INVALID_ARG                                # R > 64
    # capacity too small: flagged on the device, no slot written
    slots.fill_(-3)
    assert binding.moe_slots_noalloc(idx, 4, 2, 3, slots, n_recv, status) == binding.MOE_OK
    torch.cuda.synchronize()
    assert int(status.item()) == binding.MOE_ERR_CAPACITY and bool((slots == -3).all())
    # a routing index outside [0, E): flagged, and the call after it is clean again
    idx[3, 1] = 4
    assert binding.moe_slots_noalloc(idx, 4, 2, 64, slots, n_recv, status) == binding.MOE_OK
    torch.cuda.synchronize()
    assert int(status.item()) == binding.MOE_ERR_BAD_INDEX
    idx[3, 1] = 1
    assert binding.moe_slots_noalloc(idx, 4, 2, 64, slots, n_recv, status) == binding.MOE_OK
    torch.cuda.synchronize()
    want, _ = reference_slots(idx, 4, 2, 64, None)
    assert int(status.item()) == 0 and torch.equal(slots, want)
