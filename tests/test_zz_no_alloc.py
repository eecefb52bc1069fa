"""moe_slots_noalloc against the CPU oracle and against the workspace-based entry points.

Some users of the library run where nothing may allocate device memory: inside an
engine that took all of HBM for its own pool, or in a decode loop that must never
stall on an allocation.  They call moe_slots_noalloc, whose planning scratch is a
fixed array inside the library.  This test calls it through the C ABI twice in a
row (the array keeps the first call's contents, so the second call proves that
stale state does no harm) and requires exactly the slots and receive counts that
the oracle computes from the definitions, and that moe_plan + moe_slots produce --
integers, so the tolerance is zero.

Collected last on purpose: if it fails, every other test has already run.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth

pytestmark = pytest.mark.gpu


def workspace_slots(idx, E, R, C, rts):
    """The existing entry points: moe_plan(DECODE) + moe_slots with a caller workspace."""
    T, K = idx.shape
    comm = binding.MoeComm(max(T, 1), 8, E, R, K, idx.device)
    comm.moe_plan(binding.MOE_SCHED_DECODE, idx, T, rts)
    slots = torch.full((T, K), -9, dtype=torch.int32, device=idx.device)
    comm.moe_slots(C, slots)
    assert comm.moe_status() == 0
    n_recv = comm.moe_plan_view()["n_recv"].clone()
    comm.close()
    return slots, n_recv


def oracle_slots(idx_host, E, R, C, rts):
    """The definition: plan (counts, small and large offsets) and the two-level offset rule, on the host."""
    p = oracle.plan(idx_host.numpy(), E, R, rts)
    assert p.status == oracle.OK
    st, slots = oracle.slots(idx_host.numpy(), E, R, p, C, rts)
    assert st == oracle.OK
    return slots, p.n_recv


def make_case(T, K, E, R, routing, per, dev):
    wl = synth.Workload("noalloc", T, 8, E, R, K, synth.DECODE, routing, "identity", 900 + T + R, rank_tokens=per)
    idx, _, _, _ = synth.make_routing(wl)
    rts = None if per is None else synth.rank_tok_start(wl)
    return (wl, idx, idx.to(dev), rts,
            torch.full((T, K), -3, dtype=torch.int32, device=dev),
            torch.full((R,), -3, dtype=torch.int32, device=dev),
            torch.full((1,), -3, dtype=torch.int32, device=dev))


def ragged(T, R, seed):
    """R token counts summing to T, none a multiple of 32 where avoidable, so that every rank ends in a
    partial 256-branch tile."""
    rng = np.random.default_rng(seed)
    cuts = np.sort(rng.choice(np.arange(1, T), R - 1, replace=False))
    return tuple(int(v) for v in np.diff(np.concatenate([[0], cuts, [T]])))


def test_noalloc_matches_oracle_and_workspace_path_on_two_calls_in_a_row():
    dev = torch.device("cuda:0")
    cases = [
        # T, K, E, R, routing, tokens per rank
        (2048, 8, 256, 16, "uniform", None),
        (777, 4, 24, 3, "replace", (500, 0, 277)),
    ]
    # every buffer the entry point touches is created up front; the calls themselves allocate nothing
    bufs = [make_case(*c, dev) for c in cases]
    C = 4096
    for (wl, idx_h, idx, rts, slots, n_recv, status) in bufs:    # two calls in a row, no sync in between
        rc = binding.moe_slots_noalloc(idx, wl.E, wl.R, C, slots, n_recv, status, rts)
        assert rc == binding.MOE_OK
    torch.cuda.synchronize()
    for (wl, idx_h, idx, rts, slots, n_recv, status) in bufs:
        assert int(status.item()) == 0
        want_slots, want_n_recv = oracle_slots(idx_h, wl.E, wl.R, C, rts)
        assert np.array_equal(slots.cpu().numpy().astype(np.int64), want_slots)
        assert np.array_equal(n_recv.cpu().numpy(), want_n_recv)
        ws_slots, ws_n_recv = workspace_slots(idx, wl.E, wl.R, C, rts)
        assert torch.equal(slots, ws_slots)
        assert torch.equal(n_recv, ws_n_recv)

    # same inputs again, in the opposite order: results do not depend on what the array held before
    for (wl, idx_h, idx, rts, slots, n_recv, status) in reversed(bufs):
        first = slots.clone()
        slots.fill_(-3)
        assert binding.moe_slots_noalloc(idx, wl.E, wl.R, C, slots, n_recv, status, rts) == binding.MOE_OK
        torch.cuda.synchronize()
        assert torch.equal(slots, first) and int(status.item()) == 0


@pytest.mark.parametrize("R", [64, 16])
def test_noalloc_at_the_limits_of_the_built_in_scratch(R):
    """T*K = 65536 branches and E = 512 experts exactly, ragged ranks so that every rank ends in a partial tile
    (the tile count reaches its maximum); R = 16 is the shape whose Notify step stages the whole count matrix in
    shared memory (the largest shared-memory request an admitted shape makes)."""
    dev = torch.device("cuda:0")
    T, K, E = 8192, 8, 512
    wl, idx_h, idx, rts, slots, n_recv, status = make_case(T, K, E, R, "uniform", ragged(T, R, R), dev)
    C = T * K
    for _ in range(2):
        slots.fill_(-3)
        assert binding.moe_slots_noalloc(idx, E, R, C, slots, n_recv, status, rts) == binding.MOE_OK
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want_slots, want_n_recv = oracle_slots(idx_h, E, R, C, rts)
        assert np.array_equal(slots.cpu().numpy().astype(np.int64), want_slots)
        assert np.array_equal(n_recv.cpu().numpy(), want_n_recv)


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
    # a routing index outside [0, E): flagged, no slot written either, and the call after it is clean again
    idx[3, 1] = 4
    assert binding.moe_slots_noalloc(idx, 4, 2, 64, slots, n_recv, status) == binding.MOE_OK
    torch.cuda.synchronize()
    assert int(status.item()) == binding.MOE_ERR_BAD_INDEX and bool((slots == -3).all())
    idx[3, 1] = 1
    assert binding.moe_slots_noalloc(idx, 4, 2, 64, slots, n_recv, status) == binding.MOE_OK
    torch.cuda.synchronize()
    want, _ = oracle_slots(idx.cpu(), 4, 2, 64, None)
    assert int(status.item()) == 0 and np.array_equal(slots.cpu().numpy().astype(np.int64), want)
