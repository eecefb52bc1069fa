"""GPU parity of the overlapped launch: moe_plan_dispatch starts its dispatch kernel while the
planner runs.  It must give exactly the bytes of the separate, serialised calls and of the oracle;
nothing is synchronised between the calls here, so a dispatch that read planner output before its
wait would show as wrong rows.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().view(torch.int16).numpy().view(np.uint16).copy()


def canary(shape, dev):
    return torch.from_numpy(np.full(shape, harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)


def identity(wl):
    return dataclasses.replace(wl, expert_op="identity")


CASES = [
    ("c1_tiny", identity(synth.config(1)), None),
    ("c2_decode", identity(synth.config(2)), None),
    ("c2_shape_prefill_schedule", identity(synth.config(2)), PREFILL),
    ("c5_T1024_decode", identity(synth.config(5, 1024, DECODE)), None),
    ("c5_T8192_prefill", identity(synth.config(5, 8192, PREFILL)), None),          # tile-planned, large job
    ("ragged_empty_rank", Workload("ragged", 1000, 256, 32, 4, 8, DECODE, "uniform", "identity", 77,
                                   rank_tokens=(0, 517, 0, 483)), None),
    ("K3_generic", Workload("k3", 129, 264, 12, 3, 3, DECODE, "replace", "identity", 78, rank_tokens=(40, 0, 89)), None),
    ("one_token", Workload("one", 2, 512, 4, 2, 2, DECODE, "uniform", "identity", 79), None),
    ("tile_planned_decode", Workload("tiles", 6000, 64, 16, 2, 2, DECODE, "uniform", "identity", 80,
                                     rank_tokens=(5000, 1000)), None),
    ("long_rows", Workload("long", 512, 16384, 16, 4, 4, DECODE, "uniform", "identity", 81), None),
]


@pytest.mark.parametrize("overlap", [1, 0])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_fused_plan_dispatch_then_combine_matches_the_oracle(case, overlap):
    _, wl, schedule = case
    sch = wl.schedule if schedule is None else schedule
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + 2
    o = harness.oracle_run(inp, C)
    dev = torch.device(DEV)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_set_option(binding.MOE_OPT_OVERLAP, overlap)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    rts = None if wl.rank_tokens is None else inp.rank_tok_start
    for _ in range(3):                       # cold and warm; repeated launches with nothing in between
        win, Y = canary((wl.R * C, wl.H), dev), canary((wl.T, wl.H), dev)
        torch.cuda.synchronize()
        comm.moe_plan_dispatch(sch, idx, X, win, C, wl.T, rts)
        comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == 0
        assert np.array_equal(u16(win), o.windows)
        assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
        view = comm.moe_plan_view()
        assert np.array_equal(view["small_off"].cpu().numpy(), o.plan.s)
        assert np.array_equal(view["large_off"].cpu().numpy(), o.plan.o)
        assert np.array_equal(view["n_recv"].cpu().numpy(), o.plan.n_recv)
    comm.close()


def test_back_to_back_layers_with_different_routing_do_not_see_each_other():
    """Three layer calls of different routing enqueued with no synchronisation: each overlapped
    kernel may start while the previous layer's kernels still run and must read only its own plan."""
    dev = torch.device(DEV)
    base = identity(synth.config(2))
    comm = binding.MoeComm(base.T, base.H, base.E, base.R, base.K, dev)
    layers = []
    for i in range(3):
        wl = dataclasses.replace(base, seed=9000 + i)
        inp = synth.make_inputs(wl)
        p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
        C = int(p.n_recv.max())
        layers.append((inp, C, harness.oracle_run(inp, C), inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev),
                       canary((wl.R * C, wl.H), dev), canary((wl.T, wl.H), dev)))
    for rounds in range(2):
        torch.cuda.synchronize()
        for inp, C, o, X, idx, w, win, Y in layers:
            comm.moe_plan_dispatch(DECODE, idx, X, win, C)
            comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == 0
        for inp, C, o, X, idx, w, win, Y in layers:
            assert np.array_equal(u16(win), o.windows)
            assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
    comm.close()


def test_separate_calls_with_nothing_in_between_give_the_same_bytes():
    dev = torch.device(DEV)
    wl = synth.config(2)                      # scale experts: a kernel sits between dispatch and combine
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    for path in (binding.MOE_DISPATCH_BULK, binding.MOE_DISPATCH_REGISTERS):
        g = harness.gpu_run(inp, C, dispatch_path=path)
        harness.assert_parity(g, o, wl.schedule)
    # identity experts: combine directly behind dispatch, both dispatch kernels
    wl_id = identity(wl)
    inp_id = synth.make_inputs(wl_id)
    o_id = harness.oracle_run(inp_id, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp_id.X.to(dev), inp_id.topk_idx.to(dev), inp_id.topk_w.to(dev)
    for path in (binding.MOE_DISPATCH_BULK, binding.MOE_DISPATCH_REGISTERS):
        comm.moe_set_option(binding.MOE_OPT_DISPATCH_PATH, path)
        win, Y = canary((wl.R * C, wl.H), dev), canary((wl.T, wl.H), dev)
        comm.moe_plan(DECODE, idx)
        comm.moe_dispatch(X, win, C)
        comm.moe_combine(win, C, w, Y)
        comm.moe_combine(win, C, w, Y)        # a second combine behind a combine: plain launch
        assert comm.moe_status() == 0
        assert np.array_equal(u16(win), o_id.windows)
        assert harness.max_ulp_diff(u16(Y), o_id.Y) <= 1
    comm.close()


def test_fused_call_errors_write_nothing_and_leave_nothing_in_flight():
    dev = torch.device(DEV)
    T, H, E, R, K = 2048, 7168, 256, 16, 8
    wl = Workload("err_fused", T, H, E, R, K, DECODE, "uniform", "identity", 91)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), E, R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(T, H, E, R, K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    win, Y = canary((R * C, H), dev), canary((T, H), dev)
    canary_only = lambda t: bool((t.view(torch.int16) == np.int16(harness.CANARY)).all())

    # host-detected
    assert comm.moe_plan_dispatch(DECODE, idx, X, win, -1, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_plan_dispatch(DECODE, idx, X.view(-1)[1:], win, C, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_plan_dispatch(5, idx, X, win, C, check=False) == binding.MOE_ERR_INVALID_ARG
    for sch in (DECODE, PREFILL):
        # the early loads are in flight when the capacity check fails: the kernel waits for them and ends
        comm.moe_plan_dispatch(sch, idx, X, win, C - 1)
        comm.moe_combine(win, C - 1, w, Y)
        assert comm.moe_status() == binding.MOE_ERR_CAPACITY
        assert canary_only(win) and canary_only(Y)
        idx_bad = idx.clone()
        idx_bad[T // 3, 2] = E
        comm.moe_plan_dispatch(sch, idx_bad, X, win, C)
        comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == binding.MOE_ERR_BAD_INDEX
        assert canary_only(win) and canary_only(Y)
        comm.moe_plan_dispatch(sch, idx, X, win, C)
        comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == 0
        assert np.array_equal(u16(win), o.windows)
        assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
        win, Y = canary((R * C, H), dev), canary((T, H), dev)
    comm.close()


def test_overlapped_step_is_capturable_and_replayable():
    dev = torch.device(DEV)
    wl = identity(synth.config(2))
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_plan_dispatch(DECODE, idx, X, win, C)     # warm-up outside capture
    comm.moe_combine(win, C, w, Y)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        comm.moe_plan_dispatch(DECODE, idx, X, win, C)
        comm.moe_combine(win, C, w, Y)
    for n in (1, 2, 5):
        win.zero_()
        Y.zero_()
        for _ in range(n):
            g.replay()
        comm.moe_dispatch(X, win, C)                   # eager calls right behind the replays
        comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == 0
        assert np.array_equal(u16(win), o.windows_zero_init)
        assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
    comm.close()


@pytest.mark.parametrize("cluster", [1, 0])
@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
@pytest.mark.parametrize("case", [
    ("c2_shape", 2048, 7168, 256, 16, 8, None),
    ("R8_ragged_empty_rank", 1500, 256, 64, 8, 6, (0, 400, 1, 99, 500, 0, 250, 250)),
    ("R2_big_E", 900, 64, 2048, 2, 8, None),           # E above the wide planner's limit: 8-warp CTAs
    ("R4_tiny", 8, 64, 4, 4, 1, None),
    ("R16_E16", 320, 128, 16, 16, 4, None),            # one expert per rank
], ids=lambda c: c[0])
def test_single_launch_planner_as_a_cluster_and_with_the_last_cta(case, schedule, cluster):
    """The small-batch planner gives the same table whether its CTAs exchange their count rows through
    distributed shared memory (one cluster of R CTAs) or through global memory and a ticket."""
    name, T, H, E, R, K, per = case
    wl = Workload(name, T, H, E, R, K, schedule, "uniform", "scale", 6100 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    for align in (1, 8):
        p = oracle.plan(inp.topk_idx.numpy(), E, R, inp.rank_tok_start, align=align)
        C = int(p.n_recv.max()) + 1
        o = harness.oracle_run(inp, C, align=align)
        comm = binding.MoeComm(T, H, E, R, K, torch.device(DEV))
        comm.moe_set_option(binding.MOE_OPT_CLUSTER_PLAN, cluster)
        for _ in range(2):
            g = harness.gpu_run(inp, C, schedule, comm=comm, align=align)
            harness.assert_parity(g, o, schedule, align=align)
        comm.close()


@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
def test_tile_planner_chain_is_capturable_and_replayable(schedule):
    """The three chained planner kernels (the scan kernel as one cluster) inside a CUDA graph, with the
    dispatch behind them, replayed several times and mixed with eager calls."""
    dev = torch.device(DEV)
    wl = Workload("tile_graph", 24000, 256, 32, 8, 4, schedule, "uniform", "identity", 6400)   # 12000 branches per rank
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_plan_dispatch(schedule, idx, X, win, C)
    comm.moe_combine(win, C, w, Y)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        comm.moe_plan_dispatch(schedule, idx, X, win, C)
        comm.moe_combine(win, C, w, Y)
    for n in (1, 3):
        win.zero_()
        Y.zero_()
        for _ in range(n):
            g.replay()
        comm.moe_plan(schedule, idx)                   # eager calls right behind the replays
        comm.moe_combine(win, C, w, Y)
        assert comm.moe_status() == 0
        assert np.array_equal(u16(win), o.windows_zero_init)
        assert harness.max_ulp_diff(u16(Y), o.Y) <= 1
        v = comm.moe_plan_view()
        assert np.array_equal(v["large_off"].cpu().numpy(), o.plan.o)
        if schedule == PREFILL:
            assert np.array_equal(v["small_off"].cpu().numpy(), o.plan.s)
    comm.close()


@pytest.mark.parametrize("shape", [(2048, 1024, 256, 16, 8, DECODE), (24000, 64, 32, 8, 4, PREFILL),
                                   (24000, 64, 32, 8, 4, DECODE), (96, 256, 16, 4, 2, PREFILL)],
                         ids=["decode_cluster_planner", "tile_planner_prefill", "tile_planner_decode", "tiny"])
def test_chained_front_equals_the_serialised_calls_on_fresh_random_routings(shape):
    """gate -> plan -> dispatch as ONE chained call (+ combine) against the same steps enqueued one by one
    on a context with every overlap switched off, on new logits and rows every iteration: the same
    indexes, offsets, window bytes and outputs, bit for bit.  (The serialised path is the one the rest
    of the suite checks against the oracle.)"""
    T, H, E, R, K, sch = shape
    dev = torch.device(DEV)
    a = binding.MoeComm(T, H, E, R, K, dev)
    b = binding.MoeComm(T, H, E, R, K, dev)
    b.moe_set_option(binding.MOE_OPT_OVERLAP, 0)
    b.moe_set_option(binding.MOE_OPT_CLUSTER_PLAN, 0)
    C = (T * K // R) * 2 + 64
    gen = torch.Generator(device=dev).manual_seed(4242)
    for it in range(60):
        logits = torch.randn(T, E, device=dev, generator=gen)
        X = torch.randn(T, H, device=dev, generator=gen).bfloat16()
        ia = torch.empty(T, K, dtype=torch.int32, device=dev)
        wa = torch.empty(T, K, device=dev)
        ib, wb = torch.empty_like(ia), torch.empty_like(wa)
        wina = torch.zeros(R * C, H, dtype=torch.bfloat16, device=dev)
        winb = torch.zeros_like(wina)
        Ya, Yb = torch.empty_like(X), torch.empty_like(X)
        a.moe_gate_plan_dispatch(sch, logits, ia, wa, X, wina, C)
        a.moe_combine(wina, C, wa, Ya)
        binding.moe_gate_topk(logits, K, ib, wb)
        b.moe_plan(sch, ib)
        b.moe_dispatch(X, winb, C)
        b.moe_combine(winb, C, wb, Yb)
        va, vb = a.moe_plan_view(), b.moe_plan_view()
        assert torch.equal(ia, ib) and torch.equal(wa, wb)
        assert torch.equal(va["large_off"], vb["large_off"]) and torch.equal(va["n_recv"], vb["n_recv"])
        assert torch.equal(va["small_off"], vb["small_off"])
        assert torch.equal(wina.view(torch.int16), winb.view(torch.int16))
        assert torch.equal(Ya.view(torch.int16), Yb.view(torch.int16))
    assert a.moe_status() == 0 and b.moe_status() == 0
    a.close()
    b.close()
