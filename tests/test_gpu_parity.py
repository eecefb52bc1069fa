"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle,
element by element, on the same seeded inputs.

Bar: bit-exact counts, offsets, slots and dispatched window bytes (canaries
included); combine within 1 bf16 ulp (both sides accumulate in fp32 with one
fma per term, j ascending, so the observed distance is normally 0).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu


PATHS = [binding.MOE_DISPATCH_BULK, binding.MOE_DISPATCH_REGISTERS]


def run_and_check(wl, schedule=None, slack=3, paths=PATHS, granule=0):
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + slack if wl.T else slack
    o = harness.oracle_run(inp, C)
    sch = wl.schedule if schedule is None else schedule
    worst = 0
    for path in paths:                      # every dispatch kernel must give the same bytes
        g = harness.gpu_run(inp, C, sch, dispatch_path=path, granule=granule)
        worst = max(worst, harness.assert_parity(g, o, sch))
    return worst


# ------------------------------------------------------------------ the benchmark configurations
def test_config1_tiny_prefill():
    assert run_and_check(synth.config(1)) == 0


def test_config1_under_decode_schedule():
    run_and_check(synth.config(1), DECODE)


def test_config2_decode_dsv3_full_size():
    run_and_check(synth.config(2))


def test_config2_under_prefill_schedule():
    run_and_check(synth.config(2), PREFILL)


@pytest.mark.parametrize("T", [128, 1024, 8192])
@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
def test_config5_mixtral_sweep(T, schedule):
    run_and_check(synth.config(5, T, schedule))


def test_config3_shape_reduced_tokens():
    # DeepSeek-V3-like prefill shape at 1/8 of the tokens: several 1024-branch tiles per rank plus a ragged tail.
    wl = Workload("c3_reduced", 8 * 517, 7168, 256, 8, 8, PREFILL, "uniform", "identity", 3003)
    run_and_check(wl)


def test_config4_zipf_reduced_tokens():
    wl = Workload("c4_reduced", 4096, 7168, 256, 8, 8, PREFILL, "zipf", "identity", 3004)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    assert p.n_exp.max() >= 10 * wl.B / wl.E
    C = int(p.n_recv.max())                      # capacity sized exactly from the actual counts
    g = harness.gpu_run(inp, C)
    harness.assert_parity(g, harness.oracle_run(inp, C), PREFILL)


# ------------------------------------------------------------------ shapes, tails, degenerate cases
EDGE = [
    # name, T, H, E, R, K, routing, rank_tokens
    ("K1", 200, 64, 8, 4, 1, "uniform", None),
    ("R1", 96, 128, 8, 1, 2, "uniform", None),
    ("E_eq_R", 64, 64, 4, 4, 2, "uniform", None),
    ("H8", 300, 8, 16, 4, 4, "uniform", None),
    ("H_not_mult_of_warp_row", 77, 1000, 16, 2, 6, "uniform", (30, 47)),
    ("K3_generic", 129, 264, 12, 3, 3, "replace", (40, 0, 89)),
    ("K5_generic_dups", 250, 520, 10, 5, 5, "replace", (1, 100, 49, 0, 100)),
    ("K7", 300, 1032, 16, 4, 7, "uniform", None),
    ("K10", 200, 2048, 64, 4, 10, "uniform", (50, 70, 0, 80)),
    ("K12_dups", 150, 520, 24, 3, 12, "replace", None),
    ("K16", 120, 4096, 32, 2, 16, "uniform", None),
    ("K9_generic", 90, 264, 16, 2, 9, "uniform", None),
    ("K32_max", 40, 64, 64, 2, 32, "uniform", None),
    ("K20_of_24", 100, 264, 64, 2, 20, "uniform", None),                   # combine forms with spare branches
    ("K27_of_32", 90, 136, 64, 4, 27, "uniform", (30, 0, 40, 20)),
    ("K13_of_16", 150, 4096, 32, 2, 13, "uniform", None),
    ("duplicates_in_token", 333, 72, 4, 2, 4, "replace", (300, 33)),
    ("empty_rank_ragged", 1000, 256, 32, 4, 8, "uniform", (0, 517, 0, 483)),
    ("many_ranks", 512, 64, 256, 64, 8, "uniform", None),
    # more ranks than a cluster holds: the counting CTAs are followed by a launch that builds every window's offsets
    ("many_ranks_tiles", 19200, 32, 64, 32, 8, "uniform", None),           # 4800 branches per rank: tile planner
    ("max_ranks", 768, 64, 256, 256, 2, "uniform", None),                  # R = 256, one expert per rank
    ("many_ranks_ragged", 3000, 40, 96, 48, 4, "zipf", tuple([0, 125] * 24)),
    ("big_E", 3000, 32, 2048, 2, 8, "uniform", None),
    ("tile_boundary_exact", 2048, 32, 8, 2, 2, "uniform", None),   # 2048 branches per rank = exactly two tiles
    ("tile_boundary_plus1", 2050, 32, 8, 2, 2, "uniform", None),
    ("rank_above_compact_decode_limit", 6000, 16, 16, 2, 2, "uniform", (5000, 1000)),   # 10000 branches in rank 0
    ("compact_decode_several_passes", 1200, 16, 1024, 2, 6, "uniform", (682, 518)),     # E > 768: 8-warp planner
    ("compact_several_passes_empty_ranks", 900, 64, 32, 4, 8, "uniform", (0, 500, 0, 400)),   # 4 passes of the 32-warp planner beside ranks that arrive at once
    ("max_ranks_max_experts", 4096, 64, 4096, 256, 8, "uniform", None),                 # R = MOE_MAX_R, E = MOE_MAX_E
    ("many_tiles", 200000, 32, 64, 8, 8, "uniform", None),                              # 1.6 M branches, 98 tiles per rank
    ("long_rows_two_items_per_row", 512, 16384, 16, 4, 4, "uniform", None),             # 32 KB rows
    ("row_of_three_units_and_a_tail", 700, 808, 8, 2, 2, "uniform", None),              # 1616-byte rows: 3 units + 80 B
    ("leftover_rows_cut_finer", 1280, 7168, 256, 16, 8, "uniform", None),               # 1280 = 1184 warps + 96 rows
    ("leftover_rows_cut_finer_ragged", 2500, 4104, 8, 4, 2, "uniform", (700, 600, 1100, 100)),   # 17 units per row
]


@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_edge_shapes(case, schedule):
    name, T, H, E, R, K, routing, rank_tokens = case
    wl = Workload(name, T, H, E, R, K, schedule, routing, "scale", 4000 + T, rank_tokens=rank_tokens)
    run_and_check(wl)


@pytest.mark.parametrize("granule", [1, 3, 5, 28, 1000])
def test_any_work_item_size_gives_the_same_result(granule):
    wl = Workload("granule", 300, 7168, 64, 4, 8, DECODE, "uniform", "scale", 4242)
    run_and_check(wl, granule=granule)
    wl = Workload("granule_ragged_row", 123, 1000, 16, 2, 6, PREFILL, "uniform", "scale", 4243, rank_tokens=(23, 100))
    run_and_check(wl, granule=granule)


def test_empty_batch():
    dev = torch.device("cuda:0")
    comm = binding.MoeComm(64, 64, 8, 2, 2, dev)
    idx = torch.zeros((0, 2), dtype=torch.int32, device=dev)
    for sch in (PREFILL, DECODE):
        comm.moe_plan(sch, idx, 0)
        win = torch.zeros((2 * 4, 64), dtype=torch.bfloat16, device=dev)
        comm.moe_dispatch(torch.zeros((0, 64), dtype=torch.bfloat16, device=dev), win, 4)
        comm.moe_combine(win, 4, torch.zeros((0, 2), device=dev), torch.zeros((0, 64), dtype=torch.bfloat16, device=dev))
        assert comm.moe_status() == 0
        v = comm.moe_plan_view()
        assert int(v["n_recv"].abs().sum()) == 0 and int(v["large_off"].abs().sum()) == 0


def test_all_branches_to_one_expert_and_one_empty_expert():
    T, H, E, R, K = 700, 64, 8, 4, 2
    g = torch.Generator().manual_seed(5)
    idx = torch.full((T, K), 5, dtype=torch.int32)
    idx[:, 1] = torch.randint(0, 4, (T,), generator=g).to(torch.int32)     # experts 6,7 (rank 3) and 4 stay empty
    wl = Workload("one_hot_expert", T, H, E, R, K, PREFILL, "replace", "scale", 77)
    inp = synth.make_inputs(wl)
    inp.topk_idx = idx
    p = oracle.plan(idx.numpy(), E, R, inp.rank_tok_start)
    assert p.n_exp[5] == T and p.n_exp[6] == 0
    C = int(p.n_recv.max())
    for sch in (PREFILL, DECODE):
        harness.assert_parity(harness.gpu_run(inp, C, sch), harness.oracle_run(inp, C), sch)


# ------------------------------------------------------------------ properties of the path
def test_identity_round_trip_returns_x_exactly():
    wl = Workload("roundtrip", 1024, 2048, 64, 8, 8, PREFILL, "uniform", "identity", 99)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    g = harness.gpu_run(inp, C)
    assert np.array_equal(g.Y, synth.bf16_to_u16(inp.X))       # sum_j W_j = 1 and identity experts => Y == X


def test_schedules_agree_and_runs_are_bitwise_repeatable():
    wl = synth.config(5, 1024, PREFILL)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max()) + 1
    a = harness.gpu_run(inp, C, PREFILL)
    b = harness.gpu_run(inp, C, DECODE)
    c = harness.gpu_run(inp, C, PREFILL)
    for x in (b, c):
        assert np.array_equal(a.slots, x.slots) and np.array_equal(a.windows, x.windows) and np.array_equal(a.Y, x.Y)
        assert np.array_equal(a.view["small_off"], x.view["small_off"])
        assert np.array_equal(a.view["large_off"], x.view["large_off"])
    assert b.view["counts"] is None and b.view["c_rank"] is None and b.view["n_exp"] is None


def test_context_reuse_across_plans_and_repeated_dispatch():
    dev = torch.device("cuda:0")
    comm = binding.MoeComm(1024, 256, 16, 4, 2, dev)
    for seed, T, sch in [(1, 1024, DECODE), (2, 512, PREFILL), (3, 768, DECODE), (4, 1024, PREFILL)]:
        wl = Workload("reuse", T, 256, 16, 4, 2, sch, "uniform", "identity", seed)
        inp = synth.make_inputs(wl)
        p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
        C = int(p.n_recv.max()) + 2
        o = harness.oracle_run(inp, C)
        g = harness.gpu_run(inp, C, sch, comm=comm)
        harness.assert_parity(g, o, sch)
        # a second dispatch + combine on the same plan gives the same bytes
        X = inp.X.to(dev)
        win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
        Y = torch.empty((T, wl.H), dtype=torch.bfloat16, device=dev)
        comm.moe_dispatch(X, win, C)
        comm.moe_combine(win, C, inp.topk_w.to(dev), Y)
        assert comm.moe_status() == 0
        assert np.array_equal(Y.cpu().view(torch.int16).numpy().view(np.uint16), g.Y)
    comm.close()


def test_decode_combine_without_dispatch_resolves_the_same_rows():
    dev = torch.device("cuda:0")
    wl = Workload("combine_only", 640, 128, 32, 4, 4, DECODE, "uniform", "identity", 31)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    idx = inp.topk_idx.to(dev)
    comm.moe_plan(DECODE, idx)
    win = torch.from_numpy(o.windows.view(np.int16)).to(dev).view(torch.bfloat16)   # expert outputs from elsewhere
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_combine(win, C, inp.topk_w.to(dev), Y)
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), o.Y) <= 1


# ------------------------------------------------------------------ errors (made on the host; nothing faults)
def test_errors_leave_memory_untouched():
    dev = torch.device("cuda:0")
    T, H, E, R, K = 256, 64, 16, 4, 2
    comm = binding.MoeComm(T, H, E, R, K, dev)
    wl = Workload("err", T, H, E, R, K, PREFILL, "uniform", "identity", 8)
    inp = synth.make_inputs(wl)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    p = oracle.plan(inp.topk_idx.numpy(), E, R)
    C = int(p.n_recv.max())
    win = torch.from_numpy(np.full((R * C, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    Y = torch.from_numpy(np.full((T, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    canary_only = lambda t: bool((t.view(torch.int16) == np.int16(harness.CANARY)).all())

    # before any plan
    assert comm.moe_dispatch(X, win, C, check=False) == binding.MOE_ERR_NOT_PLANNED
    assert comm.moe_combine(win, C, w, Y, check=False) == binding.MOE_ERR_NOT_PLANNED
    with pytest.raises(binding.MoeError):
        comm.moe_plan_view()
    # host-detected argument errors
    assert comm.moe_plan(PREFILL, idx, T + 1, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_plan(PREFILL, idx, T, np.array([0, 10, 5, 100, T]), check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_plan(PREFILL, idx, T - 1, check=False) == binding.MOE_ERR_INVALID_ARG    # T % R with no map
    assert comm.moe_plan(7, idx, T, check=False) == binding.MOE_ERR_INVALID_ARG

    for sch in (PREFILL, DECODE):
        # capacity one row short: status CAPACITY, no row written, Y untouched
        comm.moe_plan(sch, idx)
        assert comm.moe_status() == 0
        comm.moe_dispatch(X, win, C - 1)
        assert comm.moe_status() == binding.MOE_ERR_CAPACITY
        comm.moe_combine(win, C - 1, w, Y)
        assert comm.moe_status() == binding.MOE_ERR_CAPACITY
        assert canary_only(win) and canary_only(Y)
        # misaligned payload pointer
        assert comm.moe_dispatch(X.view(-1)[1:], win, C, check=False) == binding.MOE_ERR_INVALID_ARG

        # index == E and index == -1: BAD_INDEX, later calls write nothing until the status is read
        for bad in (E, -1):
            idx_bad = idx.clone()
            idx_bad[T // 2, 1] = bad
            comm.moe_plan(sch, idx_bad)
            comm.moe_dispatch(X, win, C)
            comm.moe_combine(win, C, w, Y)
            assert comm.moe_status() == binding.MOE_ERR_BAD_INDEX
            assert comm.moe_status() == 0                      # cleared by the read
            assert canary_only(win) and canary_only(Y)
            # the plan that saw the bad index does not survive the report: no call may go on to skip the branch
            assert comm.moe_dispatch(X, win, C, check=False) == binding.MOE_ERR_NOT_PLANNED
            assert comm.moe_combine(win, C, w, Y, check=False) == binding.MOE_ERR_NOT_PLANNED
            assert comm.moe_slots(C, torch.empty((T, K), dtype=torch.int32, device=dev), check=False) == \
                binding.MOE_ERR_NOT_PLANNED
            assert canary_only(win) and canary_only(Y)

    # and the context still works afterwards
    comm.moe_plan(PREFILL, idx)
    comm.moe_dispatch(X, win, C)
    comm.moe_combine(win, C, w, Y)
    assert comm.moe_status() == 0
    assert np.array_equal(Y.cpu().view(torch.int16).numpy().view(np.uint16), synth.bf16_to_u16(inp.X))
    comm.close()


def test_forward_host_entry_point():
    dev = torch.device("cuda:0")
    wl = synth.config(5, 1024, DECODE)
    inp = synth.make_inputs(wl, pin=True)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    x_dev = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    idx_dev = torch.empty((wl.T, wl.K), dtype=torch.int32, device=dev)
    w_dev = torch.empty((wl.T, wl.K), dtype=torch.float32, device=dev)
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    y_dev = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    y_host = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16).pin_memory()
    for sch in (DECODE, PREFILL):
        y_host.zero_()
        comm.moe_forward_host(sch, wl.T, None, inp.X, inp.topk_idx.pin_memory(), inp.topk_w.pin_memory(),
                              x_dev, idx_dev, w_dev, win, C, y_dev, y_host)
        assert comm.moe_status() == 0
        o = harness.oracle_run(inp, C)
        assert harness.max_ulp_diff(synth.bf16_to_u16(y_host), o.Y) <= 1
    comm.close()


def test_cuda_graph_replays_and_eager_calls_mix_freely():
    """The path is capturable (no allocation, no synchronisation, host arrays passed by value), and a
    captured call can be replayed any number of times between eager calls: every launch leaves the
    work counters as it found them."""
    dev = torch.device("cuda:0")
    wl = synth.config(2)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(Workload_identity(inp), C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_plan(wl.schedule, idx)
    comm.moe_dispatch(X, win, C)                 # warm-up outside capture
    torch.cuda.synchronize()
    g_dispatch, g_step = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_dispatch):
        comm.moe_dispatch(X, win, C)
    with torch.cuda.graph(g_step):
        comm.moe_plan(wl.schedule, idx)
        comm.moe_dispatch(X, win, C)
        comm.moe_combine(win, C, w, Y)
    for n_replays in (1, 3):                     # odd counts of a single captured launch
        win.zero_()
        for _ in range(n_replays):
            g_dispatch.replay()
        comm.moe_combine(win, C, w, Y)           # eager call right after
        assert comm.moe_status() == 0
        assert np.array_equal(win.cpu().view(torch.int16).numpy().view(np.uint16), o.windows_zero_init)
        assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), o.Y) <= 1
    Y.zero_()
    win.zero_()
    g_step.replay()
    g_dispatch.replay()
    g_step.replay()
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), o.Y) <= 1
    comm.close()


class Workload_identity:
    """Inputs of a workload with the expert op forced to identity and zero-initialised windows (for graphs)."""

    def __new__(cls, inp):
        import copy
        import dataclasses
        out = copy.copy(inp)
        out.wl = dataclasses.replace(inp.wl, expert_op="identity")
        return out


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """Failure path without a fault: one warp of the bulk-copy dispatch waits for bytes that never
    come; its bounded wait expires, the kernel ends normally with MOE_ERR_TIMEOUT in the status word,
    and the next call on the same context is correct."""
    dev = torch.device("cuda:0")
    wl = Workload("starve", 1024, 2048, 32, 4, 4, PREFILL, "uniform", "identity", 61)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_plan(PREFILL, idx)
    comm.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 50)
    comm.moe_dispatch(X, win, C)
    assert comm.moe_status() == binding.MOE_ERR_TIMEOUT
    assert comm.moe_status() == 0                                   # cleared by the read
    comm.moe_combine(win, C, w, Y)                                  # runs (the status is clear), on incomplete windows
    assert comm.moe_status() == 0
    comm.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 0)
    win.zero_()
    comm.moe_dispatch(X, win, C)
    comm.moe_combine(win, C, w, Y)
    assert comm.moe_status() == 0
    assert np.array_equal(win.cpu().view(torch.int16).numpy().view(np.uint16), o.windows_zero_init)
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), o.Y) <= 1
    comm.close()


def test_token_ranges_in_any_partition_give_the_same_bytes():
    dev = torch.device("cuda:0")
    wl = Workload("ranges", 1500, 1000, 32, 4, 6, PREFILL, "uniform", "identity", 88, rank_tokens=(400, 0, 600, 500))
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    comm.moe_plan(PREFILL, idx, wl.T, inp.rank_tok_start)
    for path in PATHS:
        comm.moe_set_option(binding.MOE_OPT_DISPATCH_PATH, path)
        win = torch.zeros((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
        Y = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
        cuts = [0, 1, 2, 700, 700, 1499, 1500]
        for a, b in reversed(list(zip(cuts[:-1], cuts[1:]))):            # any order, empty ranges included
            comm.moe_dispatch_range(X, win, C, a, b)
        for a, b in zip(cuts[:-1], cuts[1:]):
            comm.moe_combine_range(win, C, w, Y, a, b)
        assert comm.moe_status() == 0
        assert np.array_equal(win.cpu().view(torch.int16).numpy().view(np.uint16), o.windows_zero_init)
        assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), o.Y) <= 1
    assert comm.moe_dispatch_range(X, win, C, 5, 1501, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_dispatch_range(X, win, C, 7, 3, check=False) == binding.MOE_ERR_INVALID_ARG
    comm.close()


def test_contexts_of_different_shapes_coexist():
    """Kernel attributes (opt-in shared memory) are per kernel, not per context: creating a small-E
    context after a large-E one must not break the first."""
    dev = torch.device("cuda:0")
    big = Workload("bigE", 600, 64, 4096, 2, 8, PREFILL, "uniform", "identity", 5)       # 128 KB of planner counters
    mid = Workload("midE", 600, 64, 2048, 2, 8, PREFILL, "uniform", "identity", 6)       # 64 KB
    rank_big = Workload("bigE_tiles", 6000, 64, 4096, 2, 8, PREFILL, "uniform", "identity", 7, rank_tokens=(5000, 1000))
    inps = [synth.make_inputs(w) for w in (big, mid, rank_big)]
    comms = [binding.MoeComm(i.wl.T, i.wl.H, i.wl.E, i.wl.R, i.wl.K, dev) for i in inps]   # created in this order
    for inp, comm in zip(inps, comms):                                                      # first one used last-created-first
        p = oracle.plan(inp.topk_idx.numpy(), inp.wl.E, inp.wl.R, inp.rank_tok_start)
        C = int(p.n_recv.max())
        rts = None if inp.wl.rank_tokens is None else inp.rank_tok_start
        g = harness.gpu_run(inp, C, PREFILL, comm=comm)
        harness.assert_parity(g, harness.oracle_run(inp, C), PREFILL)
    for c in comms:
        c.close()


def test_option_values_are_validated():
    dev = torch.device("cuda:0")
    comm = binding.MoeComm(64, 64, 8, 2, 2, dev)
    bad = binding.MOE_ERR_INVALID_ARG
    for opt, good, wrong in [(binding.MOE_OPT_DISPATCH_PATH, [0, 1, 2], [-1, 3]),
                             (binding.MOE_OPT_GRANULE, [0, 1, 1 << 20], [-1, (1 << 20) + 1]),
                             (binding.MOE_OPT_TEST_STARVE_WAIT_MS, [0], [-1, 10001]),
                             (binding.MOE_OPT_OVERLAP, [0, 1], [-1, 2]),
                             (binding.MOE_OPT_EXPERT_ALIGN, [1, 128, 4096], [0, -5, 4097]),
                             (binding.MOE_OPT_CLUSTER_PLAN, [0, 1], [-1, 2]),
                             (binding.MOE_OPT_SLOT_REUSE, [0, 1], [-1, 2])]:
        for v in wrong:
            assert comm.moe_set_option(opt, v, check=False) == bad, (opt, v)
        for v in good:
            assert comm.moe_set_option(opt, v, check=False) == binding.MOE_OK, (opt, v)
    assert comm.moe_set_option(99, 0, check=False) == bad
    comm.close()
