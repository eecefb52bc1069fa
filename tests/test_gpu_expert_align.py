"""GPU parity of the aligned window layout (MOE_OPT_EXPERT_ALIGN): every expert's run starts on a
multiple of A rows of its window.  Offsets, slots, window bytes (padding rows keep their canaries)
and expert row ranges are bit-exact against the oracle; combine within 1 bf16 ulp."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu

CASES = [
    # name, T, H, E, R, K, routing, rank_tokens
    ("tiny", 64, 64, 8, 2, 2, "uniform", None),
    ("compact_planner", 1000, 256, 32, 4, 8, "uniform", (0, 517, 0, 483)),
    ("tile_planner", 6000, 32, 16, 2, 2, "uniform", (5000, 1000)),
    ("dups_generic_K", 250, 520, 10, 5, 5, "replace", (1, 100, 49, 0, 100)),
    ("empty_experts", 40, 64, 64, 2, 4, "uniform", None),          # most experts get no row: padding of 0 is 0
    ("direct_notify_path", 4096, 64, 4096, 256, 8, "uniform", None),   # R*E above the staged Notify limit
]


@pytest.mark.parametrize("align", [8, 128])
@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_aligned_layout_matches_the_oracle(case, schedule, align):
    name, T, H, E, R, K, routing, rank_tokens = case
    wl = Workload(name, T, H, E, R, K, schedule, routing, "scale", 5100 + T, rank_tokens=rank_tokens)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), E, R, inp.rank_tok_start, align=align)
    C = int(p.n_recv.max())                       # exactly the padded need
    o = harness.oracle_run(inp, C, align=align)
    for path in (binding.MOE_DISPATCH_BULK, binding.MOE_DISPATCH_REGISTERS):
        g = harness.gpu_run(inp, C, schedule, dispatch_path=path, align=align)
        harness.assert_parity(g, o, schedule, align=align)
        assert (g.expert_start % C % align == 0).all()


def test_config3_shape_with_128_row_expert_tiles():
    wl = Workload("c3_reduced_aligned", 8 * 517, 7168, 256, 8, 8, PREFILL, "uniform", "identity", 3003)
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, align=128)
    C = int(p.n_recv.max())
    o = harness.oracle_run(inp, C, align=128)
    g = harness.gpu_run(inp, C, align=128)
    harness.assert_parity(g, o, wl.schedule, align=128)


def test_alignment_changes_need_a_new_plan_and_capacity_counts_padding():
    dev = torch.device("cuda:0")
    T, H, E, R, K = 256, 64, 16, 4, 2
    wl = Workload("align_err", T, H, E, R, K, PREFILL, "uniform", "identity", 8)
    inp = synth.make_inputs(wl)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    comm = binding.MoeComm(T, H, E, R, K, dev)
    packed = oracle.plan(inp.topk_idx.numpy(), E, R)
    padded = oracle.plan(inp.topk_idx.numpy(), E, R, align=32)
    C_packed, C_padded = int(packed.n_recv.max()), int(padded.n_recv.max())
    assert C_padded > C_packed
    win = torch.from_numpy(np.full((R * C_padded, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    comm.moe_plan(PREFILL, idx)
    assert comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, 0, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, 5000, check=False) == binding.MOE_ERR_INVALID_ARG
    comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, 32)
    assert comm.moe_dispatch(X, win, C_padded, check=False) == binding.MOE_ERR_NOT_PLANNED   # the old plan is gone
    comm.moe_plan(PREFILL, idx)
    comm.moe_dispatch(X, win, C_packed)            # enough for the rows, not for the padded layout
    assert comm.moe_status() == binding.MOE_ERR_CAPACITY
    assert bool((win.view(torch.int16) == np.int16(harness.CANARY)).all())
    comm.moe_dispatch(X, win, C_padded)
    Y = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    comm.moe_combine(win, C_padded, w, Y)
    assert comm.moe_status() == 0
    assert np.array_equal(comm.moe_plan_view()["n_recv"].cpu().numpy(), padded.n_recv)
    assert np.array_equal(Y.cpu().view(torch.int16).numpy().view(np.uint16), synth.bf16_to_u16(inp.X))
    comm.close()


@pytest.mark.parametrize("align,tile_rows", [(1, 16), (128, 128), (8, 5), (1, 100000)])
@pytest.mark.parametrize("schedule", [PREFILL, DECODE])
def test_expert_tile_list_matches_the_oracle(schedule, align, tile_rows):
    dev = torch.device("cuda:0")
    for name, T, H, E, R, K, routing, per in CASES[:5]:
        wl = Workload(name, T, H, E, R, K, schedule, routing, "identity", 5200 + T, rank_tokens=per)
        inp = synth.make_inputs(wl)
        p = oracle.plan(inp.topk_idx.numpy(), E, R, inp.rank_tok_start, align=align)
        C = int(p.n_recv.max()) + 1
        bound = T * K // tile_rows + E
        st, w_e, w_row, w_valid, w_n = oracle.expert_tiles(E, R, C, p.n_exp, tile_rows, bound, align=align)
        assert st == oracle.OK and w_n <= bound
        comm = binding.MoeComm(max(T, 1), H, E, R, K, dev)
        comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, align)
        rts = None if per is None else inp.rank_tok_start
        comm.moe_plan(schedule, inp.topk_idx.to(dev), T, rts)
        t_e = torch.full((bound,), -1, dtype=torch.int32, device=dev)
        t_row = torch.full((bound,), -1, dtype=torch.int64, device=dev)
        t_valid = torch.full((bound,), -1, dtype=torch.int32, device=dev)
        n = torch.full((1,), -1, dtype=torch.int32, device=dev)
        comm.moe_expert_tiles(C, tile_rows, t_e, t_row, t_valid, n)
        assert comm.moe_status() == 0
        assert int(n.item()) == w_n
        assert np.array_equal(t_e.cpu().numpy(), w_e) and np.array_equal(t_row.cpu().numpy(), w_row)
        assert np.array_equal(t_valid.cpu().numpy(), w_valid)
        if align == tile_rows:
            assert ((t_row[:w_n] % C) % tile_rows == 0).all()          # tiles start on tile boundaries of their window
        # a buffer that is too short: the count is the full one, nothing is written beyond the buffer
        if w_n > 2:
            short = torch.full((2,), -1, dtype=torch.int32, device=dev)
            comm.moe_expert_tiles(C, tile_rows, short, t_row[:2].clone(), t_valid[:2].clone(), n)
            assert comm.moe_status() == 0 and int(n.item()) == w_n and np.array_equal(short.cpu().numpy(), w_e[:2])
        comm.close()


def test_an_expert_op_driven_by_the_tile_list_gives_the_oracle_result():
    """End to end with the expert side consuming the windows in place through the tile list alone
    (no routing indexes, no counts): dispatch, scale every tile's rows by its expert's factor, combine."""
    dev = torch.device("cuda:0")
    tile = 64
    wl = Workload("tiles_e2e", 3000, 512, 32, 4, 6, DECODE, "uniform", "scale", 5300, rank_tokens=(900, 0, 1300, 800))
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start, align=tile)
    C = int(p.n_recv.max())
    want = harness.oracle_run(inp, C, align=tile)
    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    comm.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, tile)
    idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
    win = torch.from_numpy(np.full((wl.R * C, wl.H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    comm.moe_plan_dispatch(wl.schedule, idx, X, win, C, wl.T, inp.rank_tok_start)
    bound = wl.T * wl.K // tile + wl.E
    t_e = torch.empty(bound, dtype=torch.int32, device=dev)
    t_row = torch.empty(bound, dtype=torch.int64, device=dev)
    t_valid = torch.empty(bound, dtype=torch.int32, device=dev)
    n = torch.empty(1, dtype=torch.int32, device=dev)
    comm.moe_expert_tiles(C, tile, t_e, t_row, t_valid, n)
    assert comm.moe_status() == 0
    k = int(n.item())
    assert np.array_equal(win.cpu().view(torch.int16).numpy().view(np.uint16), want.windows)
    # the stand-in expert op, tile by tile (harness code): rows [row, row + valid) of a tile belong to one expert
    valid = t_valid[:k].long()
    first = torch.repeat_interleave(t_row[:k], valid)
    within = torch.arange(int(valid.sum()), device=dev) - torch.repeat_interleave(torch.cumsum(valid, 0) - valid, valid)
    rows = first + within
    factor = torch.repeat_interleave(inp.scale.to(dev)[t_e[:k].long()], valid)
    assert rows.numel() == wl.T * wl.K and (t_row[:k] % C % tile == 0).all()
    win[rows] = win[rows] * factor[:, None]
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    comm.moe_combine(win, C, w, Y)
    assert comm.moe_status() == 0
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), want.Y) <= 1
    comm.close()
