"""Row-wise quantised dispatch on the GPU against the CPU oracle.

Codes are bytes and the scale comes from two IEEE fp32 divisions of the same
operands on both sides, so everything is compared bit for bit: e4m3 code rows,
fp32 scales, and the untouched padding rows / scale slots.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

pytestmark = pytest.mark.gpu

CASES = [
    # name, T, H, E, R, K, schedule, routing, rank_tokens
    ("c2_decode_full", 2048, 7168, 256, 16, 8, DECODE, "uniform", None),
    ("c3_reduced", 2048, 7168, 256, 8, 8, PREFILL, "uniform", None),
    ("mixtral_like", 1024, 4096, 8, 8, 2, PREFILL, "uniform", None),
    ("H16_min", 300, 16, 16, 4, 4, PREFILL, "uniform", None),
    ("ragged_units", 123, 1008, 16, 2, 6, DECODE, "uniform", (23, 100)),
    ("K5_dups_empty_rank", 250, 528, 10, 5, 5, PREFILL, "replace", (1, 100, 49, 0, 100)),
    ("max_row", 64, 16384, 8, 2, 2, DECODE, "uniform", None),
    ("tile_planned_decode", 6000, 64, 16, 2, 2, DECODE, "uniform", (5000, 1000)),
    ("one_row", 2, 512, 4, 2, 2, DECODE, "uniform", None),
    ("K32", 40, 64, 64, 2, 32, DECODE, "uniform", None),
    ("many_rows_per_sm", 20000, 256, 32, 4, 4, PREFILL, "uniform", None),
    # rows at the edges of the register forms: 16 chunks per lane (8 KB), one chunk more, 32 chunks (16 KB), one more
    ("row_8k", 700, 4096, 8, 4, 2, DECODE, "uniform", None),
    ("row_8k_plus", 300, 4096 + 16, 8, 4, 2, DECODE, "uniform", None),
    ("row_16k", 300, 8192, 8, 4, 2, PREFILL, "uniform", None),
    ("row_16k_plus", 200, 8192 + 16, 8, 2, 2, PREFILL, "uniform", None),
    ("row_partial_last_chunk_group", 500, 3600, 16, 4, 4, DECODE, "uniform", None),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_quantised_dispatch_bit_exact(case):
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    wl = Workload(name, T, H, E, R, K, sch, routing, "identity", 5000 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    X = inp.X.clone()
    X[T // 3] = 0                                     # an all-zero row
    X[T // 2, H // 2] = 3.0e4                         # an outlier: the rest of that row lands in the subnormal codes
    X[1, 0] = -0.0
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, E, R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + 2
    _, slots = oracle.slots(idx_np, E, R, p, C, inp.rank_tok_start)
    want_q = np.full((R * C, H), 0xAB, np.uint8)
    want_s = np.full((R * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(X), slots, want_q, want_s, 4) == oracle.OK

    comm = binding.MoeComm(T, H, E, R, K, dev)
    rts = None if per is None else inp.rank_tok_start
    comm.moe_plan(sch, inp.topk_idx.to(dev), T, rts)
    wq = torch.full((R * C, H), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((R * C,), -1.0, dtype=torch.float32, device=dev)
    Xd = X.to(dev)
    for _ in range(2):                                # twice: the second launch starts from the counters the first left
        comm.moe_dispatch_quant(Xd, wq, sc, C)
    assert comm.moe_status() == 0
    assert np.array_equal(wq.cpu().numpy(), want_q)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    # planning folded into the call (the kernel starts behind the planner): the same bytes
    wq2 = torch.full((R * C, H), 0xAB, dtype=torch.uint8, device=dev)
    sc2 = torch.full((R * C,), -1.0, dtype=torch.float32, device=dev)
    for _ in range(2):
        comm.moe_plan_dispatch_quant(sch, inp.topk_idx.to(dev), Xd, wq2, sc2, C, T, rts)
    assert comm.moe_status() == 0
    assert np.array_equal(wq2.cpu().numpy(), want_q)
    assert np.array_equal(sc2.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    if sch == DECODE:                                 # the launch also records delta, like moe_dispatch
        assert np.array_equal(comm.moe_plan_view()["small_off"].cpu().numpy(), p.s)
    # a consumer's view: dequantised rows are within the format's error of the bf16 rows
    deq = wq[torch.from_numpy(slots[:, 0]).to(dev)].view(torch.float8_e4m3fn).float() * \
        sc[torch.from_numpy(slots[:, 0]).to(dev)][:, None]
    xf = X.to(dev).float()
    scale = xf.abs().amax(1) / 448.0
    assert bool(((deq - xf).abs() <= xf.abs() * 2.0 ** -4 * 1.00001 + scale[:, None] * 2.0 ** -10 * 1.00001).all())
    comm.close()


GROUP_CASES = [
    # name, T, H, E, R, K, schedule, routing, rank_tokens  (H % 128 == 0)
    ("c2_decode_full", 2048, 7168, 256, 16, 8, DECODE, "uniform", None),
    ("c3_reduced", 2048, 7168, 256, 8, 8, PREFILL, "uniform", None),
    ("mixtral_like", 1024, 4096, 8, 8, 2, PREFILL, "uniform", None),
    ("one_group", 300, 128, 16, 4, 4, PREFILL, "uniform", None),
    ("odd_groups_half_slab", 123, 128 * 7, 16, 2, 6, DECODE, "uniform", (23, 100)),
    ("K5_dups_empty_rank", 250, 640, 10, 5, 5, PREFILL, "replace", (1, 100, 49, 0, 100)),
    ("max_row", 64, 16384, 8, 2, 2, DECODE, "uniform", None),
    ("tile_planned_decode", 6000, 256, 16, 2, 2, DECODE, "uniform", (5000, 1000)),
    ("K32", 40, 384, 64, 2, 32, DECODE, "uniform", None),
    ("many_rows_per_sm", 20000, 256, 32, 4, 4, PREFILL, "uniform", None),
    ("row_8k_plus_one_group", 300, 4096 + 128, 8, 4, 2, DECODE, "uniform", None),
    ("row_16k", 300, 8192, 8, 4, 2, PREFILL, "uniform", None),
    ("row_16k_plus_one_group", 200, 8192 + 128, 8, 2, 2, PREFILL, "uniform", None),
]


@pytest.mark.parametrize("case", GROUP_CASES, ids=[c[0] for c in GROUP_CASES])
def test_group_quantised_dispatch_bit_exact(case):
    """One scale per 128 elements: codes and all H/128 scales of every window row against the oracle, bit for bit;
    padding rows keep their fill."""
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    G = H // 128
    wl = Workload(name, T, H, E, R, K, sch, routing, "identity", 5100 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    X = inp.X.clone()
    X[T // 3] = 0                                     # an all-zero row: every scale 1
    X[T // 2, H // 2] = 3.0e4                         # an outlier: only its own group is pushed into the small codes
    X[T // 4, :128] = 0                               # an all-zero group in a live row
    X[:, -128:] *= 2.0 ** -9                          # a group far smaller than the others
    X[1, 0] = -0.0
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, E, R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + 2
    _, slots = oracle.slots(idx_np, E, R, p, C, inp.rank_tok_start)
    want_q = np.full((R * C, H), 0xAB, np.uint8)
    want_s = np.full((R * C, G), -1.0, np.float32)
    assert oracle.dispatch_quant_group(synth.bf16_to_u16(X), slots, want_q, want_s, 128, 4) == oracle.OK

    comm = binding.MoeComm(T, H, E, R, K, dev)
    rts = None if per is None else inp.rank_tok_start
    comm.moe_plan(sch, inp.topk_idx.to(dev), T, rts)
    wq = torch.full((R * C, H), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((R * C, G), -1.0, dtype=torch.float32, device=dev)
    Xd = X.to(dev)
    for _ in range(2):                                # twice: the second launch starts from the counters the first left
        comm.moe_dispatch_quant_group(Xd, wq, sc, C)
    assert comm.moe_status() == 0
    assert np.array_equal(wq.cpu().numpy(), want_q)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    # planning folded into the call: the same bytes
    wq2 = torch.full((R * C, H), 0xAB, dtype=torch.uint8, device=dev)
    sc2 = torch.full((R * C, G), -1.0, dtype=torch.float32, device=dev)
    for _ in range(2):
        comm.moe_plan_dispatch_quant_group(sch, inp.topk_idx.to(dev), Xd, wq2, sc2, C, 128, T, rts)
    assert comm.moe_status() == 0
    assert np.array_equal(wq2.cpu().numpy(), want_q)
    assert np.array_equal(sc2.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    # a consumer's view: group by group within the format's error -- the small group keeps its precision
    first = torch.from_numpy(slots[:, 0]).to(dev)
    deq = wq[first].view(torch.float8_e4m3fn).float().view(T, G, 128) * sc[first][:, :, None]
    xf = Xd.float().view(T, G, 128)
    scale = xf.abs().amax(2) / 448.0
    assert bool(((deq - xf).abs() <= xf.abs() * 2.0 ** -4 * 1.00001 + scale[:, :, None] * 2.0 ** -10 * 1.00001).all())
    comm.close()


def test_group_quantised_dispatch_errors():
    dev = torch.device("cuda:0")
    idx = torch.zeros((64, 2), dtype=torch.int32, device=dev)
    comm = binding.MoeComm(64, 192, 8, 2, 2, dev)     # H % 128 != 0
    comm.moe_plan(PREFILL, idx)
    x = torch.zeros((64, 192), dtype=torch.bfloat16, device=dev)
    wq = torch.zeros((2 * 128, 192), dtype=torch.uint8, device=dev)
    sc = torch.zeros((2 * 128, 2), dtype=torch.float32, device=dev)
    assert comm.moe_dispatch_quant_group(x, wq, sc, 128, check=False) == binding.MOE_ERR_INVALID_ARG
    assert comm.moe_plan_dispatch_quant_group(PREFILL, idx, x, wq, sc, 128, check=False) == binding.MOE_ERR_INVALID_ARG
    comm.close()
    comm = binding.MoeComm(64, 256, 8, 2, 2, dev)
    x = torch.ones((64, 256), dtype=torch.bfloat16, device=dev)
    wq = torch.full((2 * 128, 256), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((2 * 128, 2), -1.0, dtype=torch.float32, device=dev)
    assert comm.moe_dispatch_quant_group(x, wq, sc, 128, check=False) == binding.MOE_ERR_NOT_PLANNED
    comm.moe_plan(PREFILL, idx)                        # all 128 branches go to expert 0 of rank 0
    assert comm.moe_dispatch_quant_group(x, wq, sc, 128, group_size=64, check=False) == binding.MOE_ERR_INVALID_ARG
    comm.moe_dispatch_quant_group(x, wq, sc, 127)      # one row short
    assert comm.moe_status() == binding.MOE_ERR_CAPACITY
    assert bool((wq == 0xAB).all()) and bool((sc == -1.0).all())
    comm.moe_dispatch_quant_group(x, wq, sc, 128)
    assert comm.moe_status() == 0
    assert bool((wq[:128] == 0x7E).all()) and bool((sc[:128] == 1.0 / 448.0).all()) and bool((wq[128:] == 0xAB).all())
    assert bool((sc[128:] == -1.0).all())
    comm.close()


def test_quantised_dispatch_errors():
    dev = torch.device("cuda:0")
    comm = binding.MoeComm(64, 24, 8, 2, 2, dev)      # H % 16 != 0
    idx = torch.zeros((64, 2), dtype=torch.int32, device=dev)
    comm.moe_plan(PREFILL, idx)
    x = torch.zeros((64, 24), dtype=torch.bfloat16, device=dev)
    wq = torch.zeros((2 * 128, 24), dtype=torch.uint8, device=dev)
    sc = torch.zeros((2 * 128,), dtype=torch.float32, device=dev)
    assert comm.moe_dispatch_quant(x, wq, sc, 128, check=False) == binding.MOE_ERR_INVALID_ARG
    comm.close()
    comm = binding.MoeComm(64, 32, 8, 2, 2, dev)
    x = torch.ones((64, 32), dtype=torch.bfloat16, device=dev)
    wq = torch.full((2 * 128, 32), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((2 * 128,), -1.0, dtype=torch.float32, device=dev)
    assert comm.moe_dispatch_quant(x, wq, sc, 128, check=False) == binding.MOE_ERR_NOT_PLANNED
    comm.moe_plan(PREFILL, idx)                        # all 128 branches go to expert 0 of rank 0
    comm.moe_dispatch_quant(x, wq, sc, 127)            # one row short
    assert comm.moe_status() == binding.MOE_ERR_CAPACITY
    assert bool((wq == 0xAB).all()) and bool((sc == -1.0).all())
    comm.moe_dispatch_quant(x, wq, sc, 128)
    assert comm.moe_status() == 0
    assert bool((wq[:128] == 0x7E).all()) and bool((sc[:128] == 1.0 / 448.0).all()) and bool((wq[128:] == 0xAB).all())
    comm.close()
