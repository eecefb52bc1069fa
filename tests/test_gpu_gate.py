"""Top-k gating on the GPU (stand-alone and fused with the planner) against the CPU oracle.

Indexes are compared bit for bit.  Weights are fp32 softmax values whose exponentials come from two
different libms (device expf: <= 2 ulp, host expf: <= 1 ulp: 3 ulp = 6 half-ulps between the two sides' terms),
followed on each side by a K-term fp32 sum in ascending j -- each of its K-1 additions rounds by up to half an
ulp of the running sum, and when many selected logits are equal those roundings all fall the same way, while a
one-ulp difference in the addend can turn them the other way on the other side: up to 2(K-1) half-ulps between
the sides -- and a division (one half-ulp each side).  Relative budget: (2K + 8) * 2^-24, e.g. 1.4e-6 at K = 8,
4.3e-6 at K = 32 (a seeded case with K = 28 and two thirds of the logits equal reaches 2.3e-6).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL

pytestmark = pytest.mark.gpu


def gate_rtol(K: int) -> float:
    return (2 * K + 8) * 2.0 ** -24


def logits_for(T, E, seed, ties=False):
    g = torch.Generator().manual_seed(seed)
    l = torch.randn(T, E, generator=g) * 3
    if ties:
        l = torch.round(l)            # many equal logits: the lower index must win
    return l.contiguous()


@pytest.mark.parametrize("T,E,K,ties", [(256, 16, 2, False), (2048, 256, 8, False), (500, 256, 8, True),
                                        (77, 8, 8, True), (300, 40, 1, False), (64, 4096, 32, False),
                                        (1000, 1000, 6, True),
                                        # every register form, full and partly filled lanes, K up to the limit
                                        (333, 200, 8, True), (333, 40, 8, True), (257, 96, 4, True),
                                        (129, 250, 8, True), (200, 512, 8, True), (96, 1024, 32, True),
                                        (100, 32, 32, True), (5000, 256, 8, "few"), (300, 128, 32, "few"),
                                        (64, 256, 8, "zeros"),
                                        # batches large enough for two tokens per warp: an odd token count, ties,
                                        # every long-row form, K at the limit of that path and beyond it
                                        (6001, 256, 8, False), (5000, 128, 8, True), (4097, 512, 16, True),
                                        (3000, 1024, 8, False), (3001, 96, 4, True), (2600, 256, 17, True),
                                        (4000, 256, 8, "zeros")])
def test_gate_topk_kernel(T, E, K, ties):
    dev = torch.device("cuda:0")
    l = logits_for(T, E, T + E, ties is True)
    if ties == "few":       # three distinct values: nearly every selection is decided by the index, and lanes
        l = torch.round(l / 6)   # are popped many times over (the cache rebuild runs in most rounds)
    if ties == "zeros":     # -0 and +0 are equal: the lower index wins whatever the sign
        l = torch.zeros(T, E)
        l[torch.rand(T, E, generator=torch.Generator().manual_seed(3)) < 0.5] = -0.0
        l[:, ::7] = -1.0
    st, want_idx, want_w = oracle.gate_topk(l.numpy(), K)
    assert st == oracle.OK
    # two guard rows behind the outputs: an odd token count must not be rounded up to a pair
    idx_all = torch.full((T + 2, K), -1, dtype=torch.int32, device=dev)
    w_all = torch.full((T + 2, K), -1.0, dtype=torch.float32, device=dev)
    idx, w = idx_all[:T], w_all[:T]
    assert binding.moe_gate_topk(l.to(dev), K, idx, w) == binding.MOE_OK
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.allclose(w.cpu().numpy(), want_w, rtol=gate_rtol(K), atol=1e-12)
    assert bool((idx_all[T:] == -1).all()) and bool((w_all[T:] == -1.0).all())


@pytest.mark.parametrize("case", [
    ("decode_c2_fused", 2048, 256, 16, 8, DECODE, None),
    ("prefill_small_fused", 1024, 64, 8, 4, PREFILL, None),
    ("fused_ragged_empty_rank", 900, 32, 4, 6, DECODE, (400, 0, 137, 363)),
    ("big_E_fused_8_warps", 256, 1024, 2, 8, DECODE, None),
    ("unfused_large_ranks", 16384, 256, 2, 8, PREFILL, None),
    ("unfused_large_E", 512, 4096, 4, 8, DECODE, None),
], ids=lambda c: c[0])
def test_gate_plan_matches_oracle_gate_then_oracle_plan(case):
    name, T, E, R, K, sch, per = case
    dev = torch.device("cuda:0")
    l = logits_for(T, E, T * 7 + E, ties=(T % 2 == 0))
    st, want_idx, want_w = oracle.gate_topk(l.numpy(), K)
    rts = None if per is None else np.concatenate([[0], np.cumsum(per)]).astype(np.int32)
    p = oracle.plan(want_idx, E, R, rts)
    assert p.status == oracle.OK
    C = int(p.n_recv.max()) + 1
    _, want_slots = oracle.slots(want_idx, E, R, p, C, rts)

    comm = binding.MoeComm(T, 64, E, R, K, dev)
    idx = torch.full((T, K), -1, dtype=torch.int32, device=dev)
    w = torch.full((T, K), -1.0, dtype=torch.float32, device=dev)
    comm.moe_gate_plan(sch, l.to(dev), idx, w, T, rts)
    slots = torch.empty((T, K), dtype=torch.int32, device=dev)
    comm.moe_slots(C, slots)
    assert comm.moe_status() == 0
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.allclose(w.cpu().numpy(), want_w, rtol=gate_rtol(K), atol=1e-12)
    assert np.array_equal(slots.cpu().numpy().astype(np.int64), want_slots)
    v = comm.moe_plan_view()
    assert np.array_equal(v["large_off"].cpu().numpy(), p.o) and np.array_equal(v["n_recv"].cpu().numpy(), p.n_recv)
    if sch == PREFILL:
        assert np.array_equal(v["counts"].cpu().numpy(), p.M) and np.array_equal(v["small_off"].cpu().numpy(), p.s)
    # the indexes and weights it wrote drive the rest of the path: identity experts give X back
    x = torch.randn(T, 64, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16).to(dev)
    win = torch.zeros((R * C, 64), dtype=torch.bfloat16, device=dev)
    y = torch.empty_like(x)
    comm.moe_dispatch(x, win, C)
    comm.moe_combine(win, C, w, y)
    assert comm.moe_status() == 0
    assert torch.equal(y.view(torch.int16) & 0x7FFF, x.view(torch.int16) & 0x7FFF)
    # the same front of the layer as ONE call (gate, plan and dispatch chained), several times with nothing
    # synchronised in between: same indexes, same window bytes as the separate calls just made
    win_sep = win.clone()
    for _ in range(3):
        idx.fill_(-1)
        w.fill_(-1.0)
        win.zero_()
        comm.moe_gate_plan_dispatch(sch, l.to(dev), idx, w, x, win, C, T, rts)
        comm.moe_combine(win, C, w, y)
    assert comm.moe_status() == 0
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.allclose(w.cpu().numpy(), want_w, rtol=gate_rtol(K), atol=1e-12)
    assert torch.equal(win.view(torch.int16), win_sep.view(torch.int16))
    assert torch.equal(y.view(torch.int16) & 0x7FFF, x.view(torch.int16) & 0x7FFF)
    comm.close()


def test_gate_rows_that_do_not_start_on_16_bytes():
    """The 16-byte row loads need an aligned row; any other pointer or row length takes scalar loads."""
    dev = torch.device("cuda:0")
    for T, E, K in ((300, 256, 8), (3001, 256, 8)):
        _unaligned_rows(dev, T, E, K)


def _unaligned_rows(dev, T, E, K):
    l = logits_for(T, E, 99, True)
    st, want_idx, want_w = oracle.gate_topk(l.numpy(), K)
    buf = torch.zeros(T * E + 3, dtype=torch.float32, device=dev)
    for off in (1, 2, 3):
        shifted = buf[off:off + T * E].view(T, E)
        shifted.copy_(l)
        idx = torch.full((T, K), -1, dtype=torch.int32, device=dev)
        w = torch.full((T, K), -1.0, dtype=torch.float32, device=dev)
        assert binding.moe_gate_topk(shifted, K, idx, w) == binding.MOE_OK
        torch.cuda.synchronize()
        assert np.array_equal(idx.cpu().numpy(), want_idx)
        assert np.allclose(w.cpu().numpy(), want_w, rtol=gate_rtol(K), atol=1e-12)


def test_gate_argument_checks():
    dev = torch.device("cuda:0")
    l = torch.zeros((4, 8), device=dev)
    idx = torch.zeros((4, 9), dtype=torch.int32, device=dev)
    w = torch.zeros((4, 9), device=dev)
    assert binding.moe_gate_topk(l, 9, idx, w) == binding.MOE_ERR_INVALID_ARG      # K > E
