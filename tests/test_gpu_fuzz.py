"""Seeded random shapes through the whole path on the GPU against the oracle: every integer, every
window byte (canaries included) and the combined rows (<= 1 bf16 ulp), for random token counts,
hidden sizes, expert / rank / top-k counts, ragged rank maps (empty ranks included), both
schedules, both dispatch kernels, duplicate experts within a token, several work-item sizes and
expert alignments."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu


def random_workload(rng, i):
    R = int(rng.choice([1, 2, 3, 4, 8, 16]))
    E = R * int(rng.choice([1, 2, 3, 8, 32]))
    K = int(rng.integers(1, min(E, 12) + 1))
    replace = bool(rng.integers(0, 2))
    if replace:
        K = int(rng.integers(1, 13))
    H = 8 * int(rng.choice([1, 2, 31, 32, 33, 64, 100, 128, 257, 512, 896]))
    T = int(rng.choice([1, 2, 7, 33, 100, 257, 600, 1500, 2600]))
    cuts = np.sort(rng.integers(0, T + 1, R - 1))
    per = tuple(int(x) for x in np.diff(np.concatenate([[0], cuts, [T]])))
    sch = PREFILL if rng.integers(0, 2) else DECODE
    return Workload(f"fuzz{i}", T, H, E, R, K, sch, "replace" if replace else "uniform", "scale", 31000 + i,
                    rank_tokens=per)


N_SHAPES = int(os.environ.get("MOE_FUZZ_SHAPES", "48"))     # a soak run sets this to hundreds


@pytest.mark.parametrize("i", range(N_SHAPES))
def test_random_shape(i):
    rng = np.random.default_rng(77000 + i)
    wl = random_workload(rng, i)
    align = int(rng.choice([1, 1, 4, 16, 128]))
    granule = int(rng.choice([0, 0, 0, 1, 3, 7]))
    path = binding.MOE_DISPATCH_BULK if rng.integers(0, 2) else binding.MOE_DISPATCH_REGISTERS
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start, align=align)
    assert p.status == oracle.OK
    C = int(p.n_recv.max()) + int(rng.integers(0, 3))
    o = harness.oracle_run(inp, C, align=align)
    g = harness.gpu_run(inp, C, wl.schedule, dispatch_path=path, granule=granule, align=align)
    harness.assert_parity(g, o, wl.schedule, align=align)


@pytest.mark.parametrize("i", range(max(24, N_SHAPES // 4)))
def test_random_shape_many_ranks_and_high_degrees(i):
    """More ranks than a thread-block cluster holds (the planners' Notify step runs as a launch of its own) and
    degrees up to the maximum (the combine forms with spare branches)."""
    rng = np.random.default_rng(99000 + i)
    R = int(rng.choice([24, 32, 48, 64, 256]))
    E = R * int(rng.choice([1, 2, 4]))
    K = int(rng.integers(1, min(E, 32) + 1))
    H = 8 * int(rng.choice([1, 17, 32, 64, 129, 512]))
    T = int(rng.choice([1, 50, 257, 1000, 3000, 9000]))
    cuts = np.sort(rng.integers(0, T + 1, R - 1))
    per = tuple(int(x) for x in np.diff(np.concatenate([[0], cuts, [T]])))
    sch = PREFILL if rng.integers(0, 2) else DECODE
    wl = Workload(f"wide{i}", T, H, E, R, K, sch, "uniform", "scale", 41000 + i, rank_tokens=per)
    align = int(rng.choice([1, 1, 8]))
    inp = synth.make_inputs(wl)
    p = oracle.plan(inp.topk_idx.numpy(), wl.E, wl.R, inp.rank_tok_start, align=align)
    assert p.status == oracle.OK
    C = int(p.n_recv.max()) + int(rng.integers(0, 3))
    o = harness.oracle_run(inp, C, align=align)
    g = harness.gpu_run(inp, C, wl.schedule, align=align)
    harness.assert_parity(g, o, wl.schedule, align=align)


@pytest.mark.parametrize("i", range(max(12, N_SHAPES // 4)))
def test_random_shape_fused_call_and_quantised_dispatch(i):
    rng = np.random.default_rng(88000 + i)
    wl = random_workload(rng, 100 + i)
    if wl.H % 16:
        wl = Workload(wl.name, wl.T, wl.H + 8, wl.E, wl.R, wl.K, wl.schedule, wl.routing, "identity", wl.seed,
                      rank_tokens=wl.rank_tokens)
    dev = torch.device("cuda:0")
    inp = synth.make_inputs(wl)
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, wl.E, wl.R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx_np, wl.E, wl.R, p, C, inp.rank_tok_start)
    want = np.full((wl.R * C, wl.H), harness.CANARY, np.uint16)
    assert oracle.dispatch(synth.bf16_to_u16(inp.X), slots, want) == oracle.OK
    want_q = np.full((wl.R * C, wl.H), 0xAB, np.uint8)
    want_s = np.full((wl.R * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), slots, want_q, want_s, 4) == oracle.OK

    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx = inp.X.to(dev), inp.topk_idx.to(dev)
    win = torch.from_numpy(np.full((wl.R * C, wl.H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    wq = torch.full((wl.R * C, wl.H), 0xAB, dtype=torch.uint8, device=dev)
    sc = torch.full((wl.R * C,), -1.0, dtype=torch.float32, device=dev)
    comm.moe_plan_dispatch(wl.schedule, idx, X, win, C, wl.T, inp.rank_tok_start)
    comm.moe_dispatch_quant(X, wq, sc, C)
    assert comm.moe_status() == 0
    assert np.array_equal(win.cpu().view(torch.int16).numpy().view(np.uint16), want)
    assert np.array_equal(wq.cpu().numpy(), want_q)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    comm.close()


@pytest.mark.parametrize("i", range(max(16, N_SHAPES // 3)))
def test_random_quantised_dispatch_shape(i):
    """Row lengths on both sides of every kernel form of the quantising dispatch (16 / 32 chunks per lane in
    registers, the two-pass form beyond 16 KB, whole and partial 512-byte slabs), batch sizes on both sides of the
    large-job rule, one scale per row and one per 128 elements: codes and scales bit-exact, padding untouched."""
    rng = np.random.default_rng(99000 + i)
    R = int(rng.choice([1, 2, 4, 8]))
    E = R * int(rng.choice([1, 2, 8]))
    K = int(rng.integers(1, min(E, 8) + 1))
    H = 128 * int(rng.choice([1, 2, 3, 7, 16, 28, 31, 32, 33, 56, 63, 64, 65, 100, 128]))
    # few long rows, many short ones: the largest cases stay near 100 MB of rows
    T = int(rng.choice([1, 5, 40, 300, 1500] if H > 4096 else [1, 5, 40, 300, 1500, 6000, 20000 if H <= 512 else 9000]))
    cuts = np.sort(rng.integers(0, T + 1, R - 1))
    per = tuple(int(x) for x in np.diff(np.concatenate([[0], cuts, [T]])))
    sch = PREFILL if rng.integers(0, 2) else DECODE
    wl = Workload(f"qfuzz{i}", T, H, E, R, K, sch, "replace" if rng.integers(0, 2) else "uniform", "identity", 41000 + i,
                  rank_tokens=per)
    dev = torch.device("cuda:0")
    inp = synth.make_inputs(wl)
    X = inp.X.clone()
    X[rng.integers(0, T)] = 0                                  # an all-zero row
    X[rng.integers(0, T), rng.integers(0, H)] = 2.0e4          # an outlier
    X[:, :128] *= 2.0 ** -7                                    # a group far smaller than the others
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, E, R, inp.rank_tok_start)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx_np, E, R, p, C, inp.rank_tok_start)
    x_u16 = synth.bf16_to_u16(X)
    comm = binding.MoeComm(T, H, E, R, K, dev)
    Xd, idx = X.to(dev), inp.topk_idx.to(dev)
    comm.moe_plan(sch, idx, T, inp.rank_tok_start)
    for group in (0, 128):
        G = 1 if group == 0 else H // group
        want_q = np.full((R * C, H), 0xAB, np.uint8)
        want_s = np.full((R * C, G), -1.0, np.float32)
        wq = torch.full((R * C, H), 0xAB, dtype=torch.uint8, device=dev)
        sc = torch.full((R * C, G), -1.0, dtype=torch.float32, device=dev)
        if group == 0:
            assert oracle.dispatch_quant(x_u16, slots, want_q, want_s.reshape(-1), 4) == oracle.OK
            comm.moe_dispatch_quant(Xd, wq, sc.view(-1), C)
        else:
            assert oracle.dispatch_quant_group(x_u16, slots, want_q, want_s, group, 4) == oracle.OK
            comm.moe_dispatch_quant_group(Xd, wq, sc, C, group)
        assert comm.moe_status() == 0
        assert np.array_equal(wq.cpu().numpy(), want_q), (group, T, H, K)
        assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_s.view(np.uint32)), (group, T, H, K)
    comm.close()


@pytest.mark.parametrize("i", range(max(16, N_SHAPES // 3)))
def test_random_gate_shape(i):
    """Top-k gating on random row lengths (every register form and the shared-memory form), top-k degrees up to
    the limit, batches on both sides of the two-tokens-per-warp switch, with and without many equal logits, rows
    that do and do not start on 16 bytes: indexes bit for bit, weights within the softmax budget."""
    rng = np.random.default_rng(99000 + i)
    E = int(rng.choice([1, 2, 7, 8, 31, 32, 33, 60, 64, 100, 128, 129, 200, 256, 257, 384, 512, 700, 1024, 1025, 2000]))
    K = int(rng.integers(1, min(E, 32) + 1))
    T = int(rng.choice([1, 2, 3, 50, 333, 1000, 2368, 2369, 3001, 5000]))
    kind = int(rng.integers(0, 4))
    g = torch.Generator().manual_seed(99000 + i)
    l = torch.randn(T, E, generator=g) * 3
    if kind == 1:
        l = torch.round(l)                 # many equal logits
    elif kind == 2:
        l = torch.round(l / 6)             # three distinct values: the index decides nearly everything
    elif kind == 3:
        l[:, ::3] = -0.0                   # signed zeros among ordinary values
        l[:, 1::3] = 0.0
    st, want_idx, want_w = oracle.gate_topk(l.contiguous().numpy(), K)
    assert st == oracle.OK
    dev = torch.device("cuda:0")
    off = int(rng.integers(0, 4))          # 0: aligned rows (if E % 4 == 0); else rows start off 16 bytes
    buf = torch.zeros(T * E + 3, dtype=torch.float32, device=dev)
    logits = buf[off:off + T * E].view(T, E)
    logits.copy_(l)
    idx = torch.full((T, K), -1, dtype=torch.int32, device=dev)
    w = torch.full((T, K), -1.0, dtype=torch.float32, device=dev)
    assert binding.moe_gate_topk(logits, K, idx, w) == binding.MOE_OK
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), want_idx), (E, K, T, kind, off)
    rtol = (2 * K + 8) * 2.0 ** -24        # libm difference of the terms, two K-term sums, two divisions (see test_gpu_gate.py)
    assert np.allclose(w.cpu().numpy(), want_w, rtol=rtol, atol=1e-12), (E, K, T, kind, off)
