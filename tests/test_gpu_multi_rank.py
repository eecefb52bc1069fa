"""The multi-rank decomposition (moe_layout -> gather counts -> moe_notify -> moe_dispatch_peers ->
experts -> moe_combine_peers) on ONE GPU: every expert-parallel rank gets its own context, its own
token slice and its own window allocation, as R processes on R GPUs would have; the calls run one rank
after the other (they never wait on one another).  The union of the windows and the outputs must be
bit-identical to the oracle's single global result.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth
from paper_2605_06055_b200.synth import DECODE, PREFILL, Workload

import harness

pytestmark = pytest.mark.gpu

CASES = [
    ("decode_like", 1024, 1024, 64, 8, 8, DECODE, "uniform", None),
    ("prefill_ragged", 3000, 512, 32, 4, 4, PREFILL, "uniform", (1000, 0, 1500, 500)),
    ("large_rank_tile_path", 6000, 64, 16, 2, 2, PREFILL, "replace", (5000, 1000)),
    ("large_rank_tile_path_decode", 6000, 64, 16, 2, 2, DECODE, "replace", (5000, 1000)),
    ("generic_k", 500, 264, 12, 3, 3, DECODE, "replace", (100, 150, 250)),
]


@pytest.mark.parametrize("align", [1, 16])
@pytest.mark.parametrize("path", [binding.MOE_DISPATCH_BULK, binding.MOE_DISPATCH_REGISTERS])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_per_rank_contexts_and_separate_windows_reproduce_the_global_result(case, path, align):
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    wl = Workload(name, T, H, E, R, K, sch, routing, "scale", 7000 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    rts = inp.rank_tok_start
    p = oracle.plan(inp.topk_idx.numpy(), E, R, rts, align=align)
    C = int(p.n_recv.max()) + 1
    want = harness.oracle_run(inp, C, align=align)

    idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
    comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
    for c in comms:
        c.moe_set_option(binding.MOE_OPT_DISPATCH_PATH, path)
        c.moe_set_option(binding.MOE_OPT_EXPERT_ALIGN, align)
    # Layout on every rank, then the count "all-gather" (here: rows of one tensor), then Notify on every rank
    counts = torch.full((R, E), -1, dtype=torch.int32, device=dev)
    for r, c in enumerate(comms):
        assert c.moe_dispatch_peers(X[:0], torch.zeros(R, dtype=torch.int64, device=dev), C, check=False) == \
            binding.MOE_ERR_NOT_PLANNED
        c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, counts[r])
    assert np.array_equal(counts.cpu().numpy(), p.M)
    for c in comms:
        c.moe_notify(counts)
    # one window allocation per rank, addressed through a base-pointer table
    windows = [torch.from_numpy(np.full((C, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
               for _ in range(R)]
    bases = torch.tensor([wd.data_ptr() for wd in windows], dtype=torch.int64, device=dev)
    for r, c in enumerate(comms):
        c.moe_dispatch_peers(X[rts[r]:rts[r + 1]].contiguous(), bases, C)
        assert c.moe_status() == 0
        v = c.moe_plan_view()
        assert np.array_equal(v["large_off"].cpu().numpy(), p.o) and np.array_equal(v["n_recv"].cpu().numpy(), p.n_recv)
        assert np.array_equal(v["small_off"].cpu().numpy(), p.s[rts[r]:rts[r + 1]])
    got = torch.cat(windows).cpu().view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want.windows)
    # experts (harness op on the concatenated view), then every rank combines its own tokens from all windows
    allwin = torch.cat(windows)
    harness.gpu_expert_scale(allwin, idx, E, R, C, inp.scale.to(dev), align)
    for d in range(R):
        windows[d].copy_(allwin[d * C:(d + 1) * C])
    Y = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
    for r, c in enumerate(comms):
        y_r = torch.empty((int(rts[r + 1] - rts[r]), H), dtype=torch.bfloat16, device=dev)
        c.moe_combine_peers(bases, C, w[rts[r]:rts[r + 1]].contiguous(), y_r)
        assert c.moe_status() == 0
        Y[rts[r]:rts[r + 1]] = y_r
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), want.Y) <= 1
    for c in comms:
        c.close()


@pytest.mark.parametrize("case", CASES[:3], ids=[c[0] for c in CASES[:3]])
def test_quantised_dispatch_into_per_rank_windows(case):
    """The quantising dispatch in the multi-rank decomposition: every rank quantises its own tokens and
    writes codes and scales into every rank's own allocations; the union equals the oracle's global result."""
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    wl = Workload(name, T, H, E, R, K, sch, routing, "identity", 7100 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    rts = inp.rank_tok_start
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, E, R, rts)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx_np, E, R, p, C, rts)
    want_q = np.full((R * C, H), 0xAB, np.uint8)
    want_s = np.full((R * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), slots, want_q, want_s, 4) == oracle.OK

    idx, X = inp.topk_idx.to(dev), inp.X.to(dev)
    comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
    counts = torch.zeros((R, E), dtype=torch.int32, device=dev)
    for r, c in enumerate(comms):
        c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, counts[r])
    for c in comms:
        c.moe_notify(counts)
    wq = [torch.full((C, H), 0xAB, dtype=torch.uint8, device=dev) for _ in range(R)]
    sc = [torch.full((C,), -1.0, dtype=torch.float32, device=dev) for _ in range(R)]
    q_bases = torch.tensor([t.data_ptr() for t in wq], dtype=torch.int64, device=dev)
    s_bases = torch.tensor([t.data_ptr() for t in sc], dtype=torch.int64, device=dev)
    for r, c in enumerate(comms):
        c.moe_dispatch_quant_peers(X[rts[r]:rts[r + 1]].contiguous(), q_bases, s_bases, C)
        assert c.moe_status() == 0
    assert np.array_equal(torch.cat(wq).cpu().numpy(), want_q)
    assert np.array_equal(torch.cat(sc).cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    for c in comms:
        c.close()


# ------------------------------------------------------------------ two processes, windows shared over CUDA IPC
def _ipc_rank(rank, world, port, q_to, results):
    """One expert-parallel rank as its own process on the one GPU: its window lives in its own
    allocation, the other rank's window is mapped in over CUDA IPC, counts travel over a gloo group,
    phases are ordered by host barriers (no kernel waits on another process's kernel)."""
    import os
    import torch.distributed as dist
    from paper_2605_06055_b200 import ep
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    try:
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        T, H, E, K = 600, 512, 16, 4
        wl = Workload("ipc", T, H, E, world, K, DECODE, "uniform", "identity", 7300, rank_tokens=(250, 350))
        inp = synth.make_inputs(wl)
        rts = inp.rank_tok_start
        lo, hi = int(rts[rank]), int(rts[rank + 1])
        me = ep.EpRank(hi - lo, H, E, K, dev)
        me.plan(DECODE, inp.topk_idx[lo:hi].contiguous().to(dev))
        C = int(me.comm.moe_plan_view()["n_recv"].max().item()) + 1
        mine = torch.from_numpy(np.full((C, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
        q_to[1 - rank].put(mine)                       # the other process maps this allocation (CUDA IPC)
        other = q_to[rank].get(timeout=60)
        wins = [mine, other] if rank == 0 else [other, mine]
        bases = torch.tensor([w.data_ptr() for w in wins], dtype=torch.int64, device=dev)
        me.dispatch(inp.X[lo:hi].contiguous().to(dev), bases, C)
        y = torch.empty((hi - lo, H), dtype=torch.bfloat16, device=dev)
        me.combine(bases, C, inp.topk_w[lo:hi].contiguous().to(dev), y)
        st = me.status()
        # the quantising dispatch into per-process code windows and scale tensors, mapped the same way
        my_q = torch.full((C, H), 0xAB, dtype=torch.uint8, device=dev)
        my_s = torch.full((C,), -1.0, dtype=torch.float32, device=dev)
        q_to[1 - rank].put((my_q, my_s))
        other_q, other_s = q_to[rank].get(timeout=60)
        qs = [my_q, other_q] if rank == 0 else [other_q, my_q]
        ss = [my_s, other_s] if rank == 0 else [other_s, my_s]
        q_bases = torch.tensor([t.data_ptr() for t in qs], dtype=torch.int64, device=dev)
        s_bases = torch.tensor([t.data_ptr() for t in ss], dtype=torch.int64, device=dev)
        me.dispatch_quant(inp.X[lo:hi].contiguous().to(dev), q_bases, s_bases, C)
        st = st or me.status()
        dist.barrier()                                 # nobody frees a window another rank may still read
        results[rank] = ("ok", st, C, mine.cpu().view(torch.int16).numpy().view(np.uint16).copy(),
                         y.cpu().view(torch.int16).numpy().view(np.uint16).copy(), my_q.cpu().numpy().copy(),
                         my_s.cpu().numpy().copy())
        dist.barrier()
        dist.destroy_process_group()
    except Exception as exc:                           # reported to the parent, which decides between skip and fail
        results[rank] = ("error", repr(exc))


def test_two_processes_exchange_rows_through_ipc_mapped_windows():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    world = 2
    with ctx.Manager() as m:
        results = m.dict()
        q_to = [ctx.Queue(), ctx.Queue()]
        procs = [ctx.Process(target=_ipc_rank, args=(r, world, 35000 + os.getpid() % 2000, q_to, results))
                 for r in range(world)]
        for p_ in procs:
            p_.start()
        for p_ in procs:
            p_.join(timeout=180)
        alive = [p_ for p_ in procs if p_.is_alive()]
        for p_ in alive:
            p_.terminate()
        assert not alive, "a rank did not finish"
        res = dict(results)
    errors = [v for v in res.values() if v[0] == "error"]
    if errors and any("ipc" in e[1].lower() or "not supported" in e[1].lower() for e in errors):
        pytest.skip("CUDA IPC is not available here: " + errors[0][1])
    assert not errors and len(res) == world, res
    T, H, E, K = 600, 512, 16, 4
    wl = Workload("ipc", T, H, E, world, K, DECODE, "uniform", "identity", 7300, rank_tokens=(250, 350))
    inp = synth.make_inputs(wl)
    C = res[0][2]
    assert res[1][2] == C
    want = harness.oracle_run(inp, C)
    rts = inp.rank_tok_start
    want_q = np.full((world * C, H), 0xAB, np.uint8)
    want_s = np.full((world * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), want.slots, want_q, want_s, 2) == oracle.OK
    for r in range(world):
        _, st, _, win, y, q, sc = res[r]
        assert st == 0
        assert np.array_equal(win, want.windows[r * C:(r + 1) * C])            # rows from both processes, bit-exact
        assert harness.max_ulp_diff(y, want.Y[int(rts[r]):int(rts[r + 1])]) <= 1
        assert np.array_equal(q, want_q[r * C:(r + 1) * C])
        assert np.array_equal(sc.view(np.uint32), want_s[r * C:(r + 1) * C].view(np.uint32))
