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
    # Notify from the gathered counts at the ends of its range: 2048 experts per window, and 64 windows of two
    ("many_experts_per_rank", 400, 64, 4096, 2, 8, PREFILL, "uniform", (150, 250)),
    ("many_ranks", 640, 64, 128, 64, 4, DECODE, "uniform", None),
    ("k11_masked_combine", 300, 512, 32, 4, 11, PREFILL, "uniform", (100, 50, 0, 150)),
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
        # the rows this rank's dispatch recorded for its combine: the global numbering d*C + row in window d
        if rts[r + 1] > rts[r]:
            assert v["rows_capacity"] == C
            assert np.array_equal(v["rows"].cpu().numpy().astype(np.int64), want.slots[rts[r]:rts[r + 1]])
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


def test_installed_address_table_and_generation_stamp_in_one_process():
    """moe_peers_set / moe_dispatch_cached / moe_combine_cached with every rank a context of this process: the
    installed table gives the same bytes as passing the table with every call; a stamp that does not match the
    installed generations is refused before anything is enqueued; a re-installed table takes effect."""
    name, T, H, E, R, K, sch, routing, per = CASES[1]
    dev = torch.device("cuda:0")
    wl = Workload(name, T, H, E, R, K, sch, routing, "scale", 7000 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    rts = inp.rank_tok_start
    p = oracle.plan(inp.topk_idx.numpy(), E, R, rts)
    C = int(p.n_recv.max()) + 1
    want = harness.oracle_run(inp, C)
    idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
    comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
    counts = torch.zeros((R, E), dtype=torch.int32, device=dev)
    for r, c in enumerate(comms):
        c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, counts[r])
    for c in comms:
        c.moe_notify(counts)
    fill = lambda: torch.from_numpy(np.full((C, H), harness.CANARY, np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    u16 = lambda ts: torch.cat(ts).cpu().view(torch.int16).numpy().view(np.uint16)
    windows = [fill() for _ in range(R)]
    gens = np.arange(1, R + 1, dtype=np.int32)
    xs = [X[rts[r]:rts[r + 1]].contiguous() for r in range(R)]
    for r, c in enumerate(comms):
        assert c.moe_dispatch_cached(xs[r], gens, check=False) == binding.MOE_ERR_STALE_PEERS     # nothing installed
        assert c.moe_peers_check(gens) == binding.MOE_ERR_STALE_PEERS
        c.moe_peers_set([t.data_ptr() for t in windows], gens, C)
        assert c.moe_peers_check(gens) == binding.MOE_OK
        stale = gens.copy()
        stale[(r + 1) % R] += 1
        assert c.moe_dispatch_cached(xs[r], stale, check=False) == binding.MOE_ERR_STALE_PEERS
        assert c.moe_status() == 0
    assert (u16(windows) == harness.CANARY).all()               # every refusal left the windows alone
    for r, c in enumerate(comms):
        c.moe_dispatch_cached(xs[r], gens)
        assert c.moe_status() == 0
    assert np.array_equal(u16(windows), want.windows)
    # the windows move to new allocations: new table, new generations; the old stamp is refused
    windows2 = [fill() for _ in range(R)]
    gens2 = gens + 10
    for r, c in enumerate(comms):
        c.moe_peers_set([t.data_ptr() for t in windows2], gens2, C)
        assert c.moe_dispatch_cached(xs[r], gens, check=False) == binding.MOE_ERR_STALE_PEERS
        c.moe_dispatch_cached(xs[r], gens2)
        assert c.moe_status() == 0
    assert np.array_equal(u16(windows2), want.windows)
    allwin = torch.cat(windows2)
    harness.gpu_expert_scale(allwin, idx, E, R, C, inp.scale.to(dev))
    for d in range(R):
        windows2[d].copy_(allwin[d * C:(d + 1) * C])
    Y = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
    for r, c in enumerate(comms):
        y_r = torch.empty((int(rts[r + 1] - rts[r]), H), dtype=torch.bfloat16, device=dev)
        assert c.moe_combine_cached(gens, w[rts[r]:rts[r + 1]].contiguous(), y_r, check=False) == binding.MOE_ERR_STALE_PEERS
        c.moe_combine_cached(gens2, w[rts[r]:rts[r + 1]].contiguous(), y_r)
        assert c.moe_status() == 0
        Y[rts[r]:rts[r + 1]] = y_r
    assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), want.Y) <= 1
    for c in comms:
        assert c.moe_peers_close() == binding.MOE_OK
        assert c.moe_peers_check(gens2) == binding.MOE_ERR_STALE_PEERS
        c.close()


@pytest.mark.parametrize("case", [c for c in CASES if c[2] % 128 == 0], ids=[c[0] for c in CASES if c[2] % 128 == 0])
def test_group_quantised_dispatch_through_the_installed_table(case):
    """Windows made with MOE_WINDOW_QUANT_GROUP: every rank's codes and its [C, H/128] group scales land in the
    parts of its allocation that the flag reserves, bit-identical to the oracle's single global result; the sizes
    and flags the library accepts are the documented ones."""
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    G = H // 128
    wl = Workload(name, T, H, E, R, K, sch, routing, "identity", 7300 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    rts = inp.rank_tok_start
    p = oracle.plan(inp.topk_idx.numpy(), E, R, rts)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(inp.topk_idx.numpy(), E, R, p, C, rts)
    want_q = np.full((R * C, H), 0, np.uint8)
    want_s = np.full((R * C, G), 0.0, np.float32)
    assert oracle.dispatch_quant_group(synth.bf16_to_u16(inp.X), slots, want_q, want_s, 128, 4) == oracle.OK

    idx, X = inp.topk_idx.to(dev), inp.X.to(dev)
    comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
    counts = torch.zeros((R, E), dtype=torch.int32, device=dev)
    for r, c in enumerate(comms):
        c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, counts[r])
    for c in comms:
        c.moe_notify(counts)
    FLAGS = binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_QUANT_GROUP
    up = lambda n: (n + 255) // 256 * 256
    total = comms[0].moe_window_bytes(C, FLAGS)
    assert total == up(C * H * 2) + binding.moe_state_bytes(R) + up(C * H) + up(C * G * 4)
    # both quantised forms at once, or an unknown bit, are refused (size 0)
    assert comms[0].moe_window_bytes(C, FLAGS | binding.MOE_WINDOW_QUANT) == 0
    assert comms[0].moe_window_bytes(C, 8) == 0
    backings = [torch.zeros(total // 2, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    bases = [b.data_ptr() for b in backings]
    for r, c in enumerate(comms):
        c.moe_peers_set(bases, None, C, my_rank=r, flags=FLAGS)
    for r, c in enumerate(comms):
        x_r = X[rts[r]:rts[r + 1]].contiguous()
        # the row-wise call needs windows with row-wise parts
        assert c.moe_dispatch_quant_cached(x_r, check=False) == binding.MOE_ERR_STALE_PEERS
        assert c.moe_dispatch_quant_group_cached(x_r, group_size=64, check=False) == binding.MOE_ERR_INVALID_ARG
        c.moe_dispatch_quant_group_cached(x_r)
        assert c.moe_status() == 0
    codes_at = up(C * H * 2) + binding.moe_state_bytes(R)
    scales_at = codes_at + up(C * H)
    got_q = np.concatenate([b.view(torch.uint8)[codes_at:codes_at + C * H].view(C, H).cpu().numpy() for b in backings])
    got_s = np.concatenate([b.view(torch.uint8)[scales_at:scales_at + 4 * C * G].view(torch.float32).view(C, G).cpu().numpy()
                            for b in backings])
    assert np.array_equal(got_q, want_q) and np.array_equal(got_s.view(np.uint32), want_s.view(np.uint32))
    # a table installed with the row-wise parts refuses the group-wise call
    comms[0].moe_peers_set(bases, None, C, my_rank=0, flags=binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_QUANT)
    assert comms[0].moe_dispatch_quant_group_cached(X[:int(rts[1])].contiguous(), check=False) == binding.MOE_ERR_STALE_PEERS
    for c in comms:
        c.close()


@pytest.mark.parametrize("case", [CASES[0], CASES[1], CASES[3]], ids=lambda c: c[0])
def test_counts_exchanged_through_the_mailboxes_of_one_process(case):
    """The count exchange by the library's own stores (moe_push_counts, moe_notify_peers), every rank a context of
    this process, so every push is enqueued before any notify: the offsets and receive counts equal the oracle's, two
    steps with different routing use the two buffers in turn, dispatch and combine through the table reproduce the
    global result, and a notify nobody pushed for runs out after its bound, reports MOE_ERR_TIMEOUT without
    trapping and leaves no plan behind."""
    name, T, H, E, R, K, sch, routing, per = case
    dev = torch.device("cuda:0")
    FLAGS = binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_COUNTS
    comms, backings, bases, C_alloc = None, None, None, None
    for step, seed in enumerate((7100, 7200, 7300)):
        wl = Workload(name, T, H, E, R, K, sch, routing, "identity", seed + T, rank_tokens=per)
        inp = synth.make_inputs(wl)
        rts = inp.rank_tok_start
        p = oracle.plan(inp.topk_idx.numpy(), E, R, rts)
        idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
        if comms is None:
            comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
            C_alloc = int(p.n_recv.max()) + 64                       # room for the other steps' routing
            total = comms[0].moe_window_bytes(C_alloc, FLAGS) // 2
            backings = [torch.zeros(total, dtype=torch.bfloat16, device=dev) for _ in range(R)]   # state and mailbox zeroed
            bases = [b.data_ptr() for b in backings]
            # a table without the mailbox refuses the exchange; so does a context that has not laid out its tokens
            comms[0].moe_peers_set(bases, None, C_alloc, my_rank=0, flags=binding.MOE_WINDOW_STATE)
            comms[0].moe_layout(sch, idx[rts[0]:rts[1]].contiguous(), 0, torch.zeros(E, dtype=torch.int32, device=dev))
            assert comms[0].moe_push_counts(1, check=False) == binding.MOE_ERR_STALE_PEERS
            assert comms[0].moe_notify_peers(1, check=False) == binding.MOE_ERR_STALE_PEERS
            for r, c in enumerate(comms):
                c.moe_peers_set(bases, None, C_alloc, my_rank=r, flags=FLAGS)
            assert comms[1].moe_push_counts(1, check=False) == binding.MOE_ERR_NOT_PLANNED
            assert comms[1].moe_layout_push(sch, idx[rts[1]:rts[2]].contiguous(), 0, 1, check=False) == \
                binding.MOE_ERR_STALE_PEERS                          # not the rank of the installed table
        C = C_alloc
        assert int(p.n_recv.max()) <= C
        want = harness.oracle_run(inp, C)
        epoch = step + 1
        row = torch.zeros(E, dtype=torch.int32, device=dev)
        for r, c in enumerate(comms):                              # every rank lays out and pushes ...
            if step == 1:                                          # ... as one call (one kernel for small batches)
                c.moe_layout_push(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, epoch)
            else:
                c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, row)
                c.moe_push_counts(epoch)
        for r, c in enumerate(comms):                              # ... then every rank builds its offsets
            c.moe_notify_peers(epoch)
            assert c.moe_status() == 0
            v = c.moe_plan_view()
            assert np.array_equal(v["large_off"].cpu().numpy(), p.o), (step, r)
            assert np.array_equal(v["n_recv"].cpu().numpy(), p.n_recv)
            if sch == PREFILL:
                assert np.array_equal(v["counts"].cpu().numpy(), p.M) and np.array_equal(v["n_exp"].cpu().numpy(), p.n_exp)
                assert np.array_equal(v["c_rank"].cpu().numpy(), p.c_rank)
        rows = [b[:C * H].view(C, H) for b in backings]
        for t in rows:
            t.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
        for r, c in enumerate(comms):
            c.moe_dispatch_cached(X[rts[r]:rts[r + 1]].contiguous())
            assert c.moe_status() == 0
        assert np.array_equal(torch.cat(rows).cpu().view(torch.int16).numpy().view(np.uint16), want.windows)
        Y = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
        for r, c in enumerate(comms):
            y_r = torch.empty((int(rts[r + 1] - rts[r]), H), dtype=torch.bfloat16, device=dev)
            c.moe_combine_cached(None, w[rts[r]:rts[r + 1]].contiguous(), y_r)
            assert c.moe_status() == 0
            Y[rts[r]:rts[r + 1]] = y_r
        assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), want.Y) <= 1
    # epoch 4: only rank 0 pushes; rank 1's notify is bounded (50 ms here), reports, and leaves no plan
    c = comms[1]
    c.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 50)
    row = torch.zeros(E, dtype=torch.int32, device=dev)
    for r in (0, 1):
        comms[r].moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, row)
    comms[0].moe_push_counts(4)
    c.moe_notify_peers(4)
    assert c.moe_status() == binding.MOE_ERR_TIMEOUT
    assert c.moe_dispatch_cached(X[rts[1]:rts[2]].contiguous(), check=False) == binding.MOE_ERR_NOT_PLANNED
    c.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 0)
    # the others push: the same epoch now completes
    for r in range(1, R):
        comms[r].moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, row)
        comms[r].moe_push_counts(4)
    c.moe_notify_peers(4)
    assert c.moe_status() == 0
    assert np.array_equal(c.moe_plan_view()["large_off"].cpu().numpy(), p.o)
    for cc in comms:
        cc.close()


def test_signals_and_bounded_waits_between_ranks_of_one_process():
    """The device-side phase order with every rank a context of this process (all on the one GPU, so every signal
    is enqueued before any wait): signals reach every rank's state region, waits pass once all R signals of the
    epoch are there, and a wait nobody answers runs out after its bound, raises MOE_ERR_TIMEOUT without
    trapping, and leaves the context usable."""
    name, T, H, E, R, K, sch, routing, per = CASES[0]
    dev = torch.device("cuda:0")
    wl = Workload(name, T, H, E, R, K, sch, routing, "identity", 7000 + T, rank_tokens=per)
    inp = synth.make_inputs(wl)
    rts = inp.rank_tok_start
    p = oracle.plan(inp.topk_idx.numpy(), E, R, rts)
    C = int(p.n_recv.max()) + 1
    want = harness.oracle_run(inp, C)
    idx, w, X = inp.topk_idx.to(dev), inp.topk_w.to(dev), inp.X.to(dev)
    comms = [binding.MoeComm(max(int(rts[r + 1] - rts[r]), 1), H, E, R, K, dev) for r in range(R)]
    counts = torch.zeros((R, E), dtype=torch.int32, device=dev)
    for r, c in enumerate(comms):
        c.moe_layout(sch, idx[rts[r]:rts[r + 1]].contiguous(), r, counts[r])
    for c in comms:
        c.moe_notify(counts)
    FLAGS = binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_QUANT
    total = comms[0].moe_window_bytes(C, FLAGS) // 2
    state_at = (comms[0].moe_window_bytes(C, binding.MOE_WINDOW_STATE) - binding.moe_state_bytes(R)) // 4
    assert total * 2 >= C * H * 2 + binding.moe_state_bytes(R) + C * H + 4 * C
    backings = [torch.zeros(total, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    rows = [b[:C * H].view(C, H) for b in backings]
    for t in rows:
        t.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
    bases = [b.data_ptr() for b in backings]
    # without a state region the signals have nowhere to go
    comms[0].moe_peers_set(bases, None, C, my_rank=0, flags=0)
    assert comms[0].moe_signal_peers(0, 1, check=False) == binding.MOE_ERR_STALE_PEERS
    assert comms[0].moe_wait_peers(0, 1, check=False) == binding.MOE_ERR_STALE_PEERS
    for r, c in enumerate(comms):
        c.moe_peers_set(bases, None, C, my_rank=r, flags=FLAGS)
    state = lambda d: backings[d].view(torch.int32)[state_at:state_at + binding.MOE_SYNC_SLOTS * R].view(binding.MOE_SYNC_SLOTS, R)
    for epoch in (1, 2):
        for r, c in enumerate(comms):                      # every rank dispatches and signals ...
            c.moe_dispatch_cached(X[rts[r]:rts[r + 1]].contiguous())
            c.moe_signal_peers(0, epoch)
        for c in comms:                                    # ... then every rank waits: all signals are there
            c.moe_wait_peers(0, epoch)
            assert c.moe_status() == 0
        for d in range(R):
            assert state(d)[0].tolist() == [epoch] * R and state(d)[1].tolist() == [epoch - 1] * R
        assert np.array_equal(torch.cat(rows).cpu().view(torch.int16).numpy().view(np.uint16), want.windows)
        for r, c in enumerate(comms):
            c.moe_signal_peers(1, epoch)
        Y = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
        for r, c in enumerate(comms):
            c.moe_wait_peers(1, epoch)
            y_r = torch.empty((int(rts[r + 1] - rts[r]), H), dtype=torch.bfloat16, device=dev)
            c.moe_combine_cached(None, w[rts[r]:rts[r + 1]].contiguous(), y_r)
            assert c.moe_status() == 0
            Y[rts[r]:rts[r + 1]] = y_r
        assert harness.max_ulp_diff(Y.cpu().view(torch.int16).numpy().view(np.uint16), want.Y) <= 1
    # the quantised dispatch through the same table: codes and scales land in the parts of every allocation that
    # MOE_WINDOW_QUANT reserves; a table installed without that flag refuses the call
    want_q = np.full((R * C, H), 0, np.uint8)
    want_s = np.full((R * C,), 0.0, np.float32)
    assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), want.slots, want_q, want_s, 4) == oracle.OK
    for r, c in enumerate(comms):
        c.moe_dispatch_quant_cached(X[rts[r]:rts[r + 1]].contiguous())
        assert c.moe_status() == 0
    up = lambda n: (n + 255) // 256 * 256
    codes_at = up(C * H * 2) + binding.moe_state_bytes(R)
    scales_at = codes_at + up(C * H)
    got_q = np.concatenate([b.view(torch.uint8)[codes_at:codes_at + C * H].view(C, H).cpu().numpy() for b in backings])
    got_s = np.concatenate([b.view(torch.uint8)[scales_at:scales_at + 4 * C].view(torch.float32).cpu().numpy() for b in backings])
    assert np.array_equal(got_q, want_q) and np.array_equal(got_s.view(np.uint32), want_s.view(np.uint32))
    comms[0].moe_peers_set(bases, None, C, my_rank=0, flags=binding.MOE_WINDOW_STATE)
    assert comms[0].moe_dispatch_quant_cached(X[:int(rts[1])].contiguous(), check=False) == binding.MOE_ERR_STALE_PEERS
    comms[0].moe_peers_set(bases, None, C, my_rank=0, flags=FLAGS)
    # only one of R signals arrives for epoch 3: the wait is bounded (50 ms here), reports, and nothing hangs
    c = comms[1]
    c.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 50)
    comms[0].moe_signal_peers(0, 3)
    c.moe_wait_peers(0, 3)
    y_r = torch.full((int(rts[2] - rts[1]), H), 7.0, dtype=torch.bfloat16, device=dev)
    c.moe_combine_cached(None, w[rts[1]:rts[2]].contiguous(), y_r)       # behind a failed wait: writes nothing
    assert c.moe_status() == binding.MOE_ERR_TIMEOUT
    assert bool((y_r == 7.0).all())
    c.moe_set_option(binding.MOE_OPT_TEST_STARVE_WAIT_MS, 0)
    for cc in comms[1:]:
        cc.moe_signal_peers(0, 3)
    c.moe_wait_peers(0, 3)                                               # now all R are there
    c.moe_combine_cached(None, w[rts[1]:rts[2]].contiguous(), y_r)
    assert c.moe_status() == 0
    assert harness.max_ulp_diff(y_r.cpu().view(torch.int16).numpy().view(np.uint16), want.Y[int(rts[1]):int(rts[2])]) <= 1
    for c in comms:
        c.close()


# ------------------------------------------------------------------ two processes, windows mapped into each other
IPC_SHAPE = dict(T=600, H=512, E=16, K=4, per=(250, 350), seed=7300)


def _ipc_workload(world):
    c = IPC_SHAPE
    return Workload("ipc", c["T"], c["H"], c["E"], world, c["K"], DECODE, "uniform", "identity", c["seed"],
                    rank_tokens=c["per"])


def _ipc_rank(rank, world, port, mode, sync, results):
    """One expert-parallel rank as its own process on the one GPU: its window lives in its own allocation, the
    other rank's window is mapped in through the library's handle exchange (moe_window_export over a gloo group,
    moe_peers_open), counts travel over the same group, phases are ordered by host barriers (no kernel waits on
    another process's kernel)."""
    import os
    import torch.distributed as dist
    from paper_2605_06055_b200 import ep
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    try:
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        wl = _ipc_workload(world)
        T, H, E, K = wl.T, wl.H, wl.E, wl.K
        inp = synth.make_inputs(wl)
        rts = inp.rank_tok_start
        lo, hi = int(rts[rank]), int(rts[rank + 1])
        idx, x, w = (inp.topk_idx[lo:hi].contiguous().to(dev), inp.X[lo:hi].contiguous().to(dev),
                     inp.topk_w[lo:hi].contiguous().to(dev))
        # ranks share the GPU here: with the device-side phase order every signal is sent before any wait is enqueued
        me = ep.EpRank(hi - lo, H, E, K, dev, mode=mode, sync=sync, host_fence=True)
        me.plan(DECODE, idx)                               # first plan: learn the capacity the windows need
        C = int(me.comm.moe_plan_view()["n_recv"].max().item()) + 1
        log = {}
        # nothing installed yet: the cached calls refuse instead of dereferencing anything
        log["refused_without_table"] = me.comm.moe_dispatch_cached(x, me.announced, check=False)
        # every window is a slice of a backing allocation of its own (large enough that the caching allocator
        # gives it a device allocation to itself): the exported handle names that allocation, plus an offset
        # (rows first, then the zeroed state region of the device-side phase order)
        def new_window(offset_rows):
            backing = torch.zeros(12 << 20, dtype=torch.bfloat16, device=dev)
            # (the handshake mode carries the group-wise quantised parts, the other modes the row-wise ones)
            flags = binding.MOE_WINDOW_STATE | (binding.MOE_WINDOW_QUANT_GROUP if mode == "handshake"
                                                else binding.MOE_WINDOW_QUANT)
            flat = backing[offset_rows * H:offset_rows * H + me.comm.moe_window_bytes(C, flags) // 2]
            win = flat[:C * H].view(C, H)
            win.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
            me.attach_window(flat, C, flags)
            return backing, win
        backing, mine = new_window(0)
        y = torch.empty((hi - lo, H), dtype=torch.bfloat16, device=dev)
        u16 = lambda t: t.cpu().view(torch.int16).numpy().view(np.uint16).copy()

        def step():
            me.plan(DECODE, idx)
            me.dispatch(x)
            me.combine(w, y)
            return me.status()

        st = step()                                        # first step: the handshake happens here in both modes
        log["handshakes_after_step_1"] = me.handshakes
        win_1, y_1 = u16(mine), u16(y)
        dist.barrier()                                     # both have read their windows before anyone refills
        mine.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
        torch.cuda.synchronize()
        dist.barrier()
        st = st or step()                                  # same windows: the cached mode exchanges nothing
        log["handshakes_after_step_2"] = me.handshakes
        win_2, y_2 = u16(mine), u16(y)
        # a stale stamp is refused and nothing is enqueued: rows stay as they are
        wrong = (me.announced if me.announced is not None else me.table_generations).copy()
        wrong[1 - rank] += 5
        before = u16(mine)
        log["refused_stale"] = me.comm.moe_dispatch_cached(x, wrong, check=False)
        log["refused_stale_combine"] = me.comm.moe_combine_cached(wrong, w, y, check=False)
        log["check_fresh"] = me.comm.moe_peers_check(me.announced if me.announced is not None else me.table_generations)
        log["check_stale"] = me.comm.moe_peers_check(wrong)
        torch.cuda.synchronize()
        dist.barrier()
        log["untouched_after_refusal"] = bool(np.array_equal(u16(mine), before))
        # rank 1 moves its window to a new allocation: every rank's table is stale at the next plan
        dist.barrier()
        if rank == 1 and mode != "static":             # ("static": the caller promises that no window moves)
            keep_old = backing                         # stays mapped on the other rank until its next handshake
            backing, mine = new_window(8)              # the new window starts 8 rows into its allocation
        else:
            mine.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
        torch.cuda.synchronize()
        dist.barrier()
        st = st or step()
        log["handshakes_after_step_3"] = me.handshakes
        win_3, y_3 = u16(mine), u16(y)
        # the quantising dispatch: codes and scales go into the parts of every rank's window allocation that
        # MOE_WINDOW_QUANT reserves, through the same address table as the rows
        me.plan(DECODE, idx)
        me.dispatch_quant(x)
        st = st or me.status()
        my_q, my_s = me.quant_views()
        dist.barrier()                                 # nobody frees a window another rank may still read
        results[rank] = ("ok", st, C, (win_1, y_1), (win_2, y_2), (win_3, y_3), my_q.cpu().numpy().copy(),
                         my_s.cpu().numpy().copy(), log)
        me.close()
        dist.barrier()
        dist.destroy_process_group()
    except Exception as exc:                           # reported to the parent, which decides between skip and fail
        import traceback
        results[rank] = ("error", repr(exc) + "\n" + traceback.format_exc())


@pytest.mark.parametrize("mode,sync", [("cached", "host"), ("handshake", "host"), ("cached", "device"),
                                       ("static", "device")])
def test_two_processes_exchange_rows_through_mapped_windows(mode, sync):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    world = 2
    with ctx.Manager() as m:
        results = m.dict()
        port = 35000 + (os.getpid() * 8 + 4 * (mode == "static") + 2 * (mode == "cached") + (sync == "device")) % 2000
        procs = [ctx.Process(target=_ipc_rank, args=(r, world, port, mode, sync, results)) for r in range(world)]
        for p_ in procs:
            p_.start()
        for p_ in procs:
            p_.join(timeout=240)
        alive = [p_ for p_ in procs if p_.is_alive()]
        for p_ in alive:
            p_.terminate()
        assert not alive, "a rank did not finish"
        res = dict(results)
    errors = [v for v in res.values() if v[0] == "error"]
    if errors and any("ipc" in e[1].lower() or "not supported" in e[1].lower() for e in errors):
        pytest.skip("CUDA IPC is not available here: " + errors[0][1])
    assert not errors and len(res) == world, res
    wl = _ipc_workload(world)
    H = wl.H
    inp = synth.make_inputs(wl)
    C = res[0][2]
    assert res[1][2] == C
    want = harness.oracle_run(inp, C)
    rts = inp.rank_tok_start
    want_q = np.full((world * C, H), 0, np.uint8)          # the allocations start zeroed
    if mode == "handshake":                                # windows with one scale per 128 elements
        want_s = np.full((world * C, H // 128), 0.0, np.float32)
        assert oracle.dispatch_quant_group(synth.bf16_to_u16(inp.X), want.slots, want_q, want_s, 128, 2) == oracle.OK
    else:
        want_s = np.full((world * C,), 0.0, np.float32)
        assert oracle.dispatch_quant(synth.bf16_to_u16(inp.X), want.slots, want_q, want_s, 2) == oracle.OK
    for r in range(world):
        _, st, _, s1, s2, s3, q, sc, log = res[r]
        assert st == 0
        for (win, y) in (s1, s2, s3):
            assert np.array_equal(win, want.windows[r * C:(r + 1) * C])        # rows from both processes, bit-exact
            assert harness.max_ulp_diff(y, want.Y[int(rts[r]):int(rts[r + 1])]) <= 1
        assert np.array_equal(q, want_q[r * C:(r + 1) * C])
        assert sc.shape == want_s[r * C:(r + 1) * C].shape
        assert np.array_equal(sc.view(np.uint32), want_s[r * C:(r + 1) * C].view(np.uint32))
        assert log["refused_without_table"] == binding.MOE_ERR_STALE_PEERS
        assert log["refused_stale"] == binding.MOE_ERR_STALE_PEERS
        assert log["refused_stale_combine"] == binding.MOE_ERR_STALE_PEERS
        assert log["check_fresh"] == binding.MOE_OK and log["check_stale"] == binding.MOE_ERR_STALE_PEERS
        assert log["untouched_after_refusal"]
        if mode == "cached":      # one handshake for the first step, none for the second, one after the move
            assert (log["handshakes_after_step_1"], log["handshakes_after_step_2"], log["handshakes_after_step_3"]) == (1, 1, 2)
        elif mode == "static":    # exchanged once
            assert (log["handshakes_after_step_1"], log["handshakes_after_step_2"], log["handshakes_after_step_3"]) == (1, 1, 1)
        else:                     # the handshake mode exchanges addresses before every dispatch
            assert (log["handshakes_after_step_1"], log["handshakes_after_step_2"], log["handshakes_after_step_3"]) == (1, 2, 3)


# ------------------------------------------------------------------ the benchmark's expert-parallel leg
def _ep_leg_rank(rank, world, port, results):
    import os
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    try:
        import bench
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        results[rank] = ("ok", bench.ep_leg(dev, 3, None, shapes=("decode",)))
        dist.barrier()
        dist.destroy_process_group()
    except Exception as exc:
        import traceback
        results[rank] = ("error", repr(exc) + "\n" + traceback.format_exc())


def test_benchmark_expert_parallel_leg_as_two_processes_on_one_gpu():
    """The code `bench.py --gpus N` runs for N > 1 (rank = process, windows mapped into each other), here as two
    processes that share the one GPU and talk over gloo: it verifies its own windows and outputs before it times
    anything, exchanges no addresses in the timed steps of the cached mode and one set per step in the handshake
    mode, and orders its phases by host barriers or by arrival flags."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    world = 2
    with ctx.Manager() as m:
        results = m.dict()
        procs = [ctx.Process(target=_ep_leg_rank, args=(r, world, 37000 + os.getpid() % 2000, results))
                 for r in range(world)]
        for p_ in procs:
            p_.start()
        for p_ in procs:
            p_.join(timeout=300)
        alive = [p_ for p_ in procs if p_.is_alive()]
        for p_ in alive:
            p_.terminate()
        assert not alive, "a rank did not finish"
        res = dict(results)
    assert all(v[0] == "ok" for v in res.values()) and len(res) == world, res
    for r in range(world):
        leg = res[r][1]
        assert leg["ranks"] == 2 and "decode" in leg
        assert leg["ranks_share_a_gpu"] is True
        for variant, want_handshakes in (("cached_addresses__host_phase_order", 0),
                                         ("handshake_addresses__host_phase_order", 3),
                                         ("cached_addresses__device_phase_order", 0),
                                         ("static_addresses__device_phase_order", 0),
                                         ("static_addresses__device_phase_order__counts_through_mailboxes", 0)):
            got = leg["decode"][variant]
            assert got["verified"]["window_equals_single_gpu_path"] and got["verified"]["Y_equals_X"]
            assert got["handshakes_in_timed_steps"] == want_handshakes
            assert got["step_us"] > 0 and got["dispatch_phase_us"] > 0 and got["combine_phase_us"] > 0


def _ep_leg_nccl_single_rank(port, results):
    import os
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1")
    try:
        import bench
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
        results[0] = ("ok", bench.ep_leg(dev, 3, None, shapes=("decode",)))
        dist.destroy_process_group()
    except Exception as exc:
        import traceback
        results[0] = ("error", repr(exc) + "\n" + traceback.format_exc())


def test_benchmark_expert_parallel_leg_over_nccl_with_one_rank():
    """The same leg over the backend a multi-GPU run uses (NCCL: device tensors in every exchange), with the one
    rank this machine can give it: the exchanges, the handshake with no peer to map, and the device-side phase order
    WITHOUT the host barrier between signal and wait (one rank per GPU), which a single rank satisfies by itself."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        results = m.dict()
        p_ = ctx.Process(target=_ep_leg_nccl_single_rank, args=(38000 + os.getpid() % 2000, results))
        p_.start()
        p_.join(timeout=300)
        if p_.is_alive():
            p_.terminate()
            raise AssertionError("the rank did not finish")
        res = dict(results)
    assert res[0][0] == "ok", res
    leg = res[0][1]
    assert leg["ranks"] == 1 and leg["ranks_share_a_gpu"] is False
    for variant in ("cached_addresses__host_phase_order", "handshake_addresses__host_phase_order",
                    "cached_addresses__device_phase_order", "static_addresses__device_phase_order"):
        got = leg["decode"][variant]
        assert got["verified"]["window_equals_single_gpu_path"] and got["verified"]["Y_equals_X"]
        assert got["step_us"] > 0
    first = leg["decode"]["cached_addresses__host_phase_order"]
    assert first["verified"]["quantised_codes_and_scales_equal_single_gpu_path"] and first["quantised_dispatch_phase_us"] > 0


def test_expert_parallel_child_mode_of_the_benchmark_two_ranks_on_one_gpu():
    """`bench.py --ep-child`, which a multi-GPU run of the benchmark starts once per rank, here as two processes on
    the one GPU over gloo: rank 0 prints the leg's JSON object."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    port = 39000 + os.getpid() % 2000
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(root, "bench.py"), "--ep-child", "--ep-backend", "gloo",
                                       "--ep-device", "0", "--ep-shapes", "decode", "--steps", "3"], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p_.communicate(timeout=300) for p_ in procs]
    assert all(p_.returncode == 0 for p_ in procs), [o[1][-600:] for o in outs]
    leg = json.loads([ln for ln in outs[0][0].splitlines() if ln.startswith("{")][-1])
    assert leg["ranks"] == 2 and leg["ranks_share_a_gpu"] is True
    for variant in ("cached_addresses__host_phase_order", "handshake_addresses__host_phase_order",
                    "cached_addresses__device_phase_order"):
        assert leg["decode"][variant]["verified"]["window_equals_single_gpu_path"]
        assert leg["decode"][variant]["verified"]["Y_equals_X"]
    assert not [ln for ln in outs[1][0].splitlines() if ln.startswith("{")]       # only rank 0 prints
