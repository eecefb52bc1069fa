"""Host logic of the multi-GPU bench path on CPU: two gloo ranks, the reduction
that turns per-replica device times into the job's number (max over ranks), and
the replica aggregation."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 1.25 if rank == 0 else 2.5            # ms per step measured by this replica
    slowest = bench.reduce_max_over_ranks(mine, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = slowest
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_bytes():
    import bench
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29000 + os.getpid() % 2000, out), nprocs=world, join=True)
        assert out[0] == 2.5 and out[1] == 2.5
    wl = bench.WORKLOADS["c2"]()
    one = bench.aggregate_value(bench.bytes_step(wl), 1, 2.5)
    two = bench.aggregate_value(bench.bytes_step(wl), 2, 2.5)
    assert abs(two - 2 * one) < 1e-9 * two
    assert bench.reduce_max_over_ranks(3.0, None, torch.device("cpu")) == 3.0


def test_algorithmic_bytes_match_the_stated_formulas():
    import bench
    wl = bench.WORKLOADS["c3"]()
    # per token: one row read + K rows written (dispatch) / K rows read + one written (combine), rows of 2H bytes
    assert bench.bytes_dispatch(wl) == 2 * 7168 * 32768 * 9 + 8 * 32768 * 8 + 4 * 256 * 8 == 4229963776
    assert bench.bytes_combine(wl) == 2 * 7168 * 32768 * 9 + 12 * 32768 * 8 + 4 * 256 * 8
    assert round(bench.bytes_dispatch(bench.WORKLOADS["c2"]()) / 1e6, 1) == 264.4


def _gather_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2605_06055_b200 import ep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    row = torch.arange(6, dtype=torch.int32) + 100 * rank          # this rank's row of the count matrix
    out[rank] = ep.all_gather_counts(row).tolist()
    dist.destroy_process_group()


def test_count_exchange_between_two_ranks_builds_the_same_matrix_everywhere():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_gather_worker, args=(world, 31000 + os.getpid() % 2000, out), nprocs=world, join=True)
        want = [[0, 1, 2, 3, 4, 5], [100, 101, 102, 103, 104, 105]]
        assert out[0] == want and out[1] == want


def _protocol_worker(rank, world, port, out):
    """One expert-parallel rank on CPU: local Layout (the oracle on this rank's tokens), the count
    exchange over the process group, Notify on the gathered matrix."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import numpy as np
    import oracle
    from paper_2605_06055_b200 import ep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    E, K, align = 12, 3, 4
    rng = np.random.default_rng(5)
    counts = [37, 21]
    idx_all = rng.integers(0, E, (sum(counts), K)).astype(np.int32)
    lo = sum(counts[:rank])
    local = idx_all[lo:lo + counts[rank]]
    only_me = np.array([0] * (rank + 1) + [len(local)] * (world - rank), np.int32)
    mine = oracle.plan(local, E, world, only_me, align=align)
    gathered = ep.all_gather_counts(torch.from_numpy(mine.M[rank].copy())).numpy()
    st, c_rank, o, n_exp, n_recv = oracle.notify(gathered, align=align)
    out[rank] = (st, mine.s.tolist(), o.tolist(), n_recv.tolist(), gathered.tolist())
    dist.destroy_process_group()


def test_two_ranks_layout_exchange_notify_reproduce_the_global_plan():
    import numpy as np
    import oracle
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_protocol_worker, args=(world, 33000 + os.getpid() % 2000, out), nprocs=world, join=True)
        results = dict(out)
    E, K, align = 12, 3, 4
    rng = np.random.default_rng(5)
    counts = [37, 21]
    idx_all = rng.integers(0, E, (sum(counts), K)).astype(np.int32)
    whole = oracle.plan(idx_all, E, world, np.array([0, 37, 58], np.int32), align=align)
    lo = 0
    for rank in range(world):
        st, s_local, o, n_recv, gathered = results[rank]
        assert st == oracle.OK
        assert gathered == whole.M.tolist()                       # every rank holds the same matrix
        assert o == whole.o.tolist() and n_recv == whole.n_recv.tolist()
        assert s_local == whole.s[lo:lo + counts[rank]].tolist()   # Layout is local
        lo += counts[rank]


def _address_protocol_worker(rank, world, port, out):
    """The address side of the multi-rank protocol on CPU: every step the ranks announce their window generation
    along with their count row, decide from it whether the cached address table is still valid, and exchange
    handles (plain bytes) only when it is not."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import numpy as np
    from paper_2605_06055_b200 import ep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    E = 5
    generation, table, log = 1, None, []
    for step in range(5):
        if step == 3 and rank == 1:
            generation += 1                                      # this rank moved its window
        message = torch.cat([torch.full((E,), 10 * rank + step, dtype=torch.int32),
                             torch.tensor([generation], dtype=torch.int32)])
        gathered = ep.all_gather_rows(message)
        counts, announced = gathered[:, :E], gathered[:, E].numpy()
        assert counts.tolist() == [[10 * r + step] * E for r in range(world)]
        stale = ep.addresses_stale(table, announced)
        if stale:                                                # the handshake: handles are opaque bytes
            mine = bytes([rank, generation]) + bytes(94)
            handles = ep.all_gather_bytes(mine, torch.device("cpu"))
            assert len(handles) == 96 * world
            table = np.array([handles[96 * r + 1] for r in range(world)], np.int32)
            assert [handles[96 * r] for r in range(world)] == list(range(world))
        log.append((bool(stale), announced.tolist(), table.tolist()))
    out[rank] = log
    dist.destroy_process_group()


def test_cached_addresses_are_re_exchanged_only_when_a_generation_changes():
    from paper_2605_06055_b200 import ep
    assert ep.addresses_stale(None, [1, 1])
    assert not ep.addresses_stale([1, 2], [1, 2])
    assert ep.addresses_stale([1, 2], [1, 3]) and ep.addresses_stale([1, 2], [2, 2])
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_address_protocol_worker, args=(world, 36000 + os.getpid() % 2000, out), nprocs=world, join=True)
        logs = dict(out)
    assert logs[0] == logs[1]                                    # every rank takes the same decisions
    assert [s for s, _, _ in logs[0]] == [True, False, False, True, False]
    assert logs[0][2][2] == [1, 1] and logs[0][4][2] == [1, 2]


def test_expert_parallel_child_that_fails_or_hangs_costs_only_its_own_entry():
    """bench.py runs the expert-parallel leg of a multi-GPU run in child processes; a child that exits badly, prints
    nothing or never returns becomes an `error` entry (the child is ended after the timeout), a good one's last
    JSON line is returned."""
    import sys
    import bench
    env = dict(os.environ)
    ok = bench.spawn_ep_child([sys.executable, "-c", "print('noise'); print('{\"ranks\": 2, \"decode\": {}}')"], env, 30)
    assert ok == {"ranks": 2, "decode": {}}
    bad = bench.spawn_ep_child([sys.executable, "-c", "import sys; sys.stderr.write('boom'); sys.exit(3)"], env, 30)
    assert "error" in bad and "3" in bad["error"] and "boom" in bad["stderr_tail"]
    hung = bench.spawn_ep_child([sys.executable, "-c", "import time; time.sleep(60)"], env, 1.5)
    assert "error" in hung and "did not finish" in hung["error"]
    assert bench.spawn_ep_child([sys.executable, "-c", "pass"], env, 30) == {}
