"""Property tests over random small shapes (hypothesis).

CPU part: invariants of the oracle that hold for every routing (conservation,
bijection, contiguity, round trip).  GPU part: the CUDA path equals the oracle
on shapes and routings drawn at random, including non-uniform ranks, empty
ranks, duplicate experts within a token and both schedules.
"""
import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
from paper_2605_06055_b200 import synth


@st.composite
def routings(draw, max_T=96):
    R = draw(st.sampled_from([1, 2, 3, 4, 8]))
    E = R * draw(st.integers(1, 4))
    K = draw(st.integers(1, min(8, max(1, E))))
    T = draw(st.integers(0, max_T))
    replace = draw(st.booleans())
    seed = draw(st.integers(0, 2 ** 31 - 1))
    rng = np.random.default_rng(seed)
    if T == 0:
        idx = np.zeros((0, K), np.int32)
    elif replace:
        idx = rng.integers(0, E, (T, K)).astype(np.int32)
    else:
        idx = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32)
    cuts = np.sort(rng.integers(0, T + 1, R - 1))
    rts = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    return T, K, E, R, idx, rts, seed


@settings(max_examples=150, deadline=None)
@given(routings())
def test_oracle_invariants_hold_for_any_routing(case):
    T, K, E, R, idx, rts, seed = case
    p = oracle.plan(idx, E, R, rts)
    assert p.status == oracle.OK
    E_r = E // R
    assert p.M.sum() == T * K and np.array_equal(p.M.sum(1), np.diff(rts) * K)
    assert np.array_equal(p.c_rank.sum(1), np.diff(rts) * K) and np.array_equal(p.c_rank.sum(0), p.n_recv)
    assert np.array_equal(p.n_exp.reshape(R, E_r).sum(1), p.n_recv)
    # offsets are the exclusive scan of counts in window order
    blocks = p.M.T.reshape(R, E_r * R)
    assert np.array_equal(p.o.reshape(R, E_r * R), np.cumsum(blocks, 1) - blocks)
    C = int(p.n_recv.max()) + 1 if T else 1
    st_, slots = oracle.slots(idx, E, R, p, C, rts)
    assert st_ == oracle.OK
    flat = slots.reshape(-1)
    assert len(np.unique(flat)) == T * K                                  # every branch exactly once
    want = np.concatenate([d * C + np.arange(p.n_recv[d]) for d in range(R)]) if T else np.zeros(0, np.int64)
    assert np.array_equal(np.sort(flat), want)
    # inside one (source rank, expert) block slots increase with the flat branch index (stable)
    src = np.repeat(np.repeat(np.arange(R), np.diff(rts)), K)
    key = src * E + idx.reshape(-1)
    for k_ in np.unique(key):
        assert (np.diff(flat[key == k_]) == 1).all()
    # identity experts and weights that sum to one give back X
    H = 8
    rng = np.random.default_rng(seed)
    X = synth.bf16_to_u16(torch.from_numpy(rng.standard_normal((T, H)).astype(np.float32)).to(torch.bfloat16)).copy()
    win = np.full((R * C, H), 0x7FC1, np.uint16)
    oracle.dispatch(X, slots, win)
    W = np.full((T, K), 1.0 / K, np.float32) if K in (1, 2, 4, 8) else None
    if W is not None:
        _, Y = oracle.combine(win, slots, W, H)
        assert np.array_equal(Y & 0x7FFF, X & 0x7FFF)                        # up to the sign of zero


@pytest.mark.gpu
@settings(max_examples=40, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(routings(max_T=400), st.sampled_from([8, 16, 72, 264, 1000]), st.sampled_from([0, 1]),
       st.sampled_from([1, 2]))
def test_gpu_equals_oracle_on_random_shapes(case, H, schedule, path):
    import harness
    T, K, E, R, idx, rts, seed = case
    wl = synth.Workload("prop", T, H, E, R, K, schedule, "replace", "scale", seed % 100000,
                        rank_tokens=tuple(int(x) for x in np.diff(rts)))
    inp = synth.make_inputs(wl)
    inp.topk_idx = torch.from_numpy(idx.reshape(T, K))
    p = oracle.plan(idx, E, R, rts)
    C = int(p.n_recv.max()) + 1 if T else 1
    g = harness.gpu_run(inp, C, schedule, dispatch_path=path)
    harness.assert_parity(g, harness.oracle_run(inp, C), schedule)
