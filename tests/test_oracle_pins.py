"""Pins for the CPU oracle: it is checked against things other than itself.

Each test compares the oracle with a textbook/library routine, the literal
definition evaluated by brute force, exact rational arithmetic, a closed form or
a hand-worked example -- never with a retyped copy of the oracle's own loop.
No GPU is needed.
"""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def src_of_tokens(rts):
    rts = np.asarray(rts)
    return np.repeat(np.arange(len(rts) - 1), np.diff(rts))


def literal_small_offsets(idx, rts):
    """Definition of s (Prefill Layout): the number of branches that come before
    (t,j) in (t,j) order, belong to the same source rank, and chose the same
    expert -- counted one pair at a time."""
    T, K = idx.shape
    src = src_of_tokens(rts)
    flat = [(t, j) for t in range(T) for j in range(K)]
    s = np.zeros((T, K), np.int64)
    for a, (t, j) in enumerate(flat):
        s[t, j] = sum(1 for (t2, j2) in flat[:a] if src[t2] == src[t] and idx[t2, j2] == idx[t, j])
    return s


def round_to_format(x: Fraction, mant_bits: int, emin: int) -> Fraction:
    """Round an exact rational to a binary float format with `mant_bits` stored
    mantissa bits and minimum normal exponent `emin`: nearest, ties to even."""
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = abs(x)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, emin)
    quantum = Fraction(2) ** (e - mant_bits)
    n = a / quantum
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * fl * quantum


def f32(x: Fraction) -> Fraction:
    return round_to_format(x, 23, -126)


def bf16(x: Fraction) -> Fraction:
    return round_to_format(x, 7, -126)


def u16_to_float(a):
    return (np.asarray(a, np.uint16).astype(np.uint32) << 16).view(np.float32)


def rand_bf16(rng, shape):
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    return synth.bf16_to_u16(x).copy()


def random_case(rng, T, K, E, R, replace=False, uniform_ranks=False):
    if replace:
        idx = rng.integers(0, E, (T, K)).astype(np.int32)
    else:
        idx = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32) if T else np.zeros((0, K), np.int32)
    if uniform_ranks and T % R == 0:
        rts = oracle.uniform_rank_tok_start(T, R)
    else:
        cuts = np.sort(rng.integers(0, T + 1, R - 1))
        rts = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    return idx, rts


SHAPES = [  # T, K, E, R
    (0, 2, 4, 2), (1, 1, 1, 1), (7, 1, 4, 4), (37, 2, 8, 4), (64, 4, 16, 1), (100, 3, 12, 3),
    (256, 2, 16, 4), (513, 8, 64, 8), (300, 6, 6, 6),
]


def cases():
    rng = np.random.default_rng(20260506)
    for (T, K, E, R) in SHAPES:
        for replace in (False, True):
            if not replace and K > E:
                continue
            yield (T, K, E, R, replace) + random_case(rng, T, K, E, R, replace)


# ----------------------------------------------------------------------------- golden
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLDEN, "worked_example.json")))
    idx = np.array(g["topk_idx"], np.int32)
    T, K, E, R, H, C = (g[k] for k in "TKERHC")
    rts = np.array(g["rank_tok_start"], np.int32)
    p = oracle.plan(idx, E, R, rts)
    assert p.status == oracle.OK
    for name in ("M", "c_rank", "s", "o", "n_exp", "n_recv"):
        assert getattr(p, name).tolist() == g[name], name
    st, slots = oracle.slots(idx, E, R, p, C, rts)
    assert st == oracle.OK and slots.tolist() == g["slots"]

    xv = torch.tensor(g["x_row_value"], dtype=torch.float32)
    X = synth.bf16_to_u16(xv[:, None].expand(T, H).to(torch.bfloat16).contiguous())
    canary = 0xDEAD
    win = np.full((R * C, H), canary, np.uint16)
    assert oracle.dispatch(X, slots, win) == oracle.OK
    for row, tok in enumerate(g["window_row_token"]):
        want = canary if tok < 0 else X[tok, 0]
        assert (win[row] == want).all(), row
    W = np.array(g["topk_w"], np.float32)
    st, Y = oracle.combine(win, slots, W, H)
    assert st == oracle.OK
    assert np.array_equal(u16_to_float(Y), np.repeat(np.array(g["y_identity_row_value"], np.float32)[:, None], H, 1))
    scale = synth.bf16_to_u16(torch.tensor(g["scale"]).to(torch.bfloat16))
    assert oracle.expert_scale(win, H, E, R, C, p.n_exp, scale) == oracle.OK
    assert (win[8:] == canary).all()
    st, Y = oracle.combine(win, slots, W, H)
    assert np.array_equal(u16_to_float(Y), np.repeat(np.array(g["y_scale_row_value"], np.float32)[:, None], H, 1))


# ----------------------------------------------------------------------------- plan
@pytest.mark.parametrize("case", list(cases()), ids=lambda c: f"T{c[0]}K{c[1]}E{c[2]}R{c[3]}{'rep' if c[4] else ''}")
def test_plan_against_library_routines(case):
    T, K, E, R, _, idx, rts = case
    p = oracle.plan(idx, E, R, rts)
    assert p.status == oracle.OK
    E_r = E // R
    src = src_of_tokens(rts)

    # Counts: a histogram of (source rank, expert) pairs (library bincount).
    key = (np.repeat(src, K) * E + idx.reshape(-1)).astype(np.int64)
    M = np.bincount(key, minlength=R * E).reshape(R, E)
    assert np.array_equal(p.M, M)
    assert p.M.sum() == T * K
    assert np.array_equal(p.M.sum(1), np.diff(rts) * K)
    assert np.array_equal(p.c_rank, M.reshape(R, R, E_r).sum(2))
    assert np.array_equal(p.c_rank.sum(1), np.diff(rts) * K)
    assert np.array_equal(p.n_exp, M.sum(0))
    assert np.array_equal(p.n_recv, M.sum(0).reshape(R, E_r).sum(1))

    # Large offsets: exclusive cumulative sum of M laid out [dst rank][local expert][src rank],
    # restarting in every destination window.
    blocks = M.T.reshape(R, E_r * R)                       # row d: (e_local, r) blocks in window order
    excl = np.cumsum(blocks, 1) - blocks
    assert np.array_equal(p.o, excl.reshape(E, R))
    assert np.array_equal(excl[:, -1] + blocks[:, -1], p.n_recv)

    # Small offsets: within each (r, e) group they are 0..M[r,e]-1, increasing in flat order.
    flat_s = p.s.reshape(-1)
    for k_ in np.unique(key):
        assert np.array_equal(flat_s[key == k_], np.arange(M.reshape(-1)[k_]))

    # Slots: a stable sort of the branches by expert IS the packed window order,
    # because the source rank never decreases with the token index.
    C = int(p.n_recv.max()) + 3 if T else 3
    st, slots = oracle.slots(idx, E, R, p, C, rts)
    assert st == oracle.OK
    order = np.argsort(idx.reshape(-1), kind="stable")
    pos = np.empty(T * K, np.int64)
    pos[order] = np.arange(T * K)
    dst = idx.reshape(-1) // E_r
    before = np.concatenate([[0], np.cumsum(p.n_recv)])[dst]   # branches bound for earlier ranks
    assert np.array_equal(slots.reshape(-1), dst * C + pos - before)

    # Expert row ranges: the rows of [start, start+count) hold exactly the branches routed to that expert.
    st, e_start, e_count = oracle.expert_ranges(E, R, C, p.n_exp)
    assert st == oracle.OK
    owner = np.full(R * C, -1)
    owner[slots.reshape(-1)] = idx.reshape(-1)
    for e in range(E):
        assert e_count[e] == (idx == e).sum()
        assert (owner[e_start[e]:e_start[e] + e_count[e]] == e).all()
    assert e_count.sum() == T * K

    # Bijection onto the used part of each segment; each expert's rows contiguous.
    used = np.sort(slots.reshape(-1))
    want = np.concatenate([d * C + np.arange(p.n_recv[d]) for d in range(R)]) if T else np.zeros(0)
    assert np.array_equal(used, want)
    start = (np.cumsum(p.n_exp.reshape(R, E_r), 1) - p.n_exp.reshape(R, E_r)).reshape(-1)
    for e in range(E):
        rows = np.sort(slots.reshape(-1)[idx.reshape(-1) == e])
        assert np.array_equal(rows, (e // E_r) * C + start[e] + np.arange(p.n_exp[e]))


@pytest.mark.parametrize("T,K,E,R", [(5, 2, 4, 2), (40, 3, 6, 3), (64, 8, 16, 4), (129, 2, 3, 1)])
def test_small_offsets_literal_definition(T, K, E, R):
    rng = np.random.default_rng(T * 1000 + K)
    for replace in (False, True):
        if not replace and K > E:
            continue
        idx, rts = random_case(rng, T, K, E, R, replace)
        p = oracle.plan(idx, E, R, rts)
        assert np.array_equal(p.s, literal_small_offsets(idx, rts))


def test_brute_force_all_routings_tiny():
    """Every routing of T=3, K=2 over E=4 experts, R=2 ranks (4^6 cases), against
    the definitions evaluated literally in Python."""
    T, K, E, R, C = 3, 2, 4, 2, 6
    rts = np.array([0, 2, 3], np.int32)
    src = [0, 0, 1]
    E_r = E // R
    for combo in itertools.product(range(E), repeat=T * K):
        idx = np.array(combo, np.int32).reshape(T, K)
        p = oracle.plan(idx, E, R, rts)
        st, slots = oracle.slots(idx, E, R, p, C, rts)
        assert st == oracle.OK
        branches = [(t, j) for t in range(T) for j in range(K)]
        for a, (t, j) in enumerate(branches):
            e = idx[t, j]
            s_lit = sum(1 for (t2, j2) in branches[:a] if src[t2] == src[t] and idx[t2, j2] == e)
            # block (r -> e) starts after every block (e', r') that precedes it in the window of dst(e)
            o_lit = sum(1 for (t2, j2) in branches
                        if idx[t2, j2] // E_r == e // E_r and (idx[t2, j2], src[t2]) < (e, src[t]))
            assert p.s[t, j] == s_lit and p.o[e, src[t]] == o_lit
            assert slots[t, j] == (e // E_r) * C + o_lit + s_lit


def test_error_codes_and_untouched_outputs():
    idx = np.array([[0, 1], [2, 4]], np.int32)
    p = oracle.plan(idx, 4, 2)
    assert p.status == oracle.ERR_BAD_INDEX
    assert (p.M == -7).all() and (p.s == -7).all() and (p.o == -7).all()
    idx[1, 1] = -1
    assert oracle.plan(idx, 4, 2).status == oracle.ERR_BAD_INDEX
    idx[1, 1] = 3
    assert oracle.plan(idx, 4, 3, np.array([0, 1, 1, 2], np.int32)).status == oracle.ERR_INVALID_ARG   # E % R != 0
    assert oracle.plan(idx, 4, 2, np.array([0, 2, 1], np.int32)).status == oracle.ERR_INVALID_ARG
    assert oracle.plan(idx, 4, 2, np.array([0, 3, 2], np.int32)).status == oracle.ERR_INVALID_ARG
    p = oracle.plan(idx, 4, 2)
    assert p.status == oracle.OK
    C = int(p.n_recv.max())
    st, sl = oracle.slots(idx, 4, 2, p, C)
    assert st == oracle.OK
    st, sl = oracle.slots(idx, 4, 2, p, C - 1)
    assert st == oracle.ERR_CAPACITY and (sl == -1).all()


def test_edge_shapes():
    # T = 0
    p = oracle.plan(np.zeros((0, 2), np.int32), 4, 2)
    assert p.status == oracle.OK and not p.M.any() and not p.o.any() and not p.n_recv.any()
    # all branches to one expert; a rank with no tokens; E == R; K == 1
    idx = np.full((10, 1), 2, np.int32)
    rts = np.array([0, 0, 4, 10], np.int32)
    p = oracle.plan(idx, 3, 3, rts)
    assert p.n_exp.tolist() == [0, 0, 10] and p.n_recv.tolist() == [0, 0, 10]
    assert p.o[2].tolist() == [0, 0, 4] and p.s.reshape(-1).tolist() == [0, 1, 2, 3, 0, 1, 2, 3, 4, 5]
    # the same expert twice in one token: consecutive slots in j order
    idx = np.array([[1, 1, 1]], np.int32)
    p = oracle.plan(idx, 2, 1)
    assert p.s.tolist() == [[0, 1, 2]]


# ----------------------------------------------------------------------------- dispatch
@pytest.mark.parametrize("T,K,E,R,H", [(37, 2, 8, 4, 8), (100, 3, 12, 3, 24), (256, 2, 16, 4, 64)])
def test_dispatch_rows_and_canaries(T, K, E, R, H):
    rng = np.random.default_rng(T)
    idx, rts = random_case(rng, T, K, E, R, replace=True)
    X = rand_bf16(rng, (T, H))
    p = oracle.plan(idx, E, R, rts)
    C = int(p.n_recv.max()) + 2
    _, slots = oracle.slots(idx, E, R, p, C, rts)
    win = np.full((R * C, H), 0xBEEF, np.uint16)
    assert oracle.dispatch(X, slots, win) == oracle.OK
    owner = np.full(R * C, -1)
    owner[slots.reshape(-1)] = np.repeat(np.arange(T), K)
    for row in range(R * C):
        if owner[row] < 0:
            assert (win[row] == 0xBEEF).all()
        else:
            assert np.array_equal(win[row], X[owner[row]])
    win2 = np.full((R * C, H), 0xBEEF, np.uint16)
    oracle.dispatch(X, slots, win2, n_threads=3)
    assert np.array_equal(win, win2)


# ----------------------------------------------------------------------------- bf16
def test_bf16_conversion_against_torch():
    rng = np.random.default_rng(7)
    vals = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(5000) * 1e30).astype(np.float32),
        (rng.standard_normal(5000) * 1e-38).astype(np.float32),           # subnormal range
        rng.integers(0, 2 ** 32, 20000, dtype=np.uint64).astype(np.uint32).view(np.float32),
        np.array([0.0, -0.0, np.inf, -np.inf, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 3.4e38], np.float32),
    ])
    want = synth.bf16_to_u16(torch.from_numpy(vals).to(torch.bfloat16))
    for v, w in zip(vals, want):
        got = oracle.float_to_bf16(v)
        if np.isnan(v):
            assert (got & 0x7F80) == 0x7F80 and (got & 0x7F) != 0
        else:
            assert got == w, (v, got, w)
    for b in list(range(0, 65536, 37)) + [0x7F80, 0xFF80, 0x8000]:
        f = oracle.bf16_to_float(b)
        t = torch.tensor([b], dtype=torch.int32).to(torch.int16).view(torch.bfloat16).float().item()
        assert (np.isnan(f) and np.isnan(t)) or f == t


# ----------------------------------------------------------------------------- combine
def _mk(rng, T, K, E, R, H, replace=False):
    idx, rts = random_case(rng, T, K, E, R, replace)
    X = rand_bf16(rng, (T, H))
    p = oracle.plan(idx, E, R, rts)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx, E, R, p, C, rts)
    win = np.full((R * C, H), 0x7FC1, np.uint16)       # NaN canary: a wrong row poisons the sum
    oracle.dispatch(X, slots, win)
    return idx, rts, X, p, C, slots, win


def test_combine_exact_rational_fma_chain():
    """acc_j = round_f32(W_j * y_j + acc_{j-1}) exactly (one rounding per term, j
    ascending), then one round to bf16 -- evaluated with exact rationals."""
    rng = np.random.default_rng(11)
    T, K, E, R, H = 12, 4, 8, 2, 8
    idx, rts, X, p, C, slots, win = _mk(rng, T, K, E, R, H)
    scale = rand_bf16(rng, (E,))
    oracle.expert_scale(win, H, E, R, C, p.n_exp, scale)
    W = rng.random((T, K)).astype(np.float32)
    st, Y = oracle.combine(win, slots, W, H)
    assert st == oracle.OK
    Xf, sf = u16_to_float(X), u16_to_float(scale)
    for t in range(T):
        for h in range(H):
            acc = Fraction(0)
            for j in range(K):
                y = bf16(Fraction(float(Xf[t, h])) * Fraction(float(sf[idx[t, j]])))   # stand-in expert, exact
                acc = f32(Fraction(float(W[t, j])) * y + acc)
            assert Fraction(float(u16_to_float(Y[t, h]))) == bf16(acc), (t, h)


def test_combine_order_matters_and_is_j_ascending():
    """Three terms chosen so that the fp32 result depends on the summation
    order; only j = 0,1,2 ascending gives the expected value."""
    H = 8
    idx = np.array([[0, 1, 2]], np.int32)
    p = oracle.plan(idx, 3, 1)
    _, slots = oracle.slots(idx, 3, 1, p, 3)
    win = np.zeros((3, H), np.uint16)
    one = synth.bf16_to_u16(torch.tensor([1.0]).to(torch.bfloat16))[0]
    win[:] = one
    W = np.array([[2.0 ** 24, 1.0, 1.0]], np.float32)   # (2^24 + 1) + 1 = 2^24 in fp32; 2^24 + (1 + 1) = 2^24 + 2
    st, Y = oracle.combine(win, slots, W, H)
    assert u16_to_float(Y[0, 0]) == np.float32(2.0 ** 24)
    W = np.array([[1.0, 1.0, 2.0 ** 24]], np.float32)
    st, Y2 = oracle.combine(win, slots, W, H)
    assert u16_to_float(Y2[0, 0]) == np.float32(2.0 ** 24)     # bf16 rounding hides +2 ...
    # ... so check the fp32 chain through a case bf16 can see: 256 + 1 + 1 in units of 2^-16 ulp is
    # invisible as well; instead use cancellation: (2^24 + 1) - 2^24 = 0 but 1 + (2^24 - 2^24) = 1.
    W = np.array([[2.0 ** 24, 1.0, -(2.0 ** 24)]], np.float32)
    _, Ya = oracle.combine(win, slots, W, H)
    assert u16_to_float(Ya[0, 0]) == 0.0
    W = np.array([[2.0 ** 24, -(2.0 ** 24), 1.0]], np.float32)
    _, Yb = oracle.combine(win, slots, W, H)
    assert u16_to_float(Yb[0, 0]) == 1.0


@pytest.mark.parametrize("T,K,E,R,H", [(64, 8, 32, 4, 64), (200, 2, 8, 8, 128), (33, 6, 12, 3, 40)])
def test_combine_within_one_ulp_of_fp64(T, K, E, R, H):
    rng = np.random.default_rng(T + K)
    idx, rts, X, p, C, slots, win = _mk(rng, T, K, E, R, H)
    scale = rand_bf16(rng, (E,))
    oracle.expert_scale(win, H, E, R, C, p.n_exp, scale)
    logits = rng.standard_normal((T, K)).astype(np.float32)
    W = (np.exp(logits) / np.exp(logits).sum(1, keepdims=True)).astype(np.float32)
    st, Y = oracle.combine(win, slots, W, H, n_threads=2)
    # closed form that never builds windows: Y[t] = sum_j W[t,j] * f_{K[t,j]}(X[t]) in fp64
    Xf = u16_to_float(X).astype(np.float64)
    sf = u16_to_float(scale)
    ref = np.zeros((T, H))
    mag = np.zeros((T, H))
    for j in range(K):
        y = torch.from_numpy((Xf * sf[idx[:, j]][:, None].astype(np.float64)).astype(np.float32)).to(torch.bfloat16)
        term = W[:, j:j + 1].astype(np.float64) * y.double().numpy()
        ref += term
        mag += np.abs(term)
    got = u16_to_float(Y).astype(np.float64)
    # Error budget of the fp32 chain: K roundings of relative size 2^-24 on partial sums bounded by
    # sum|W y|, then one bf16 rounding (half an ulp <= 2^-8 relative to the result).
    bound = np.abs(ref) * 2.0 ** -8 * (1 + 1e-6) + K * 2.0 ** -24 * mag + 1e-45
    assert (np.abs(got - ref) <= bound).all()
    # and where no cancellation occurred it is within one bf16 ulp of the rounded fp64 value
    ref_b = synth.bf16_to_u16(torch.from_numpy(ref).to(torch.float32).to(torch.bfloat16)).astype(np.int32)
    key = lambda a: np.where(a & 0x8000, 0x8000 - (a & 0x7FFF), 0x8000 + a)
    no_cancel = mag <= 4 * np.abs(ref)
    assert no_cancel.mean() > 0.5
    assert np.abs(key(Y.astype(np.int32)) - key(ref_b))[no_cancel].max() <= 1


@pytest.mark.parametrize("K", [1, 2, 8])
def test_combine_round_trip_closed_forms(K):
    rng = np.random.default_rng(K)
    T, E, R, H = 96, 16, 4, 32
    idx, rts, X, p, C, slots, win = _mk(rng, T, K, E, R, H)
    # identity experts, softmax weights (sum to 1 up to fp32 rounding): Y == X exactly,
    # because the fp32 error is far below half a bf16 ulp and X is already bf16.
    logits = rng.standard_normal((T, K)).astype(np.float32)
    W = (np.exp(logits) / np.exp(logits).sum(1, keepdims=True)).astype(np.float32)
    _, Y = oracle.combine(win, slots, W, H)
    assert np.array_equal(u16_to_float(Y), u16_to_float(X))
    # W = 1/K with K a power of two: every product and partial sum is exact.
    _, Y = oracle.combine(win, slots, np.full((T, K), 1.0 / K, np.float32), H)
    assert np.array_equal(u16_to_float(Y), u16_to_float(X))
    # one-hot weights select exactly the chosen expert's output.
    scale = rand_bf16(rng, (E,))
    oracle.expert_scale(win, H, E, R, C, p.n_exp, scale)
    hot = rng.integers(0, K, T)
    W = np.zeros((T, K), np.float32)
    W[np.arange(T), hot] = 1.0
    _, Y = oracle.combine(win, slots, W, H)
    want = torch.from_numpy(u16_to_float(X) * u16_to_float(scale)[idx[np.arange(T), hot]][:, None]).to(torch.bfloat16)
    assert np.array_equal(u16_to_float(Y), want.float().numpy())


# ----------------------------------------------------------------------------- workloads
def test_benchmark_routing_recipes():
    for n in (1, 2):
        wl = synth.config(n)
        idx, w, _, _ = synth.make_routing(wl)
        assert idx.shape == (wl.T, wl.K) and idx.min() >= 0 and idx.max() < wl.E
        srt = np.sort(idx.numpy(), 1)
        assert (np.diff(srt, axis=1) > 0).all()                 # top-k without replacement
        assert np.allclose(w.sum(1).numpy(), 1.0, atol=1e-6)
        p = oracle.plan(idx.numpy(), wl.E, wl.R)
        assert p.status == oracle.OK and p.M.sum() == wl.B
    wl = synth.config(4)
    idx, w, extra, _ = synth.make_routing(wl)
    p = oracle.plan(idx.numpy(), wl.E, wl.R)
    assert p.n_exp.max() >= 10 * wl.B / wl.E                     # hot experts hold > 10x the mean load
    assert (np.diff(np.sort(idx.numpy(), 1), axis=1) > 0).all()


# ----------------------------------------------------------------------------- quantised dispatch
def test_e4m3_conversions_against_torch():
    # decoding: all 256 codes against torch's float8_e4m3fn
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    want = codes.view(torch.float8_e4m3fn).float().numpy()
    for c in range(256):
        got = oracle.e4m3_to_float(c)
        assert (np.isnan(got) and np.isnan(want[c])) or got == want[c], c
    # encoding: every representable value, every midpoint between neighbours, and random values in [-448, 448]
    finite = np.sort(np.unique(want[np.isfinite(want)]))
    mids = (finite[:-1].astype(np.float64) + finite[1:].astype(np.float64)) / 2
    rng = np.random.default_rng(3)
    vals = np.concatenate([finite, mids.astype(np.float32), np.nextafter(mids.astype(np.float32), np.float32(1e9)),
                           np.nextafter(mids.astype(np.float32), np.float32(-1e9)),
                           rng.uniform(-448, 448, 20000).astype(np.float32),
                           (rng.standard_normal(20000) * 0.01).astype(np.float32)]).astype(np.float32)
    ref = torch.from_numpy(vals).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for v, r in zip(vals, ref):
        got = oracle.float_to_e4m3(v)
        if v == 0:
            assert got & 0x7F == 0
        else:
            assert got == r, (v, got, r)
    # beyond the largest finite value the conversion clamps (it never produces NaN from a finite input)
    for v in (448.0, 449.0, 463.9, 464.0, 480.0, 1e9, np.inf):
        assert oracle.float_to_e4m3(v) == 0x7E and oracle.float_to_e4m3(-v) == 0xFE
    assert oracle.float_to_e4m3(float("nan")) & 0x7F == 0x7F


@pytest.mark.parametrize("T,K,E,R,H", [(40, 2, 8, 4, 64), (77, 8, 16, 2, 256)])
def test_dispatch_quant_against_torch_pipeline_and_error_bound(T, K, E, R, H):
    rng = np.random.default_rng(T)
    idx, rts = random_case(rng, T, K, E, R)
    X = rand_bf16(rng, (T, H))
    X[3] = 0                                          # an all-zero row: scale 1, codes 0
    X[5, 7] = synth.bf16_to_u16(torch.tensor([300.0]).to(torch.bfloat16))[0]     # a row with an outlier
    p = oracle.plan(idx, E, R, rts)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx, E, R, p, C, rts)
    wq = np.full((R * C, H), 0xAB, np.uint8)
    sc = np.full((R * C,), -1.0, np.float32)
    assert oracle.dispatch_quant(X, slots, wq, sc) == oracle.OK

    # the same pipeline with library ops: fp32 amax, two fp32 divisions, fp32 product, torch's e4m3 rounding
    xf = torch.from_numpy(u16_to_float(X))
    amax = xf.abs().amax(dim=1)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
    # (scalar / tensor would be reciprocal-then-multiply in torch: two roundings; divide tensor by tensor)
    inv = torch.where(amax > 0, torch.full_like(amax, 448.0) / amax, torch.ones_like(amax))
    codes = (xf * inv[:, None]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    owner = np.full(R * C, -1)
    owner[slots.reshape(-1)] = np.repeat(np.arange(T), K)
    for row in range(R * C):
        t = owner[row]
        if t < 0:
            assert (wq[row] == 0xAB).all() and sc[row] == -1.0          # untouched
        else:
            assert np.array_equal(wq[row] & 0x7F != 0, codes[t] & 0x7F != 0)
            nz = codes[t] & 0x7F != 0
            assert np.array_equal(wq[row][nz], codes[t][nz]) and sc[row] == scale[t].item()
    # the largest element of every non-zero row maps to the largest code, and the round trip is within the
    # format's error: half an ulp of a 3-bit mantissa (2^-4 relative) or half a subnormal step of the scaled row
    deq = torch.from_numpy(wq[slots[:, 0]]).view(torch.float8_e4m3fn).float() * torch.from_numpy(sc[slots[:, 0]])[:, None]
    err = (deq - xf).abs()
    bound = xf.abs() * 2.0 ** -4 * (1 + 1e-5) + scale[:, None] * 2.0 ** -10 * (1 + 1e-5)
    assert bool((err <= bound).all())
    top = (wq[slots[:, 0]] & 0x7F).max(1)
    assert (top[amax.numpy() > 0] == 0x7E).all() and top[3] == 0


@pytest.mark.parametrize("T,K,E,R,H,group", [(40, 2, 8, 4, 256, 128), (33, 8, 16, 2, 384, 128), (20, 4, 8, 2, 96, 32)])
def test_dispatch_quant_group_against_torch_pipeline_rowwise_slices_and_error_bound(T, K, E, R, H, group):
    rng = np.random.default_rng(T + H)
    idx, rts = random_case(rng, T, K, E, R)
    X = rand_bf16(rng, (T, H))
    X[3] = 0                                          # an all-zero row: every scale 1, codes 0
    X[4, group:2 * group] = 0                         # one all-zero group inside a live row
    X[5, 7] = synth.bf16_to_u16(torch.tensor([300.0]).to(torch.bfloat16))[0]     # an outlier: only ITS group's scale grows
    X[:, :group] = (u16_to_float(X[:, :group]) * 64).astype(np.float32).view(np.uint32) >> 16   # groups of very different magnitude
    G = H // group
    p = oracle.plan(idx, E, R, rts)
    C = int(p.n_recv.max()) + 1
    _, slots = oracle.slots(idx, E, R, p, C, rts)
    wq = np.full((R * C, H), 0xAB, np.uint8)
    sc = np.full((R * C, G), -1.0, np.float32)
    assert oracle.dispatch_quant_group(X, slots, wq, sc, group) == oracle.OK

    # (1) library ops: fp32 amax per group, two fp32 divisions, fp32 product, torch's e4m3 rounding
    xf = torch.from_numpy(u16_to_float(X)).view(T, G, group)
    amax = xf.abs().amax(dim=2)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
    inv = torch.where(amax > 0, torch.full_like(amax, 448.0) / amax, torch.ones_like(amax))
    codes = (xf * inv[:, :, None]).to(torch.float8_e4m3fn).view(torch.uint8).numpy().reshape(T, H)
    owner = np.full(R * C, -1)
    owner[slots.reshape(-1)] = np.repeat(np.arange(T), K)
    for row in range(R * C):
        t = owner[row]
        if t < 0:
            assert (wq[row] == 0xAB).all() and (sc[row] == -1.0).all()          # untouched
        else:
            nz = codes[t] & 0x7F != 0
            assert np.array_equal(wq[row] & 0x7F != 0, nz)
            assert np.array_equal(wq[row][nz], codes[t][nz]) and np.array_equal(sc[row], scale[t].numpy())

    # (2) every group is a row of its own for the row-wise function: X viewed as [T*G, group], one slot per little row
    little = np.ascontiguousarray(X.reshape(T * G, group))
    lw = np.zeros((T * G, group), np.uint8)
    ls = np.zeros((T * G,), np.float32)
    assert oracle.dispatch_quant(little, np.arange(T * G, dtype=np.int64)[:, None], lw, ls) == oracle.OK
    first = slots[:, 0]
    assert np.array_equal(wq[first], lw.reshape(T, H)) and np.array_equal(sc[first], ls.reshape(T, G))
    # ... and one group spanning the row IS the row-wise function
    wq1 = np.zeros((R * C, H), np.uint8)
    sc1 = np.zeros((R * C, 1), np.float32)
    wq2 = np.zeros((R * C, H), np.uint8)
    sc2 = np.zeros((R * C,), np.float32)
    assert oracle.dispatch_quant_group(X, slots, wq1, sc1, H) == oracle.OK
    assert oracle.dispatch_quant(X, slots, wq2, sc2) == oracle.OK
    assert np.array_equal(wq1, wq2) and np.array_equal(sc1[:, 0], sc2)

    # (3) round trip within the format's error, group by group; the largest element of a live group takes the top code
    deq = (torch.from_numpy(wq[first]).view(torch.float8_e4m3fn).float().view(T, G, group) *
           torch.from_numpy(sc[first])[:, :, None])
    err = (deq - xf).abs()
    bound = xf.abs() * 2.0 ** -4 * (1 + 1e-5) + scale[:, :, None] * 2.0 ** -10 * (1 + 1e-5)
    assert bool((err <= bound).all())
    top = (wq[first] & 0x7F).reshape(T, G, group).max(2)
    assert (top[amax.numpy() > 0] == 0x7E).all() and (top[3] == 0).all() and top[4, 1] == 0
    # H not a multiple of the group is refused
    assert oracle.dispatch_quant_group(X, slots, wq, sc, group - 1 if H % (group - 1) else group + 1) != oracle.OK


# ----------------------------------------------------------------------------- gating
@pytest.mark.parametrize("T,E,K", [(64, 16, 2), (200, 256, 8), (33, 8, 8), (50, 40, 1), (10, 4096, 32)])
def test_gate_topk_against_torch(T, E, K):
    rng = np.random.default_rng(E + K)
    logits = rng.standard_normal((T, E)).astype(np.float32) * 3
    st, idx, w = oracle.gate_topk(logits, K)
    assert st == oracle.OK
    top = torch.topk(torch.from_numpy(logits), K, dim=1)            # distinct values: the order is unique
    assert np.array_equal(idx, top.indices.numpy())
    ref = torch.softmax(top.values.double(), dim=1).numpy()
    assert np.abs(w - ref).max() <= 2e-7 + 4e-7 * ref.max()
    assert np.allclose(w.sum(1), 1.0, atol=3e-7)
    assert (np.diff(w, axis=1) <= 0).all()                           # descending logits => descending weights


def test_gate_topk_ties_take_the_lower_index_first():
    logits = np.array([[1.0, 5.0, 5.0, 0.0, 5.0, 2.0],
                       [0.0, 0.0, 0.0, 0.0, 0.0, 0.0],
                       [-1.0, -1.0, 3.0, 3.0, -2.0, 3.0]], np.float32)
    st, idx, w = oracle.gate_topk(logits, 4)
    # the definition, literally: sort experts by (logit descending, index ascending)
    want = [sorted(range(6), key=lambda e: (-row[e], e))[:4] for row in logits]
    assert idx.tolist() == want == [[1, 2, 4, 5], [0, 1, 2, 3], [2, 3, 5, 0]]
    assert np.allclose(w[1], 0.25) and w[0, 0] == w[0, 1] == w[0, 2]
    assert oracle.gate_topk(logits, 7)[0] == oracle.ERR_INVALID_ARG   # K > E


@pytest.mark.parametrize("K", [2, 8, 28, 32])
def test_gate_weights_within_the_fp32_budget_of_the_exact_softmax(K):
    """One side's share of the gate-weight tolerance the GPU tests use, (2K + 8) * 2^-24 between the two sides:
    against the softmax of the same fp32 differences l_j - l_0 evaluated in fp64, the oracle's fp32 weights are off by
    at most (K + 2) half-ulps -- the
    exponentials (<= 1 ulp each), the K - 1 roundings of the ascending sum, the division.  The adversarial case is
    many EQUAL selected logits: every addition of the sum then rounds the same way (a random case stays near
    sqrt(K) half-ulps), which is why the budget is linear in K."""
    E, T = 48, 4000
    rng = np.random.default_rng(K)
    worst = 0.0
    for equal_share in (0.0, 0.7):
        logits = (rng.standard_normal((T, E)) * 3).astype(np.float32)
        n_eq = int(E * equal_share)
        if n_eq:
            logits[:, :n_eq] = (rng.standard_normal((T, 1)) * 2).astype(np.float32)    # one value, repeated
        st, idx, w = oracle.gate_topk(logits, K)
        assert st == oracle.OK
        sel = np.take_along_axis(logits, idx.astype(np.int64), axis=1)
        # the fp32 differences l_j - l_0 are part of the definition (both sides form the same ones); everything
        # after them is evaluated exactly here
        ex = np.exp((sel - sel[:, :1]).astype(np.float32).astype(np.float64))
        exact = ex / ex.sum(1, keepdims=True)
        rel = np.abs(w.astype(np.float64) - exact) / exact
        assert rel.max() <= (K + 2) * 2.0 ** -24, (K, equal_share, rel.max())
        worst = max(worst, rel.max())
    if K >= 28:          # the linear term is really there: the equal-logit case gets well past a sqrt(K) budget
        assert worst > 2.5 * np.sqrt(K) * 2.0 ** -25, worst


# ----------------------------------------------------------------------------- multi-rank decomposition
def test_layout_per_rank_plus_notify_equals_the_global_plan():
    """Layout is local (Section 5.2): planning each rank's tokens alone gives that rank's row of M and
    its small offsets; Notify on the gathered rows gives the global large offsets."""
    rng = np.random.default_rng(12)
    T, K, E, R = 300, 4, 12, 4
    idx, rts = random_case(rng, T, K, E, R, replace=True)
    whole = oracle.plan(idx, E, R, rts)
    rows = []
    for r in range(R):
        local = idx[rts[r]:rts[r + 1]]
        only_r = np.array([0] * (r + 1) + [len(local)] * (R - r), np.int32)     # rank r owns every local token
        pr = oracle.plan(local, E, R, only_r)
        assert pr.status == oracle.OK
        assert np.array_equal(pr.s, whole.s[rts[r]:rts[r + 1]])
        assert not np.delete(pr.M, r, axis=0).any()
        rows.append(pr.M[r])
    M = np.stack(rows)
    st, c_rank, o, n_exp, n_recv = oracle.notify(M)
    assert st == oracle.OK and np.array_equal(M, whole.M)
    for a, b in ((c_rank, whole.c_rank), (o, whole.o), (n_exp, whole.n_exp), (n_recv, whole.n_recv)):
        assert np.array_equal(a, b)


# ----------------------------------------------------------------------------- aligned expert starts
@pytest.mark.parametrize("align", [1, 2, 8, 128])
@pytest.mark.parametrize("case", list(cases()), ids=lambda c: f"T{c[0]}K{c[1]}E{c[2]}R{c[3]}{'rep' if c[4] else ''}")
def test_aligned_layout_against_library_routines(case, align):
    """Expert runs padded to groups of `align` rows: counts and small offsets do not change, starts are
    the exclusive cumulative sum (numpy) of the padded expert counts, restarting per window, and the
    branches of an expert still fill [start, start + count) in stable order."""
    T, K, E, R, _, idx, rts = case
    base = oracle.plan(idx, E, R, rts)
    p = oracle.plan(idx, E, R, rts, align=align)
    assert p.status == oracle.OK
    E_r = E // R
    for name in ("M", "c_rank", "s", "n_exp"):
        assert np.array_equal(getattr(p, name), getattr(base, name)), name
    padded = -(-p.n_exp.astype(np.int64) // align) * align
    per_window = padded.reshape(R, E_r)
    start = (np.cumsum(per_window, 1) - per_window).reshape(-1)            # local first row of every expert
    assert (start % align == 0).all()
    within = np.cumsum(p.M.T, 1) - p.M.T                                    # [E,R]: rows of earlier source ranks
    assert np.array_equal(p.o, start[:, None] + within)
    assert np.array_equal(p.n_recv, per_window.sum(1))
    if align == 1:
        assert np.array_equal(p.o, base.o) and np.array_equal(p.n_recv, base.n_recv)

    C = int(p.n_recv.max()) + align
    st, slots = oracle.slots(idx, E, R, p, C, rts)
    assert st == oracle.OK
    st, e_start, e_count = oracle.expert_ranges(E, R, C, p.n_exp, align=align)
    assert st == oracle.OK
    assert np.array_equal(e_start, (np.arange(E) // E_r) * C + start) and np.array_equal(e_count, p.n_exp)
    flat_e, flat_slot = idx.reshape(-1), slots.reshape(-1)
    assert len(np.unique(flat_slot)) == T * K                               # no two branches share a row
    for e in range(E):
        rows = flat_slot[flat_e == e]                                       # flat (t, j) order = stable order
        assert np.array_equal(rows, e_start[e] + np.arange(p.n_exp[e]))
    # one row short of the padded need is a capacity error
    if T:
        assert oracle.slots(idx, E, R, p, int(p.n_recv.max()) - 1, rts)[0] == oracle.ERR_CAPACITY


def test_aligned_layout_moves_rows_but_not_results():
    """Dispatch + scale experts + combine give bit-identical Y for every alignment, and padding rows
    keep the caller's bytes."""
    rng = np.random.default_rng(77)
    T, K, E, R, H = 150, 4, 12, 3, 24
    idx, rts = random_case(rng, T, K, E, R, replace=True)
    X = rand_bf16(rng, (T, H))
    W = rng.random((T, K), dtype=np.float32)
    scale = rand_bf16(rng, (E,))
    outs = []
    for align in (1, 4, 16):
        p = oracle.plan(idx, E, R, rts, align=align)
        C = int(p.n_recv.max())
        st, slots = oracle.slots(idx, E, R, p, C, rts)
        win = np.full((R * C, H), 0x7FC1, np.uint16)
        assert oracle.dispatch(X, slots, win) == oracle.OK
        used = np.zeros(R * C, bool)
        used[slots.reshape(-1)] = True
        assert (win[~used] == 0x7FC1).all() and used.sum() == T * K
        assert oracle.expert_scale(win, H, E, R, C, p.n_exp, scale, align=align) == oracle.OK
        assert (win[~used] == 0x7FC1).all()                                 # the expert op skips padding rows
        st, Y = oracle.combine(win, slots, W, H)
        outs.append(Y)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_aligned_notify_rejects_bad_alignment():
    M = np.ones((2, 4), np.int32)
    assert oracle.notify(M, align=0)[0] == oracle.ERR_INVALID_ARG
    st, c_rank, o, n_exp, n_recv = oracle.notify(M, align=4)
    assert st == oracle.OK and list(n_recv) == [8, 8] and list(o[:, 0]) == [0, 4, 0, 4] and list(o[:, 1]) == [1, 5, 1, 5]


def test_brute_force_all_routings_tiny_aligned():
    """The same 4^6 routings with expert runs padded to 4 rows, against the literal definition: an
    expert starts after the padded runs of the earlier experts of its window, and inside the run the
    blocks of lower source ranks come first."""
    T, K, E, R, A = 3, 2, 4, 2, 4
    rts = np.array([0, 2, 3], np.int32)
    src = [0, 0, 1]
    E_r = E // R
    branches = [(t, j) for t in range(T) for j in range(K)]
    for combo in itertools.product(range(E), repeat=T * K):
        idx = np.array(combo, np.int32).reshape(T, K)
        p = oracle.plan(idx, E, R, rts, align=A)
        count = [sum(1 for (t, j) in branches if idx[t, j] == e) for e in range(E)]
        for e in range(E):
            start = sum(-(-count[e2] // A) * A for e2 in range((e // E_r) * E_r, e))
            for r in range(R):
                lower = sum(1 for (t, j) in branches if idx[t, j] == e and src[t] < r)
                assert p.o[e, r] == start + lower
        for d in range(R):
            assert p.n_recv[d] == sum(-(-count[e] // A) * A for e in range(d * E_r, (d + 1) * E_r))


@pytest.mark.parametrize("align,tile_rows", [(1, 4), (8, 8), (16, 5), (1, 1000)])
def test_expert_tiles_against_numpy(align, tile_rows):
    """The tile list covers every expert's run exactly once, in window order, with only the last tile of an
    expert short; its length is the sum of ceil(n_exp / tile_rows) (numpy)."""
    rng = np.random.default_rng(321 + align + tile_rows)
    T, K, E, R = 300, 4, 12, 3
    idx, rts = random_case(rng, T, K, E, R, replace=True)
    idx[idx == 5] = 4                                         # expert 5 receives nothing: it has no tile
    p = oracle.plan(idx, E, R, rts, align=align)
    C = int(p.n_recv.max()) + 3
    _, e_start, e_count = oracle.expert_ranges(E, R, C, p.n_exp, align=align)
    want_n = int(np.sum(-(-p.n_exp.astype(np.int64) // tile_rows)))
    st, t_e, t_row, t_valid, n = oracle.expert_tiles(E, R, C, p.n_exp, tile_rows, want_n + 5, align=align)
    assert st == oracle.OK and n == want_n
    assert (t_e[n:] == -1).all() and (t_row[n:] == -1).all()                      # nothing beyond the list
    assert (np.diff(t_e[:n]) >= 0).all() and 5 not in t_e[:n]                    # window order = expert order
    covered = np.zeros(R * C, np.int32)
    for k in range(n):
        e = t_e[k]
        off = t_row[k] - e_start[e]
        assert off % tile_rows == 0 and 0 <= off < e_count[e]
        assert t_valid[k] == min(tile_rows, e_count[e] - off)
        covered[t_row[k]:t_row[k] + t_valid[k]] += 1
    _, slots = oracle.slots(idx, E, R, p, C, rts)
    used = np.zeros(R * C, np.int32)
    used[slots.reshape(-1)] = 1
    assert np.array_equal(covered, used)                                          # every received row in exactly one tile
    # a short buffer: the count is still the full one, entries beyond the buffer are not written
    st, t_e2, _, _, n2 = oracle.expert_tiles(E, R, C, p.n_exp, tile_rows, 3, align=align)
    assert n2 == want_n and np.array_equal(t_e2, t_e[:3])
