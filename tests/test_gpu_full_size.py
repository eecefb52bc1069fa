"""Full benchmark sizes (configs 3 and 4) in the launch configuration bench.py times.

The oracle cannot replay 4 GB of rows in seconds, so: every integer the plan
produces is compared in full (the oracle's plan is cheap); dispatched rows and
combined outputs are compared on sampled branches / tokens that the oracle
computes one by one from the host inputs; and properties that hold at any size
cover the rest (padding rows untouched, column checksums of the windows,
identity round trip Y == X).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06055_b200 import binding, synth

import harness

pytestmark = pytest.mark.gpu


def as_u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("n", [3, 4])
def test_full_size_prefill_sampled(n):
    dev = torch.device("cuda:0")
    wl = synth.config(n)
    inp = synth.make_inputs(wl)
    idx_np = inp.topk_idx.numpy()
    p = oracle.plan(idx_np, wl.E, wl.R)
    assert p.status == oracle.OK
    if n == 4:
        assert p.n_exp.max() >= 10 * wl.B / wl.E
    C = (int(p.n_recv.max()) + 7) // 8 * 8                     # as bench.py sizes it
    st, slots = oracle.slots(idx_np, wl.E, wl.R, p, C)
    assert st == oracle.OK

    comm = binding.MoeComm(wl.T, wl.H, wl.E, wl.R, wl.K, dev)
    X, idx, w = inp.X.to(dev), inp.topk_idx.to(dev), inp.topk_w.to(dev)
    windows = torch.empty((wl.R * C, wl.H), dtype=torch.bfloat16, device=dev)
    windows.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
    Y = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device=dev)
    got_slots = torch.empty((wl.T, wl.K), dtype=torch.int32, device=dev)
    comm.moe_plan(wl.schedule, idx)
    comm.moe_slots(C, got_slots)
    comm.moe_dispatch(X, windows, C)
    comm.moe_combine(windows, C, w, Y)
    assert comm.moe_status() == 0

    # -- integers: everything, bit-exact
    v = comm.moe_plan_view()
    for k, name in {"counts": "M", "c_rank": "c_rank", "small_off": "s", "large_off": "o", "n_exp": "n_exp",
                    "n_recv": "n_recv"}.items():
        assert np.array_equal(v[k].cpu().numpy(), getattr(p, name)), k
    assert np.array_equal(got_slots.cpu().numpy().astype(np.int64), slots)

    # -- dispatched rows: sampled branches against the host rows of X, bit-exact
    rng = np.random.default_rng(n)
    bt = rng.integers(0, wl.T, 3000)
    bj = rng.integers(0, wl.K, 3000)
    rows = torch.from_numpy(slots[bt, bj]).to(dev)
    got = as_u16(windows.index_select(0, rows))
    assert np.array_equal(got, synth.bf16_to_u16(inp.X)[bt])
    # -- padding rows of every segment were never written
    for d in range(wl.R):
        pad = windows[d * C + int(p.n_recv[d]):(d + 1) * C]
        if pad.numel():
            assert bool((pad.view(torch.int16) == int(np.int16(np.uint16(harness.CANARY)))).all()), d
    # -- any-size property: every token row sits in the windows exactly K times, so the column sums of the
    #    bit patterns over the used rows equal K times the column sums over X (exact in int64)
    used = torch.cat([windows[d * C:d * C + int(p.n_recv[d])] for d in range(wl.R)]) if n == 3 else None
    if used is not None:
        lhs = (used.view(torch.int16).to(torch.int64) & 0xFFFF).sum(0)
        rhs = (X.view(torch.int16).to(torch.int64) & 0xFFFF).sum(0) * wl.K
        assert torch.equal(lhs, rhs)
        del used

    # -- combine: identity experts and weights summing to 1 => Y == X at every element
    assert torch.equal(Y.view(torch.int16), X.view(torch.int16))
    # -- planning folded into the dispatch call: the same bytes everywhere (padding rows included),
    #    and the sampled rows once more against the host copy of X
    windows2 = torch.empty_like(windows)
    windows2.view(torch.int16).fill_(int(np.int16(np.uint16(harness.CANARY))))
    comm.moe_plan_dispatch(wl.schedule, idx, X, windows2, C)
    assert comm.moe_status() == 0
    assert torch.equal(windows2.view(torch.int16), windows.view(torch.int16))
    assert np.array_equal(as_u16(windows2.index_select(0, rows)), synth.bf16_to_u16(inp.X)[bt])
    del windows2
    # -- and sampled tokens against the oracle run on their own rows (inputs come from the host copy of X)
    S = np.sort(rng.choice(wl.T, 256, replace=False))
    Xs = synth.bf16_to_u16(inp.X)[S]
    mini_slots = np.arange(len(S) * wl.K, dtype=np.int64).reshape(len(S), wl.K)
    mini_win = np.zeros((len(S) * wl.K, wl.H), np.uint16)
    assert oracle.dispatch(Xs, mini_slots, mini_win) == oracle.OK
    # scale the mini windows and the device windows with per-row factors so the check is not the identity case
    fac = torch.from_numpy(rng.uniform(0.5, 1.5, (len(S), wl.K)).astype(np.float32)).to(torch.bfloat16)
    mw = synth.u16_to_bf16(mini_win).view(len(S), wl.K, wl.H) * fac[:, :, None]
    mini_win = synth.bf16_to_u16(mw.reshape(len(S) * wl.K, wl.H).contiguous())
    st, want = oracle.combine(mini_win, mini_slots, inp.topk_w.numpy()[S], wl.H)
    srows = torch.from_numpy(slots[S].reshape(-1)).to(dev)
    windows[srows] = (windows[srows].view(len(S), wl.K, wl.H) * fac.to(dev)[:, :, None]).reshape(-1, wl.H)
    comm.moe_combine(windows, C, w, Y)
    assert comm.moe_status() == 0
    got = as_u16(Y.index_select(0, torch.from_numpy(S).to(dev)))
    assert harness.max_ulp_diff(got, want) <= 1
    comm.close()
