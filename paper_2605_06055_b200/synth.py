"""Seeded synthetic MoE routing workloads (inputs only).

This module draws the *inputs* of the dispatch/combine path -- hidden states X,
routing indexes K, routing weights W, per-expert stand-in scales -- on the host
with a seeded torch CPU generator.  It holds none of the method's arithmetic
(no counts, offsets, slots, scatter or reduction), so the CUDA path and the CPU
oracle can both be fed the same bit-identical arrays without sharing code.

Shapes follow public MoE model shapes (DeepSeek-V3-like: H=7168, E=256, K=8;
Mixtral-like: H=4096, E=8, K=2) and stand in for the serving workloads the
paper measures on; no routing trace, prompt or weight of any model is used.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

PREFILL, DECODE = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    T: int            # total tokens over all virtual ranks
    H: int
    E: int
    R: int
    K: int
    schedule: int     # PREFILL or DECODE
    routing: str      # "logits" | "uniform" | "zipf" | "replace"
    expert_op: str    # "identity" | "scale"
    seed: int
    zipf_s: float = 1.2
    rank_tokens: Optional[tuple] = None   # tokens per rank; None => uniform T/R

    @property
    def B(self) -> int:
        return self.T * self.K


def config(n: int, T: Optional[int] = None, schedule: Optional[int] = None) -> Workload:
    """The five benchmark configurations (1-based)."""
    if n == 1:
        return Workload("c1_tiny", 256, 1024, 16, 4, 2, PREFILL, "logits", "identity", 1001)
    if n == 2:
        return Workload("c2_decode_dsv3", 2048, 7168, 256, 16, 8, DECODE, "uniform", "scale", 1002)
    if n == 3:
        return Workload("c3_prefill_dsv3", 32768, 7168, 256, 8, 8, PREFILL, "uniform", "identity", 1003)
    if n == 4:
        return Workload("c4_prefill_dsv3_zipf", 32768, 7168, 256, 8, 8, PREFILL, "zipf", "identity", 1004)
    if n == 5:
        T = 8192 if T is None else T
        sch = PREFILL if schedule is None else schedule
        return Workload(f"c5_mixtral_T{T}_{'prefill' if sch == PREFILL else 'decode'}", T, 4096, 8, 8, 2, sch,
                        "uniform", "identity", 1005 * 100000 + T)
    raise ValueError(n)


@dataclass
class Inputs:
    wl: Workload
    topk_idx: torch.Tensor                 # [T,K] int32
    topk_w: torch.Tensor                   # [T,K] float32
    rank_tok_start: np.ndarray             # [R+1] int32
    X: Optional[torch.Tensor] = None       # [T,H] bfloat16
    scale: Optional[torch.Tensor] = None   # [E] bfloat16 (expert_op == "scale")
    extra: dict = field(default_factory=dict)


def bf16_to_u16(t: torch.Tensor) -> np.ndarray:
    """Reinterpret a CPU bf16 tensor as a numpy uint16 array (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def u16_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def _softmax_rows(logits: torch.Tensor) -> torch.Tensor:
    # fp32 softmax over the chosen top-k logits: exp(l - max) / sum.
    m = logits.max(dim=1, keepdim=True).values
    ex = torch.exp(logits - m)
    return (ex / ex.sum(dim=1, keepdim=True)).to(torch.float32)


def rank_tok_start(wl: Workload) -> np.ndarray:
    if wl.rank_tokens is None:
        assert wl.T % wl.R == 0
        per = [wl.T // wl.R] * wl.R
    else:
        per = list(wl.rank_tokens)
        assert len(per) == wl.R and sum(per) == wl.T
    return np.concatenate([[0], np.cumsum(per)]).astype(np.int32)


def make_routing(wl: Workload):
    """Routing indexes and weights only (cheap; used by planning tests)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed)
    T, E, K = wl.T, wl.E, wl.K
    extra = {}
    if wl.routing == "logits":
        logits = torch.randn(T, E, generator=g, dtype=torch.float32)
        top = torch.topk(logits, K, dim=1)
        idx, w = top.indices, _softmax_rows(top.values)
    elif wl.routing == "uniform":
        scores = torch.rand(T, E, generator=g, dtype=torch.float32)
        idx = torch.topk(scores, K, dim=1).indices
        w = _softmax_rows(torch.randn(T, K, generator=g, dtype=torch.float32))
    elif wl.routing == "zipf":
        perm = torch.randperm(E, generator=g)
        p = torch.arange(1, E + 1, dtype=torch.float64) ** (-wl.zipf_s)
        logp = torch.empty(E, dtype=torch.float64)
        logp[perm] = torch.log(p / p.sum())
        u = torch.rand(T, E, generator=g, dtype=torch.float64).clamp_(1e-300, 1.0)
        gumbel = -torch.log(-torch.log(u).clamp_min(1e-300))
        idx = torch.topk(logp[None, :] + gumbel, K, dim=1).indices      # K distinct experts ~ Zipf
        w = _softmax_rows(torch.randn(T, K, generator=g, dtype=torch.float32))
        extra["expert_perm"] = perm.numpy()
    elif wl.routing == "replace":
        idx = torch.randint(0, E, (T, K), generator=g)                  # duplicates allowed
        w = _softmax_rows(torch.randn(T, K, generator=g, dtype=torch.float32))
    else:
        raise ValueError(wl.routing)
    return idx.to(torch.int32).contiguous(), w.contiguous(), extra, g


def make_inputs(wl: Workload, with_x: bool = True, pin: bool = False) -> Inputs:
    idx, w, extra, g = make_routing(wl)
    X = scale = None
    if wl.expert_op == "scale":
        scale = (0.5 + torch.rand(wl.E, generator=g, dtype=torch.float32)).to(torch.bfloat16)
    if with_x:
        X = torch.empty(wl.T, wl.H, dtype=torch.bfloat16, pin_memory=pin)
        step = max(1, (1 << 24) // wl.H)
        for t0 in range(0, wl.T, step):      # chunked so the fp32 draw stays small
            t1 = min(wl.T, t0 + step)
            X[t0:t1] = torch.randn(t1 - t0, wl.H, generator=g, dtype=torch.float32).to(torch.bfloat16)
    return Inputs(wl, idx, w, rank_tok_start(wl), X, scale, extra)
