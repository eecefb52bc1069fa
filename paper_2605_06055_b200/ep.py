"""One expert-parallel rank per process: the host-side order of the multi-rank path.

    layout (local)  ->  all-gather of the count rows  ->  notify  ->  dispatch into every rank's
    window  ->  barrier  ->  experts  ->  barrier  ->  combine from every rank's window

All compute is in libmoecomm (moe_layout, moe_notify, moe_dispatch_peers, moe_combine_peers); this
module only exchanges the R x E count matrix with torch.distributed and keeps the phases in order.
The windows of the other ranks must be mapped into this process (a table of R device addresses):
`symmetric_windows` obtains them from torch's symmetric memory where that is available.

The test suite exercises this on ONE GPU: every rank a context of one process with separate window
allocations, and two ranks as two processes whose windows are mapped into each other over CUDA IPC
(counts over a gloo group).  The count exchange is also tested with two gloo ranks on CPU.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import binding


def all_gather_counts(counts_row: torch.Tensor, group=None) -> torch.Tensor:
    """Prefill Notify's metadata exchange: every rank contributes its row [E] of the count matrix and
    receives the whole matrix [R, E] (row r from rank r)."""
    world = dist.get_world_size(group)
    staged = counts_row.is_cuda and dist.get_backend(group) == "gloo"     # gloo moves host tensors only
    src = counts_row.cpu() if staged else counts_row
    flat = torch.empty(world * src.numel(), dtype=src.dtype, device=src.device)
    dist.all_gather_into_tensor(flat, src.contiguous().view(-1), group=group)
    out = flat.view(world, src.numel())
    return out.to(counts_row.device) if staged else out


def symmetric_windows(capacity_rows: int, H: int, device, group=None):
    """Allocates this rank's window in symmetric memory and returns (window, table of all ranks' window
    addresses as an int64 CUDA tensor).  Needs torch's symmetric-memory support and peer access."""
    import torch.distributed._symmetric_memory as symm_mem
    win = symm_mem.empty((capacity_rows, H), dtype=torch.bfloat16, device=device)
    hdl = symm_mem.rendezvous(win, group if group is not None else dist.group.WORLD)
    bases = torch.tensor([int(p) for p in hdl.buffer_ptrs], dtype=torch.int64, device=device)
    return win, bases


class EpRank:
    """The calls of one rank, in the order the schedules prescribe."""

    def __init__(self, T_local_max: int, H: int, E: int, K: int, device, group=None):
        self.group = group
        self.rank = dist.get_rank(group)
        self.R = dist.get_world_size(group)
        self.comm = binding.MoeComm(T_local_max, H, E, self.R, K, device)
        self.counts_row = torch.zeros(E, dtype=torch.int32, device=device)
        self.E = E

    def plan(self, schedule: int, topk_idx_local: torch.Tensor) -> torch.Tensor:
        self.comm.moe_layout(schedule, topk_idx_local, self.rank, self.counts_row)
        counts_all = all_gather_counts(self.counts_row, self.group)      # metadata only, no payload
        self.comm.moe_notify(counts_all)
        return counts_all

    def dispatch(self, x_local: torch.Tensor, window_bases: torch.Tensor, capacity_rows: int) -> None:
        self.comm.moe_dispatch_peers(x_local, window_bases, capacity_rows)
        torch.cuda.current_stream().synchronize()
        dist.barrier(self.group)                 # every rank's rows have landed before any expert reads its window

    def dispatch_quant(self, x_local: torch.Tensor, window_q_bases: torch.Tensor, scale_bases: torch.Tensor,
                       capacity_rows: int) -> None:
        """Row-wise quantised dispatch: e4m3 codes into every rank's code window, one fp32 scale per row into
        every rank's scale tensor (tables of R device addresses each)."""
        self.comm.moe_dispatch_quant_peers(x_local, window_q_bases, scale_bases, capacity_rows)
        torch.cuda.current_stream().synchronize()
        dist.barrier(self.group)

    def combine(self, window_bases: torch.Tensor, capacity_rows: int, topk_w_local: torch.Tensor,
                y_local: torch.Tensor) -> None:
        dist.barrier(self.group)                 # every expert has written its outputs
        self.comm.moe_combine_peers(window_bases, capacity_rows, topk_w_local, y_local)

    def status(self) -> int:
        return self.comm.moe_status()
