"""One expert-parallel rank per process (and per GPU): the host-side order of the multi-rank path.

    layout (local)  ->  all-gather of the count rows (+ every rank's window generation)  ->  notify
    ->  [address handshake, if the cached table is out of date]  ->  dispatch into every rank's window
    ->  barrier  ->  experts  ->  barrier  ->  combine from every rank's window

All compute is in libmoecomm (moe_layout, moe_notify, moe_dispatch_cached, moe_combine_cached); this module
exchanges the R x E count matrix and the window handles with torch.distributed and keeps the phases in order.
Only the library's own kernels touch another rank's window; no torch op is ever given a peer address.

Window addresses (Section 5.3, Decode Combine; Section 6.1): every rank exports a handle of its window
(moe_window_export); the handles are all-gathered and every rank maps the others' windows
(moe_peers_open) -- the address handshake.  In the "cached" mode the handshake is repeated only when the
cached table is out of date: every rank announces the generation of its window together with its count row,
so the test rides on the exchange Notify needs anyway and costs no collective of its own.  In the "handshake"
mode the addresses are exchanged before every dispatch.

Phase order (Section 5.4): with sync="host" the phases are separated by a stream synchronisation and a
process-group barrier.  With sync="device" they are ordered on the GPUs alone: every window allocation carries a
state region behind its rows, a rank signals all ranks after its dispatch / its experts / its combine
(moe_signal_peers) and waits for all ranks' signals before its experts read the window / before its combine /
before its next dispatch (moe_wait_peers, bounded).  A wait kernel occupies its GPU until the signals arrive, so
device ordering needs one GPU per rank; where ranks share a GPU (the tests) `host_fence=True` places a host barrier
between signal and wait, so that every wait finds its signals already there.

The test suite exercises this on ONE GPU (two processes whose windows are mapped into each other over CUDA
inter-process handles, counts over a gloo group) and the exchange logic with two gloo ranks on CPU.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist

from . import binding


def _staged(t: torch.Tensor, group) -> bool:
    return t.is_cuda and dist.get_backend(group) == "gloo"     # gloo moves host tensors only


def all_gather_rows(row: torch.Tensor, group=None) -> torch.Tensor:
    """Every rank contributes one row and receives all of them, [R, len(row)], row r from rank r."""
    world = dist.get_world_size(group)
    staged = _staged(row, group)
    src = row.cpu() if staged else row
    flat = torch.empty(world * src.numel(), dtype=src.dtype, device=src.device)
    dist.all_gather_into_tensor(flat, src.contiguous().view(-1), group=group)
    out = flat.view(world, src.numel())
    return out.to(row.device) if staged else out


def all_gather_counts(counts_row: torch.Tensor, group=None) -> torch.Tensor:
    """Prefill Notify's metadata exchange: every rank contributes its row [E] of the count matrix and
    receives the whole matrix [R, E] (row r from rank r)."""
    return all_gather_rows(counts_row, group)


def all_gather_bytes(mine: bytes, device, group=None) -> bytes:
    """Every rank contributes len(mine) bytes (the same length everywhere) and receives all ranks' bytes back to
    back in rank order.  `device`: where a device-only backend (NCCL) needs the staging tensor."""
    src = torch.frombuffer(bytearray(mine), dtype=torch.uint8)
    on_device = dist.get_backend(group) != "gloo"
    if on_device:
        src = src.to(device)
    return bytes(all_gather_rows(src, group).cpu().reshape(-1).numpy().tobytes())


def addresses_stale(table_generations, announced_generations) -> bool:
    """The cached-address test: the table this rank holds was built from `table_generations`; the ranks have
    just announced `announced_generations`.  None = no table yet."""
    if table_generations is None:
        return True
    return not np.array_equal(np.asarray(table_generations, np.int32), np.asarray(announced_generations, np.int32))


class EpRank:
    """The calls of one rank, in the order the schedules prescribe.
    mode: "handshake" exchanges the window addresses before every dispatch; "cached" tests every step whether the
    cached table is still valid (the generations that came with the count rows are read on the host: one stream
    synchronisation per step) and exchanges them only when it is not; "static" exchanges them once and takes the
    caller's word that no window moves afterwards -- with sync="device" a step then contains no host
    synchronisation at all (call handshake() yourself, on every rank, after attaching a different window)."""

    SLOT_DISPATCHED, SLOT_EXPERTS_DONE, SLOT_COMBINED = 0, 1, 2

    def __init__(self, T_local_max: int, H: int, E: int, K: int, device, group=None, mode: str = "cached",
                 sync: str = "host", host_fence: bool = False, counts: str = "collective"):
        assert mode in ("cached", "handshake", "static") and sync in ("host", "device")
        # counts="device": the count rows travel by the library's own stores into every rank's mailbox
        # (moe_push_counts / moe_notify_peers) instead of an all-gather of the process group; no generations travel
        # with them, so the addresses are static
        assert counts in ("collective", "device") and (counts == "collective" or mode == "static")
        self.counts, self.plan_epoch = counts, 0
        self.group, self.mode, self.device = group, mode, device
        self.sync, self.host_fence, self.epoch = sync, host_fence, 0
        self.rank = dist.get_rank(group)
        self.R = dist.get_world_size(group)
        self.E, self.H = E, H
        self.comm = binding.MoeComm(T_local_max, H, E, self.R, K, device)
        # what this rank sends in the metadata exchange: its count row [E], then its window generation [1]
        self.message = torch.zeros(E + 1, dtype=torch.int32, device=device)
        self.counts_row = self.message[:E]
        self.window = None
        self.capacity, self.flags = 0, 0
        self.generation = 0                 # of this rank's own window; 0 = none attached
        self.table_generations = None       # generations the installed address table was built from
        self.announced = None               # generations gathered by the latest plan()
        self.handshakes = 0

    # -- windows -------------------------------------------------------------------------------------
    def new_window(self, capacity_rows: int, quant: bool = False, quant_group: bool = False) -> torch.Tensor:
        """Allocates this rank's window with its state region behind the rows (zeroed) and, with quant=True
        (one scale per row) or quant_group=True (one per 128 elements), the code window and scale tensor of the
        quantised dispatch behind that; attaches it and returns the [capacity_rows, H] view of the rows."""
        assert not (quant and quant_group)
        flags = binding.MOE_WINDOW_STATE | (binding.MOE_WINDOW_QUANT if quant else 0) | \
            (binding.MOE_WINDOW_QUANT_GROUP if quant_group else 0) | \
            (binding.MOE_WINDOW_COUNTS if self.counts == "device" else 0)
        nbytes = self.comm.moe_window_bytes(capacity_rows, flags)
        backing = torch.zeros(nbytes // 2, dtype=torch.bfloat16, device=self.device)
        self.attach_window(backing, capacity_rows, flags)
        return backing[:capacity_rows * self.H].view(capacity_rows, self.H)

    def quant_views(self):
        """(codes [capacity_rows, H] uint8, scales fp32) of this rank's window allocation; scales are [capacity_rows]
        with MOE_WINDOW_QUANT, [capacity_rows, H // 128] with MOE_WINDOW_QUANT_GROUP."""
        assert self.flags & (binding.MOE_WINDOW_QUANT | binding.MOE_WINDOW_QUANT_GROUP)
        per_row = self.H // 128 if self.flags & binding.MOE_WINDOW_QUANT_GROUP else 1
        raw = self.window.view(torch.uint8)
        scale_bytes = self.capacity * per_row * 4
        scales_at = self.comm.moe_window_bytes(self.capacity, self.flags) - (scale_bytes + 255) // 256 * 256
        codes_at = scales_at - (self.capacity * self.H + 255) // 256 * 256
        codes = raw[codes_at:codes_at + self.capacity * self.H].view(self.capacity, self.H)
        scales = raw[scales_at:scales_at + scale_bytes].view(torch.float32)
        return codes, (scales.view(self.capacity, per_row) if per_row > 1 or self.flags & binding.MOE_WINDOW_QUANT_GROUP
                       else scales)

    def attach_window(self, window: torch.Tensor, capacity_rows: int, flags: int = 0) -> None:
        """This rank's window from now on: a contiguous bf16 tensor whose first capacity_rows * H elements are the
        rows (the same capacity on every rank) and which holds, behind them, the parts that `flags` (MOE_WINDOW_*)
        names: moe_window_bytes(capacity_rows, flags) bytes in all, every rank with the same flags.  A new window
        gets a new generation, which makes every rank's cached table stale at the next plan()."""
        assert window.dtype == torch.bfloat16 and window.is_contiguous()
        assert window.numel() * 2 >= self.comm.moe_window_bytes(capacity_rows, flags)
        new_state = self._state_region(window, capacity_rows) if flags & binding.MOE_WINDOW_STATE else None
        if self.sync == "device" and new_state is not None and self.window is not None and self.epoch > 0:
            # The epochs move with the window: once every signal of the finished step has arrived in the old state
            # region (the combine-done signals are a step's last), it is copied behind the new rows.
            old_state = self._state_region(self.window, self.capacity) if self.flags & binding.MOE_WINDOW_STATE else None
            if old_state is not None:
                self.comm.moe_wait_peers(self.SLOT_COMBINED, self.epoch)
                new_state.copy_(old_state)
        self.window, self.capacity, self.flags = window, int(capacity_rows), int(flags)
        self.generation += 1
        self.message[self.E:].fill_(self.generation)

    def _state_region(self, window: torch.Tensor, capacity_rows: int):
        """The state region behind the rows of a window allocation that has one."""
        state = binding.moe_state_bytes(self.R) // 2
        start = self.comm.moe_window_bytes(capacity_rows, binding.MOE_WINDOW_STATE) // 2 - state
        return window[start:start + state]

    def handshake(self) -> None:
        """Collective: exchanges the window handles and maps every other rank's window."""
        mine = binding.moe_window_export(self.window, self.generation, self.flags)
        handles = all_gather_bytes(mine, self.device, self.group)
        gens = [binding.MoeWindowHandle.from_buffer_copy(handles, r * binding.WINDOW_HANDLE_BYTES).generation
                for r in range(self.R)]
        self.comm.moe_peers_open(handles, self.rank, self.window, self.capacity)
        self.table_generations = np.asarray(gens, np.int32)
        self.handshakes += 1

    def install_addresses(self, window_bases, generations=None) -> None:
        """Addresses obtained elsewhere (one process holding every window; symmetric memory)."""
        gens = np.zeros(self.R, np.int32) if generations is None else np.asarray(generations, np.int32)
        self.comm.moe_peers_set(window_bases, gens, self.capacity, my_rank=self.rank, flags=self.flags)
        self.table_generations = gens

    def _ensure_addresses(self) -> None:
        # every rank holds the same table generations (handshakes are collective) and the same announcement,
        # so every rank takes the same branch
        if self.mode == "static":
            if self.table_generations is None:
                self.handshake()
        elif self.mode == "handshake" or addresses_stale(self.table_generations, self.announced):
            self.handshake()

    # -- the phases ------------------------------------------------------------------------------------
    def plan(self, schedule: int, topk_idx_local: torch.Tensor) -> torch.Tensor:
        if self.counts == "device":
            # Layout, then the row goes into every rank's mailbox and the offsets are built from this rank's own
            # mailbox once all rows are there: no collective, nothing read back on the host
            self._ensure_addresses()
            self.plan_epoch += 1
            self.comm.moe_layout_push(schedule, topk_idx_local, self.rank, self.plan_epoch)
            if self.host_fence:                  # ranks share a GPU: every push is sent before any notify is enqueued
                self._host_barrier()
            self.comm.moe_notify_peers(self.plan_epoch)
            self.announced = None
            return None
        self.comm.moe_layout(schedule, topk_idx_local, self.rank, self.counts_row)
        gathered = all_gather_rows(self.message, self.group)             # metadata only, no payload
        counts_all = gathered[:, :self.E].contiguous()
        # "static": nothing is read back, so nothing waits for the stream; the calls run without a validity test
        self.announced = None if self.mode == "static" else gathered[:, self.E].cpu().numpy().astype(np.int32)
        self.comm.moe_notify(counts_all)
        return counts_all

    def _host_barrier(self) -> None:
        torch.cuda.current_stream().synchronize()
        dist.barrier(self.group)

    def _signal_then_wait(self, slot: int) -> None:
        self.comm.moe_signal_peers(slot, self.epoch)
        if self.host_fence:                      # ranks share a GPU: every signal is sent before any wait is enqueued
            self._host_barrier()
        self.comm.moe_wait_peers(slot, self.epoch)

    def dispatch(self, x_local: torch.Tensor) -> None:
        """Rows into every rank's window; returns once the experts of this rank may be enqueued."""
        self._ensure_addresses()
        if self.sync == "device":
            self.epoch += 1
            if self.epoch > 1:                   # every rank has finished reading the windows of the step before
                self.comm.moe_wait_peers(self.SLOT_COMBINED, self.epoch - 1)
            self.comm.moe_dispatch_cached(x_local, self.announced)
            self._signal_then_wait(self.SLOT_DISPATCHED)
        else:
            self.comm.moe_dispatch_cached(x_local, self.announced)
            self._host_barrier()                 # every rank's rows have landed before any expert reads its window

    def combine(self, topk_w_local: torch.Tensor, y_local: torch.Tensor) -> None:
        """Call after this rank's experts have been enqueued: waits for every rank's experts, then combines."""
        if self.sync == "device":
            self._signal_then_wait(self.SLOT_EXPERTS_DONE)
            self.comm.moe_combine_cached(self.announced, topk_w_local, y_local)
            self.comm.moe_signal_peers(self.SLOT_COMBINED, self.epoch)
            if self.host_fence:
                self._host_barrier()
        else:
            self._host_barrier()                 # every expert has written its outputs
            self.comm.moe_combine_cached(self.announced, topk_w_local, y_local)

    def dispatch_quant(self, x_local: torch.Tensor) -> None:
        """Quantised dispatch: e4m3 codes into every rank's code window, fp32 scales (one per row, or one per 128
        elements if the windows were made with quant_group) into every rank's scale tensor -- the parts of the
        window allocations that MOE_WINDOW_QUANT / MOE_WINDOW_QUANT_GROUP reserve, reached through the same address
        table as the rows.  Returns once this rank's experts may read its codes."""
        self._ensure_addresses()
        if self.flags & binding.MOE_WINDOW_QUANT_GROUP:
            call = lambda: self.comm.moe_dispatch_quant_group_cached(x_local, self.announced)
        else:
            call = lambda: self.comm.moe_dispatch_quant_cached(x_local, self.announced)
        if self.sync == "device":
            self.epoch += 1
            if self.epoch > 1:
                self.comm.moe_wait_peers(self.SLOT_COMBINED, self.epoch - 1)
            call()
            self._signal_then_wait(self.SLOT_DISPATCHED)
        else:
            call()
            self._host_barrier()

    def status(self) -> int:
        return self.comm.moe_status()

    def close(self) -> None:
        torch.cuda.current_stream().synchronize()
        dist.barrier(self.group)                 # nobody unmaps a window another rank may still read
        self.comm.moe_peers_close()
        self.comm.close()
