"""Thin ctypes binding of libmoecomm (argument marshalling only).

Function names mirror the C ABI in ``include/moecomm.h``.  Tensors are torch
CUDA tensors used purely as device memory; every step of the path runs in the
library's CUDA kernels.  There is no CPU fallback: if ``libmoecomm.so`` has not
been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmoecomm.so")

MOE_OK, MOE_ERR_INVALID_ARG, MOE_ERR_BAD_INDEX, MOE_ERR_CAPACITY = 0, 1, 2, 3
MOE_ERR_NOT_PLANNED, MOE_ERR_TIMEOUT, MOE_ERR_CUDA, MOE_ERR_STALE_PEERS = 4, 5, 6, 7
MOE_SCHED_PREFILL, MOE_SCHED_DECODE = 0, 1

EXPORTS = [
    "moe_workspace_bytes", "moe_create", "moe_destroy", "moe_plan", "moe_plan_view", "moe_dispatch",
    "moe_combine", "moe_slots", "moe_forward_host", "moe_status", "moe_status_string", "moe_launch_count",
    "moe_slots_noalloc", "moe_set_option", "moe_dispatch_quant", "moe_expert_ranges",
    "moe_gate_topk", "moe_gate_plan", "moe_layout", "moe_notify", "moe_dispatch_peers", "moe_combine_peers",
    "moe_dispatch_range", "moe_combine_range", "moe_plan_dispatch", "moe_gate_plan_dispatch", "moe_plan_dispatch_quant", "moe_expert_tiles", "moe_dispatch_quant_peers",
    "moe_window_export", "moe_peers_open", "moe_peers_set", "moe_peers_check", "moe_peers_close",
    "moe_dispatch_cached", "moe_combine_cached", "moe_state_bytes", "moe_window_bytes", "moe_signal_peers",
    "moe_wait_peers", "moe_dispatch_quant_cached", "moe_dispatch_quant_group", "moe_plan_dispatch_quant_group",
    "moe_dispatch_quant_group_cached", "moe_push_counts", "moe_notify_peers", "moe_layout_push",
]
MOE_SYNC_SLOTS = 4
MOE_WINDOW_STATE, MOE_WINDOW_QUANT, MOE_WINDOW_QUANT_GROUP, MOE_WINDOW_COUNTS = 1, 2, 4, 8
MOE_OPT_DISPATCH_PATH, MOE_OPT_GRANULE, MOE_OPT_TEST_STARVE_WAIT_MS, MOE_OPT_OVERLAP = 0, 1, 2, 3
MOE_OPT_EXPERT_ALIGN, MOE_OPT_CLUSTER_PLAN, MOE_OPT_SLOT_REUSE = 4, 5, 6
MOE_DISPATCH_AUTO, MOE_DISPATCH_REGISTERS, MOE_DISPATCH_BULK = 0, 1, 2


class MoeShape(ctypes.Structure):
    _fields_ = [("T_max", ctypes.c_int32), ("H", ctypes.c_int32), ("E", ctypes.c_int32),
                ("R", ctypes.c_int32), ("K", ctypes.c_int32)]


class MoePlanView(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("counts", "c_rank", "small_off", "large_off", "n_exp", "n_recv",
                                               "rows")] + [("rows_capacity", ctypes.c_int64)]


class MoeWindowHandle(ctypes.Structure):
    """moe_window_handle_t: plain bytes describing one rank's window to the other ranks."""
    _fields_ = [("ipc", ctypes.c_ubyte * 64), ("offset", ctypes.c_int64), ("bytes", ctypes.c_int64),
                ("device", ctypes.c_int32), ("generation", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


WINDOW_HANDLE_BYTES = ctypes.sizeof(MoeWindowHandle)


class MoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def load() -> ctypes.CDLL:
    """Loads the built library; raises if it is missing (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is not built; run `python -m paper_2605_06055_b200.build` "
                           "(or __graft_entry__.build()). There is no CPU fallback.")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    L.moe_workspace_bytes.argtypes = [ctypes.POINTER(MoeShape)]
    L.moe_workspace_bytes.restype = ctypes.c_size_t
    L.moe_create.argtypes = [ctypes.POINTER(MoeShape), vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    L.moe_destroy.argtypes = [vp]
    L.moe_plan.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp]
    L.moe_plan_view.argtypes = [vp, ctypes.POINTER(MoePlanView)]
    L.moe_dispatch.argtypes = [vp, vp, vp, i64, vp]
    L.moe_combine.argtypes = [vp, vp, i64, vp, vp, vp]
    L.moe_dispatch_range.argtypes = [vp, vp, vp, i64, i32, i32, vp]
    L.moe_combine_range.argtypes = [vp, vp, i64, vp, vp, i32, i32, vp]
    L.moe_dispatch_range.restype = L.moe_combine_range.restype = ctypes.c_int
    L.moe_plan_dispatch.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp, vp, i64, vp]
    L.moe_plan_dispatch.restype = ctypes.c_int
    L.moe_gate_plan_dispatch.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp, vp, vp, vp, i64, vp]
    L.moe_gate_plan_dispatch.restype = ctypes.c_int
    L.moe_plan_dispatch_quant.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp, vp, vp, i64, vp]
    L.moe_plan_dispatch_quant.restype = ctypes.c_int
    L.moe_plan_dispatch_quant_group.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp, vp, vp, i64, i32, vp]
    L.moe_plan_dispatch_quant_group.restype = ctypes.c_int
    L.moe_dispatch_quant_group.argtypes = [vp, vp, vp, vp, i64, i32, vp]
    L.moe_dispatch_quant_group.restype = ctypes.c_int
    L.moe_layout.argtypes = [vp, ctypes.c_int, vp, i32, i32, vp, vp]
    L.moe_notify.argtypes = [vp, vp, vp]
    L.moe_dispatch_peers.argtypes = [vp, vp, vp, i64, vp]
    L.moe_combine_peers.argtypes = [vp, vp, i64, vp, vp, vp]
    for _n in ("moe_layout", "moe_notify", "moe_dispatch_peers", "moe_combine_peers"):
        getattr(L, _n).restype = ctypes.c_int
    L.moe_gate_topk.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    L.moe_gate_topk.restype = ctypes.c_int
    L.moe_gate_plan.argtypes = [vp, ctypes.c_int, vp, i32, vp, vp, vp, vp]
    L.moe_gate_plan.restype = ctypes.c_int
    L.moe_expert_ranges.argtypes = [vp, i64, vp, vp, vp]
    L.moe_expert_ranges.restype = ctypes.c_int
    L.moe_expert_tiles.argtypes = [vp, i64, i32, i64, vp, vp, vp, vp, vp]
    L.moe_expert_tiles.restype = ctypes.c_int
    L.moe_dispatch_quant_peers.argtypes = [vp, vp, vp, vp, i64, vp]
    L.moe_dispatch_quant_peers.restype = ctypes.c_int
    L.moe_dispatch_quant.argtypes = [vp, vp, vp, vp, i64, vp]
    L.moe_dispatch_quant.restype = ctypes.c_int
    L.moe_window_export.argtypes = [vp, i64, i32, i32, ctypes.POINTER(MoeWindowHandle)]
    L.moe_dispatch_quant_cached.argtypes = [vp, vp, vp, vp]
    L.moe_dispatch_quant_cached.restype = ctypes.c_int
    L.moe_dispatch_quant_group_cached.argtypes = [vp, vp, vp, i32, vp]
    L.moe_dispatch_quant_group_cached.restype = ctypes.c_int
    L.moe_peers_open.argtypes = [vp, vp, i32, vp, i64, vp]
    L.moe_peers_set.argtypes = [vp, vp, vp, i32, i64, i32, vp]
    L.moe_state_bytes.argtypes = [i32]
    L.moe_state_bytes.restype = ctypes.c_size_t
    L.moe_window_bytes.argtypes = [ctypes.POINTER(MoeShape), i64, i32]
    L.moe_window_bytes.restype = ctypes.c_size_t
    L.moe_signal_peers.argtypes = [vp, i32, ctypes.c_uint32, vp]
    L.moe_wait_peers.argtypes = [vp, i32, ctypes.c_uint32, vp]
    L.moe_signal_peers.restype = L.moe_wait_peers.restype = ctypes.c_int
    L.moe_push_counts.argtypes = L.moe_notify_peers.argtypes = [vp, ctypes.c_uint32, vp]
    L.moe_push_counts.restype = L.moe_notify_peers.restype = ctypes.c_int
    L.moe_layout_push.argtypes = [vp, i32, vp, i32, i32, ctypes.c_uint32, vp]
    L.moe_layout_push.restype = ctypes.c_int
    L.moe_peers_check.argtypes = [vp, vp]
    L.moe_peers_close.argtypes = [vp, vp]
    L.moe_dispatch_cached.argtypes = [vp, vp, vp, vp]
    L.moe_combine_cached.argtypes = [vp, vp, vp, vp, vp]
    for _n in ("moe_window_export", "moe_peers_open", "moe_peers_set", "moe_peers_check", "moe_peers_close",
               "moe_dispatch_cached", "moe_combine_cached"):
        getattr(L, _n).restype = ctypes.c_int
    L.moe_slots.argtypes = [vp, i64, vp, vp]
    L.moe_forward_host.argtypes = [vp, ctypes.c_int, i32, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
    L.moe_status.argtypes = [vp, vp]
    L.moe_slots_noalloc.argtypes = [vp, i32, i32, i32, i32, vp, i64, vp, vp, vp, vp]
    L.moe_slots_noalloc.restype = ctypes.c_int
    L.moe_set_option.argtypes = [vp, ctypes.c_int, i64]
    L.moe_set_option.restype = ctypes.c_int
    L.moe_status_string.argtypes = [ctypes.c_int]
    L.moe_status_string.restype = ctypes.c_char_p
    L.moe_launch_count.argtypes = [vp]
    L.moe_launch_count.restype = i64
    for name in ("moe_create", "moe_destroy", "moe_plan", "moe_plan_view", "moe_dispatch", "moe_combine",
                 "moe_slots", "moe_forward_host", "moe_status"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def status_string(code: int) -> str:
    return load().moe_status_string(int(code)).decode()


def moe_workspace_bytes(T_max: int, H: int, E: int, R: int, K: int) -> int:
    return int(load().moe_workspace_bytes(ctypes.byref(MoeShape(T_max, H, E, R, K))))


def _dev_ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _host_ptr(t, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert not t.is_cuda and t.is_contiguous()
    if dtype is not None:
        assert t.dtype == dtype
    return t.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class _NoSwitch:
    """Stands in for torch.cuda.device(...) when the context's device is already current
    (entering the real guard costs several microseconds per call)."""

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


_NO_SWITCH = _NoSwitch()


class MoeComm:
    """One libmoecomm context (opaque handle + its torch-allocated workspace)."""

    def __init__(self, T_max: int, H: int, E: int, R: int, K: int, device="cuda:0"):
        self.lib = load()
        self.device = torch.device(device)
        self.T_max, self.H, self.E, self.R, self.K = T_max, H, E, R, K
        self._shape = MoeShape(T_max, H, E, R, K)
        nbytes = int(self.lib.moe_workspace_bytes(ctypes.byref(self._shape)))
        if nbytes == 0:
            raise MoeError(MOE_ERR_INVALID_ARG, "moe_workspace_bytes")
        self._dev_index = self.device.index if self.device.index is not None else torch.cuda.current_device()
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            h = ctypes.c_void_p()
            rc = self.lib.moe_create(ctypes.byref(self._shape), self.workspace.data_ptr(), nbytes, ctypes.byref(h))
        if rc != MOE_OK:
            raise MoeError(rc, "moe_create")
        self._h = h
        self.T = 0
        self.schedule = None
        self._keep = None  # routing tensor of the live plan (the library re-reads it)

    def _on_device(self):
        """Context manager that makes this context's device current (free when it already is)."""
        return _NO_SWITCH if torch.cuda.current_device() == self._dev_index else torch.cuda.device(self.device)

    def close(self):
        if getattr(self, "_h", None):
            self.lib.moe_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI calls, same names -------------------------------------------------
    def moe_plan(self, schedule: int, topk_idx: torch.Tensor, T: Optional[int] = None, rank_tok_start=None,
                 stream=None, check: bool = True) -> int:
        T = topk_idx.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_plan(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T, _host_ptr(rts),
                                   _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_plan")
        return rc

    def moe_plan_dispatch(self, schedule: int, topk_idx: torch.Tensor, x: torch.Tensor, windows: torch.Tensor,
                          capacity_rows: int, T: Optional[int] = None, rank_tok_start=None, stream=None,
                          check: bool = True) -> int:
        T = topk_idx.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_plan_dispatch(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T, _host_ptr(rts),
                                            _dev_ptr(x, torch.bfloat16), _dev_ptr(windows, torch.bfloat16),
                                            int(capacity_rows), _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_plan_dispatch")
        return rc

    def moe_plan_dispatch_quant(self, schedule: int, topk_idx: torch.Tensor, x: torch.Tensor, windows_q: torch.Tensor,
                                scales: torch.Tensor, capacity_rows: int, T: Optional[int] = None, rank_tok_start=None,
                                stream=None, check: bool = True) -> int:
        T = topk_idx.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_plan_dispatch_quant(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T, _host_ptr(rts),
                                                  _dev_ptr(x, torch.bfloat16), _dev_ptr(windows_q, torch.uint8),
                                                  _dev_ptr(scales, torch.float32), int(capacity_rows),
                                                  _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_plan_dispatch_quant")
        return rc

    def moe_plan_dispatch_quant_group(self, schedule: int, topk_idx: torch.Tensor, x: torch.Tensor,
                                      windows_q: torch.Tensor, scales: torch.Tensor, capacity_rows: int,
                                      group_size: int = 128, T: Optional[int] = None, rank_tok_start=None,
                                      stream=None, check: bool = True) -> int:
        T = topk_idx.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_plan_dispatch_quant_group(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T,
                                                        _host_ptr(rts), _dev_ptr(x, torch.bfloat16),
                                                        _dev_ptr(windows_q, torch.uint8),
                                                        _dev_ptr(scales, torch.float32), int(capacity_rows),
                                                        int(group_size), _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_plan_dispatch_quant_group")
        return rc

    def moe_gate_plan_dispatch(self, schedule: int, logits: torch.Tensor, topk_idx: torch.Tensor, topk_w: torch.Tensor,
                               x: torch.Tensor, windows: torch.Tensor, capacity_rows: int, T: Optional[int] = None,
                               rank_tok_start=None, stream=None, check: bool = True) -> int:
        T = logits.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_gate_plan_dispatch(self._h, schedule, _dev_ptr(logits, torch.float32), T, _host_ptr(rts),
                                                 _dev_ptr(topk_idx, torch.int32), _dev_ptr(topk_w, torch.float32),
                                                 _dev_ptr(x, torch.bfloat16), _dev_ptr(windows, torch.bfloat16),
                                                 int(capacity_rows), _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_gate_plan_dispatch")
        return rc

    def moe_gate_plan(self, schedule: int, logits: torch.Tensor, topk_idx: torch.Tensor, topk_w: torch.Tensor,
                      T: Optional[int] = None, rank_tok_start=None, stream=None, check: bool = True) -> int:
        T = logits.shape[0] if T is None else T
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_gate_plan(self._h, schedule, _dev_ptr(logits, torch.float32), T, _host_ptr(rts),
                                        _dev_ptr(topk_idx, torch.int32), _dev_ptr(topk_w, torch.float32),
                                        _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_gate_plan")
        return rc

    def moe_dispatch_range(self, x, windows, capacity_rows: int, t_begin: int, t_end: int, stream=None,
                           check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_dispatch_range(self._h, _dev_ptr(x, torch.bfloat16), _dev_ptr(windows, torch.bfloat16),
                                             int(capacity_rows), t_begin, t_end, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_range")
        return rc

    def moe_combine_range(self, windows, capacity_rows: int, topk_w, y, t_begin: int, t_end: int, stream=None,
                          check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_combine_range(self._h, _dev_ptr(windows, torch.bfloat16), int(capacity_rows),
                                            _dev_ptr(topk_w, torch.float32), _dev_ptr(y, torch.bfloat16),
                                            t_begin, t_end, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_combine_range")
        return rc

    # -- multi-rank decomposition ---------------------------------------------------
    def moe_layout(self, schedule: int, topk_idx: torch.Tensor, my_rank: int, counts_row: torch.Tensor,
                   stream=None, check: bool = True) -> int:
        T = topk_idx.shape[0]
        with self._on_device():
            rc = self.lib.moe_layout(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T, my_rank,
                                     _dev_ptr(counts_row, torch.int32), _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_layout")
        return rc

    def moe_notify(self, counts_all: torch.Tensor, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_notify(self._h, _dev_ptr(counts_all, torch.int32), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_notify")
        return rc

    def moe_dispatch_peers(self, x: torch.Tensor, window_bases: torch.Tensor, capacity_rows: int, stream=None,
                           check: bool = True) -> int:
        """window_bases: int64 CUDA tensor [R] holding the device address of every rank's window."""
        with self._on_device():
            rc = self.lib.moe_dispatch_peers(self._h, _dev_ptr(x, torch.bfloat16), _dev_ptr(window_bases, torch.int64),
                                             int(capacity_rows), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_peers")
        return rc

    def moe_combine_peers(self, window_bases: torch.Tensor, capacity_rows: int, topk_w: torch.Tensor, y: torch.Tensor,
                          stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_combine_peers(self._h, _dev_ptr(window_bases, torch.int64), int(capacity_rows),
                                            _dev_ptr(topk_w, torch.float32), _dev_ptr(y, torch.bfloat16),
                                            _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_combine_peers")
        return rc

    # -- window addresses of the group: handshake and cached table ------------------------
    def moe_peers_open(self, handles: bytes, my_rank: int, my_window: torch.Tensor, capacity_rows: int, stream=None,
                       check: bool = True) -> int:
        """handles: R exported handles back to back (R * WINDOW_HANDLE_BYTES bytes), entry r from rank r."""
        assert len(handles) == self.R * WINDOW_HANDLE_BYTES
        buf = ctypes.create_string_buffer(handles, len(handles))
        with self._on_device():
            rc = self.lib.moe_peers_open(self._h, ctypes.cast(buf, ctypes.c_void_p), my_rank,
                                         _dev_ptr(my_window, torch.bfloat16), int(capacity_rows),
                                         _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_peers_open")
        return rc

    def moe_peers_set(self, window_bases, generations, capacity_rows: int, my_rank: int = 0, flags: int = 0,
                      stream=None, check: bool = True) -> int:
        """window_bases: R device addresses (ints); generations: R ints or None; flags: MOE_WINDOW_* bits saying
        what follows the rows of every window (moe_window_bytes(capacity_rows, flags) bytes were allocated)."""
        bases = np.ascontiguousarray(window_bases, dtype=np.uint64)
        gens = None if generations is None else np.ascontiguousarray(generations, dtype=np.int32)
        assert bases.shape == (self.R,) and (gens is None or gens.shape == (self.R,))
        with self._on_device():
            rc = self.lib.moe_peers_set(self._h, _host_ptr(bases), _host_ptr(gens), int(my_rank), int(capacity_rows),
                                        int(flags), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_peers_set")
        return rc

    def moe_peers_check(self, generations) -> int:
        gens = np.ascontiguousarray(generations, dtype=np.int32)
        assert gens.shape == (self.R,)
        return int(self.lib.moe_peers_check(self._h, _host_ptr(gens)))

    def moe_peers_close(self, stream=None) -> int:
        with self._on_device():
            return int(self.lib.moe_peers_close(self._h, _stream_handle(stream)))

    def moe_dispatch_cached(self, x: torch.Tensor, generations=None, stream=None, check: bool = True) -> int:
        gens = None if generations is None else np.ascontiguousarray(generations, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_dispatch_cached(self._h, _dev_ptr(x, torch.bfloat16), _host_ptr(gens),
                                              _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_cached")
        return rc

    def moe_combine_cached(self, generations, topk_w: torch.Tensor, y: torch.Tensor, stream=None,
                           check: bool = True) -> int:
        gens = None if generations is None else np.ascontiguousarray(generations, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_combine_cached(self._h, _host_ptr(gens), _dev_ptr(topk_w, torch.float32),
                                             _dev_ptr(y, torch.bfloat16), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_combine_cached")
        return rc

    def moe_window_bytes(self, capacity_rows: int, flags: int = MOE_WINDOW_STATE) -> int:
        return int(self.lib.moe_window_bytes(ctypes.byref(self._shape), int(capacity_rows), int(flags)))

    def moe_dispatch_quant_cached(self, x: torch.Tensor, generations=None, stream=None, check: bool = True) -> int:
        gens = None if generations is None else np.ascontiguousarray(generations, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_dispatch_quant_cached(self._h, _dev_ptr(x, torch.bfloat16), _host_ptr(gens),
                                                    _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_quant_cached")
        return rc

    def moe_dispatch_quant_group_cached(self, x: torch.Tensor, generations=None, group_size: int = 128, stream=None,
                                        check: bool = True) -> int:
        gens = None if generations is None else np.ascontiguousarray(generations, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_dispatch_quant_group_cached(self._h, _dev_ptr(x, torch.bfloat16), _host_ptr(gens),
                                                          int(group_size), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_quant_group_cached")
        return rc

    def moe_signal_peers(self, slot: int, epoch: int, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_signal_peers(self._h, int(slot), int(epoch) & 0xFFFFFFFF, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_signal_peers")
        return rc

    def moe_wait_peers(self, slot: int, epoch: int, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_wait_peers(self._h, int(slot), int(epoch) & 0xFFFFFFFF, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_wait_peers")
        return rc

    def moe_layout_push(self, schedule: int, topk_idx: torch.Tensor, my_rank: int, epoch: int, stream=None,
                        check: bool = True) -> int:
        T = topk_idx.shape[0]
        with self._on_device():
            rc = self.lib.moe_layout_push(self._h, schedule, _dev_ptr(topk_idx, torch.int32), T, my_rank,
                                          int(epoch) & 0xFFFFFFFF, _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx
        elif check:
            raise MoeError(rc, "moe_layout_push")
        return rc

    def moe_push_counts(self, epoch: int, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_push_counts(self._h, int(epoch) & 0xFFFFFFFF, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_push_counts")
        return rc

    def moe_notify_peers(self, epoch: int, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_notify_peers(self._h, int(epoch) & 0xFFFFFFFF, _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_notify_peers")
        return rc

    def moe_plan_view(self) -> dict:
        """Zero-copy int32 tensors over the planning state in the workspace."""
        v = MoePlanView()
        rc = self.lib.moe_plan_view(self._h, ctypes.byref(v))
        if rc != MOE_OK:
            raise MoeError(rc, "moe_plan_view")
        base = self.workspace.data_ptr()
        shapes = {"counts": (self.R, self.E), "c_rank": (self.R, self.R), "small_off": (self.T, self.K),
                  "large_off": (self.E, self.R), "n_exp": (self.E,), "n_recv": (self.R,), "rows": (self.T, self.K)}
        out = {}
        for name, shp in shapes.items():
            p = getattr(v, name)
            if p is None:
                out[name] = None
                continue
            n = int(np.prod(shp))
            off = p - base
            out[name] = self.workspace[off:off + 4 * n].view(torch.int32).view(*shp)
        out["rows_capacity"] = int(v.rows_capacity)
        return out

    def moe_dispatch(self, x: torch.Tensor, windows: torch.Tensor, capacity_rows: int, stream=None,
                     check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_dispatch(self._h, _dev_ptr(x, torch.bfloat16), _dev_ptr(windows, torch.bfloat16),
                                       int(capacity_rows), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch")
        return rc

    def moe_dispatch_quant(self, x: torch.Tensor, windows_q: torch.Tensor, scales: torch.Tensor, capacity_rows: int,
                           stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_dispatch_quant(self._h, _dev_ptr(x, torch.bfloat16), _dev_ptr(windows_q, torch.uint8),
                                             _dev_ptr(scales, torch.float32), int(capacity_rows),
                                             _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_quant")
        return rc

    def moe_dispatch_quant_group(self, x: torch.Tensor, windows_q: torch.Tensor, scales: torch.Tensor,
                                 capacity_rows: int, group_size: int = 128, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_dispatch_quant_group(self._h, _dev_ptr(x, torch.bfloat16),
                                                   _dev_ptr(windows_q, torch.uint8), _dev_ptr(scales, torch.float32),
                                                   int(capacity_rows), int(group_size), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_quant_group")
        return rc

    def moe_dispatch_quant_peers(self, x: torch.Tensor, window_q_bases: torch.Tensor, scale_bases: torch.Tensor,
                                 capacity_rows: int, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_dispatch_quant_peers(self._h, _dev_ptr(x, torch.bfloat16),
                                                   _dev_ptr(window_q_bases, torch.int64),
                                                   _dev_ptr(scale_bases, torch.int64), int(capacity_rows),
                                                   _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_dispatch_quant_peers")
        return rc

    def moe_expert_tiles(self, capacity_rows: int, tile_rows: int, tile_expert: torch.Tensor, tile_row: torch.Tensor,
                         tile_valid: torch.Tensor, n_tiles: torch.Tensor, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_expert_tiles(self._h, int(capacity_rows), int(tile_rows), int(tile_expert.numel()),
                                           _dev_ptr(tile_expert, torch.int32), _dev_ptr(tile_row, torch.int64),
                                           _dev_ptr(tile_valid, torch.int32), _dev_ptr(n_tiles, torch.int32),
                                           _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_expert_tiles")
        return rc

    def moe_expert_ranges(self, capacity_rows: int, row_start: torch.Tensor, row_count: torch.Tensor, stream=None,
                          check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_expert_ranges(self._h, int(capacity_rows), _dev_ptr(row_start, torch.int64),
                                            _dev_ptr(row_count, torch.int32), _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_expert_ranges")
        return rc

    def moe_combine(self, windows: torch.Tensor, capacity_rows: int, topk_w: torch.Tensor, y: torch.Tensor,
                    stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_combine(self._h, _dev_ptr(windows, torch.bfloat16), int(capacity_rows),
                                      _dev_ptr(topk_w, torch.float32), _dev_ptr(y, torch.bfloat16),
                                      _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_combine")
        return rc

    def moe_slots(self, capacity_rows: int, slots: torch.Tensor, stream=None, check: bool = True) -> int:
        with self._on_device():
            rc = self.lib.moe_slots(self._h, int(capacity_rows), _dev_ptr(slots, torch.int32),
                                    _stream_handle(stream))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_slots")
        return rc

    def moe_forward_host(self, schedule: int, T: int, rank_tok_start, x_host, topk_idx_host, topk_w_host,
                         x_dev, topk_idx_dev, topk_w_dev, windows_dev, capacity_rows: int, y_dev, y_host,
                         stream=None, check: bool = True) -> int:
        rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
        with self._on_device():
            rc = self.lib.moe_forward_host(
                self._h, schedule, T, _host_ptr(rts), _host_ptr(x_host), _host_ptr(topk_idx_host),
                _host_ptr(topk_w_host), _dev_ptr(x_dev), _dev_ptr(topk_idx_dev), _dev_ptr(topk_w_dev),
                _dev_ptr(windows_dev), int(capacity_rows), _dev_ptr(y_dev), _host_ptr(y_host),
                _stream_handle(stream))
        if rc == MOE_OK:
            self.T, self.schedule, self._keep = T, schedule, topk_idx_dev
        elif check:
            raise MoeError(rc, "moe_forward_host")
        return rc

    def moe_set_option(self, option: int, value: int, check: bool = True) -> int:
        rc = int(self.lib.moe_set_option(self._h, option, int(value)))
        if rc != MOE_OK and check:
            raise MoeError(rc, "moe_set_option")
        return rc

    def moe_status(self, stream=None) -> int:
        with self._on_device():
            return int(self.lib.moe_status(self._h, _stream_handle(stream)))

    def moe_launch_count(self) -> int:
        return int(self.lib.moe_launch_count(self._h))


def moe_slots_noalloc(topk_idx: torch.Tensor, E: int, R: int, capacity_rows: int, slots: torch.Tensor,
                      n_recv: torch.Tensor, status: torch.Tensor, rank_tok_start=None, stream=None) -> int:
    """Slots from routing indexes using the library's built-in scratch (see include/moecomm.h).

    For callers that cannot hand the library a workspace.  Every tensor here is the caller's; this
    wrapper allocates nothing and neither does the call.  Returns the host-side status code.
    """
    T, K = topk_idx.shape
    rts = None if rank_tok_start is None else np.ascontiguousarray(rank_tok_start, dtype=np.int32)
    with torch.cuda.device(topk_idx.device):
        return int(load().moe_slots_noalloc(_dev_ptr(topk_idx, torch.int32), T, K, E, R, _host_ptr(rts),
                                            int(capacity_rows), _dev_ptr(slots, torch.int32),
                                            _dev_ptr(n_recv, torch.int32), _dev_ptr(status, torch.int32),
                                            _stream_handle(stream)))


def moe_state_bytes(R: int) -> int:
    return int(load().moe_state_bytes(int(R)))


def moe_window_export(window: torch.Tensor, generation: int, flags: int = 0) -> bytes:
    """Handle of one rank's window allocation for the other ranks (see include/moecomm.h): WINDOW_HANDLE_BYTES plain
    bytes.  flags: MOE_WINDOW_* bits saying what the allocation holds behind its rows."""
    h = MoeWindowHandle()
    with torch.cuda.device(window.device):
        rc = int(load().moe_window_export(_dev_ptr(window), window.numel() * window.element_size(), int(generation),
                                          int(flags), ctypes.byref(h)))
    if rc != MOE_OK:
        raise MoeError(rc, "moe_window_export")
    return bytes(h)


def moe_gate_topk(logits: torch.Tensor, K: int, topk_idx: torch.Tensor, topk_w: torch.Tensor, stream=None) -> int:
    """Stand-alone top-k gate (see include/moecomm.h): K largest logits + fp32 softmax over them."""
    T, E = logits.shape
    with torch.cuda.device(logits.device):
        return int(load().moe_gate_topk(_dev_ptr(logits, torch.float32), T, E, K, _dev_ptr(topk_idx, torch.int32),
                                        _dev_ptr(topk_w, torch.float32), _stream_handle(stream)))
