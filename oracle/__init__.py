"""ctypes loader for the CPU oracle (TEST INFRASTRUCTURE ONLY).

The oracle is the plain C++ definition of plan / dispatch / combine in
``moe_oracle.cpp``.  Nothing in the product package imports this module; it is
used by the tests, the smoke check and the benchmark's cpu-baseline leg.

All arrays are numpy arrays on the host.  bf16 tensors are carried as uint16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

OK, ERR_INVALID_ARG, ERR_BAD_INDEX, ERR_CAPACITY = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
             or os.path.getmtime(_LIB) < os.path.getmtime(os.path.join(_HERE, "moe_oracle.h")))
    if force or stale:
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
                               "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32, i64, p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        L.oracle_plan.argtypes = [p, i32, i32, i32, i32, p, i32, p, p, p, p, p, p]
        L.oracle_slots.argtypes = [p, i32, i32, i32, i32, p, p, p, p, i64, p]
        L.oracle_dispatch.argtypes = [p, i32, i32, i32, p, p, i32]
        L.oracle_expert_scale.argtypes = [p, i32, i32, i32, i64, i32, p, p]
        L.oracle_combine.argtypes = [p, i32, i32, i32, p, p, p, i32]
        L.oracle_notify.argtypes = [p, i32, i32, i32, p, p, p, p]
        L.oracle_notify.restype = ctypes.c_int
        L.oracle_gate_topk.argtypes = [p, i32, i32, i32, p, p]
        L.oracle_gate_topk.restype = ctypes.c_int
        L.oracle_expert_ranges.argtypes = [i32, i32, i64, i32, p, p, p]
        L.oracle_expert_ranges.restype = ctypes.c_int
        L.oracle_expert_tiles.argtypes = [i32, i32, i64, i32, i32, p, i64, p, p, p, p]
        L.oracle_expert_tiles.restype = ctypes.c_int
        L.oracle_dispatch_quant.argtypes = [p, i32, i32, i32, p, p, p, i32]
        L.oracle_dispatch_quant.restype = ctypes.c_int
        L.oracle_dispatch_quant_group.argtypes = [p, i32, i32, i32, p, p, p, i32, i32]
        L.oracle_dispatch_quant_group.restype = ctypes.c_int
        L.oracle_float_to_e4m3.argtypes = [ctypes.c_float]
        L.oracle_float_to_e4m3.restype = ctypes.c_uint8
        L.oracle_e4m3_to_float.argtypes = [ctypes.c_uint8]
        L.oracle_e4m3_to_float.restype = ctypes.c_float
        L.oracle_float_to_bf16.argtypes = [ctypes.c_float]
        L.oracle_float_to_bf16.restype = ctypes.c_uint16
        L.oracle_bf16_to_float.argtypes = [ctypes.c_uint16]
        L.oracle_bf16_to_float.restype = ctypes.c_float
        for f in (L.oracle_plan, L.oracle_slots, L.oracle_dispatch, L.oracle_expert_scale, L.oracle_combine):
            f.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def uniform_rank_tok_start(T: int, R: int) -> np.ndarray:
    assert T % R == 0
    return (np.arange(R + 1, dtype=np.int64) * (T // R)).astype(np.int32)


@dataclass
class Plan:
    status: int
    M: np.ndarray        # [R,E]
    c_rank: np.ndarray   # [R,R]
    s: np.ndarray        # [T,K]
    o: np.ndarray        # [E,R]
    n_exp: np.ndarray    # [E]
    n_recv: np.ndarray   # [R]


def plan(topk_idx, E: int, R: int, rank_tok_start=None, align: int = 1) -> Plan:
    topk_idx = _c(topk_idx, np.int32)
    T, K = topk_idx.shape
    rts = uniform_rank_tok_start(T, R) if rank_tok_start is None else _c(rank_tok_start, np.int32)
    sentinel = -7
    M = np.full((R, E), sentinel, np.int32)
    c_rank = np.full((R, R), sentinel, np.int32)
    s = np.full((T, K), sentinel, np.int32)
    o = np.full((E, R), sentinel, np.int32)
    n_exp = np.full((E,), sentinel, np.int32)
    n_recv = np.full((R,), sentinel, np.int32)
    st = lib().oracle_plan(_ptr(topk_idx), T, K, E, R, _ptr(rts), int(align), _ptr(M), _ptr(c_rank), _ptr(s),
                           _ptr(o), _ptr(n_exp), _ptr(n_recv))
    return Plan(st, M, c_rank, s, o, n_exp, n_recv)


def slots(topk_idx, E: int, R: int, pl: Plan, C: int, rank_tok_start=None):
    topk_idx = _c(topk_idx, np.int32)
    T, K = topk_idx.shape
    rts = uniform_rank_tok_start(T, R) if rank_tok_start is None else _c(rank_tok_start, np.int32)
    out = np.full((T, K), -1, np.int64)
    st = lib().oracle_slots(_ptr(topk_idx), T, K, E, R, _ptr(rts), _ptr(pl.s), _ptr(pl.o), _ptr(pl.n_recv),
                            int(C), _ptr(out))
    return st, out


def notify(M, align: int = 1):
    """Large offsets and receive counts from a gathered count matrix M [R,E]."""
    M = _c(M, np.int32)
    R, E = M.shape
    c_rank = np.full((R, R), -7, np.int32)
    o = np.full((E, R), -7, np.int32)
    n_exp = np.full((E,), -7, np.int32)
    n_recv = np.full((R,), -7, np.int32)
    st = lib().oracle_notify(_ptr(M), E, R, int(align), _ptr(c_rank), _ptr(o), _ptr(n_exp), _ptr(n_recv))
    return st, c_rank, o, n_exp, n_recv


def gate_topk(logits, K: int):
    logits = _c(logits, np.float32)
    T, E = logits.shape
    idx = np.full((T, K), -1, np.int32)
    w = np.full((T, K), -1.0, np.float32)
    st = lib().oracle_gate_topk(_ptr(logits), T, E, K, _ptr(idx), _ptr(w))
    return st, idx, w


def expert_ranges(E: int, R: int, C: int, n_exp, align: int = 1):
    n_exp = _c(n_exp, np.int32)
    start = np.full((E,), -1, np.int64)
    count = np.full((E,), -1, np.int32)
    st = lib().oracle_expert_ranges(E, R, int(C), int(align), _ptr(n_exp), _ptr(start), _ptr(count))
    return st, start, count


def expert_tiles(E: int, R: int, C: int, n_exp, tile_rows: int, max_tiles: int, align: int = 1):
    """Tiles of at most tile_rows rows over every expert's run, in window order."""
    n_exp = _c(n_exp, np.int32)
    tile_expert = np.full((max_tiles,), -1, np.int32)
    tile_row = np.full((max_tiles,), -1, np.int64)
    tile_valid = np.full((max_tiles,), -1, np.int32)
    n_tiles = np.zeros((1,), np.int64)
    st = lib().oracle_expert_tiles(E, R, int(C), int(align), int(tile_rows), _ptr(n_exp), int(max_tiles),
                                   _ptr(tile_expert), _ptr(tile_row), _ptr(tile_valid), _ptr(n_tiles))
    return st, tile_expert, tile_row, tile_valid, int(n_tiles[0])


def dispatch(X_u16, slots_, windows_u16, n_threads: int = 1) -> int:
    """Scatter rows of X [T,H] into windows [R*C,H] (modified in place)."""
    X_u16 = _c(X_u16, np.uint16)
    slots_ = _c(slots_, np.int64)
    T, H = X_u16.shape
    K = slots_.shape[1] if slots_.ndim == 2 else 1
    assert windows_u16.dtype == np.uint16 and windows_u16.flags["C_CONTIGUOUS"]
    return lib().oracle_dispatch(_ptr(X_u16), T, H, K, _ptr(slots_), _ptr(windows_u16), n_threads)


def dispatch_quant(X_u16, slots_, windows_q, scales, n_threads: int = 1) -> int:
    """Quantise rows of X [T,H] to e4m3 with one fp32 scale per row and scatter codes + scales."""
    X_u16 = _c(X_u16, np.uint16)
    slots_ = _c(slots_, np.int64)
    T, H = X_u16.shape
    K = slots_.shape[1]
    assert windows_q.dtype == np.uint8 and windows_q.flags["C_CONTIGUOUS"]
    assert scales.dtype == np.float32 and scales.flags["C_CONTIGUOUS"]
    return lib().oracle_dispatch_quant(_ptr(X_u16), T, H, K, _ptr(slots_), _ptr(windows_q), _ptr(scales), n_threads)


def dispatch_quant_group(X_u16, slots_, windows_q, scales, group: int, n_threads: int = 1) -> int:
    """As dispatch_quant with one fp32 scale per `group` consecutive elements: scales is [rows, H // group]."""
    X_u16 = _c(X_u16, np.uint16)
    slots_ = _c(slots_, np.int64)
    T, H = X_u16.shape
    K = slots_.shape[1]
    assert windows_q.dtype == np.uint8 and windows_q.flags["C_CONTIGUOUS"]
    assert scales.dtype == np.float32 and scales.flags["C_CONTIGUOUS"]
    return lib().oracle_dispatch_quant_group(_ptr(X_u16), T, H, K, _ptr(slots_), _ptr(windows_q), _ptr(scales),
                                             int(group), n_threads)


def float_to_e4m3(x: float) -> int:
    return int(lib().oracle_float_to_e4m3(float(np.float32(x))))


def e4m3_to_float(c: int) -> float:
    return float(lib().oracle_e4m3_to_float(int(c)))


def expert_scale(windows_u16, H: int, E: int, R: int, C: int, n_exp, scale_u16, align: int = 1) -> int:
    n_exp = _c(n_exp, np.int32)
    scale_u16 = _c(scale_u16, np.uint16)
    assert windows_u16.dtype == np.uint16 and windows_u16.flags["C_CONTIGUOUS"]
    return lib().oracle_expert_scale(_ptr(windows_u16), H, E, R, int(C), int(align), _ptr(n_exp), _ptr(scale_u16))


def combine(windows_u16, slots_, W, H: int, n_threads: int = 1):
    slots_ = _c(slots_, np.int64)
    W = _c(W, np.float32)
    T, K = slots_.shape
    assert windows_u16.dtype == np.uint16 and windows_u16.flags["C_CONTIGUOUS"]
    Y = np.zeros((T, H), np.uint16)
    st = lib().oracle_combine(_ptr(windows_u16), T, H, K, _ptr(slots_), _ptr(W), _ptr(Y), n_threads)
    return st, Y


def float_to_bf16(x: float) -> int:
    return int(lib().oracle_float_to_bf16(float(np.float32(x))))


def bf16_to_float(b: int) -> float:
    return float(lib().oracle_bf16_to_float(int(b)))
