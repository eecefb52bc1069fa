"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function the header declares, and its pure host logic behaves."""
import ctypes
import os
import re

import pytest

from paper_2605_06055_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert names >= set(binding.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == names


def test_workspace_bytes_host_logic(lib):
    assert binding.moe_workspace_bytes(2048, 7168, 256, 16, 8) > 0
    small = binding.moe_workspace_bytes(256, 1024, 16, 4, 2)
    big = binding.moe_workspace_bytes(32768, 7168, 256, 8, 8)
    assert 0 < small < big < 64 << 20          # control state only: far below one window buffer
    assert binding.moe_workspace_bytes(256, 1020, 16, 4, 2) == 0    # H % 8
    assert binding.moe_workspace_bytes(256, 1024, 16, 3, 2) == 0    # E % R
    assert binding.moe_workspace_bytes(256, 1024, 16, 4, 0) == 0    # K >= 1
    assert binding.moe_workspace_bytes(256, 1024, 16, 4, 33) == 0   # K <= MOE_MAX_K
    assert binding.moe_workspace_bytes(1 << 30, 1024, 16, 4, 8) == 0  # T_max*K < 2^31
    assert lib.moe_workspace_bytes(None) == 0


def test_null_handles_and_strings(lib):
    assert lib.moe_destroy(None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_plan(None, 0, None, 0, None, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_dispatch(None, None, None, 0, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_combine(None, None, 0, None, None, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_create(None, None, 0, None) == binding.MOE_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    shape = binding.MoeShape(16, 64, 4, 2, 2)
    assert lib.moe_create(ctypes.byref(shape), None, 0, ctypes.byref(h)) == binding.MOE_ERR_INVALID_ARG
    for code in range(7):
        assert binding.status_string(code)
    assert binding.status_string(binding.MOE_ERR_CAPACITY) != binding.status_string(binding.MOE_OK)


def test_window_and_state_sizes_host_logic(lib):
    """Sizes of a window allocation with the state region of the device-side phase order behind its rows."""
    assert binding.moe_state_bytes(1) == 256 and binding.moe_state_bytes(16) == 256      # 4 slots x R epochs, 256-byte units
    assert binding.moe_state_bytes(64) == 1024 and binding.moe_state_bytes(256) == 4096
    assert binding.moe_state_bytes(0) == 0 and binding.moe_state_bytes(257) == 0
    shape = binding.MoeShape(2048, 7168, 256, 16, 8)
    rows = 1300 * 7168 * 2
    up = lambda n: (n + 255) // 256 * 256
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, 0) == rows
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_STATE) == up(rows) + 256
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_QUANT) == \
        up(rows) + up(1300 * 7168) + up(1300 * 4)
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_QUANT) == \
        up(rows) + 256 + up(1300 * 7168) + up(1300 * 4)
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_QUANT_GROUP) == \
        up(rows) + 256 + up(1300 * 7168) + up(1300 * 56 * 4)                           # one scale per 128 elements
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_QUANT | binding.MOE_WINDOW_QUANT_GROUP) == 0
    odd = binding.MoeShape(2048, 7168 + 64, 256, 16, 8)                                # H % 128 != 0: no group-wise parts
    assert lib.moe_window_bytes(ctypes.byref(odd), 1300, binding.MOE_WINDOW_QUANT_GROUP) == 0
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_COUNTS) == 0   # only behind the state region
    box = 2 * (16 * 256 + 16) * 4                                                      # two buffers of [R][E] counts + [R] epochs
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_COUNTS) == \
        up(rows) + 256 + up(box)
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, binding.MOE_WINDOW_STATE | binding.MOE_WINDOW_COUNTS |
                                binding.MOE_WINDOW_QUANT) == up(rows) + 256 + up(box) + up(1300 * 7168) + up(1300 * 4)
    assert lib.moe_window_bytes(ctypes.byref(shape), 1300, 16) == 0                      # unknown flag
    assert lib.moe_window_bytes(ctypes.byref(shape), -1, 1) == 0 and lib.moe_window_bytes(None, 8, 1) == 0
    assert ctypes.sizeof(binding.MoeWindowHandle) == 96
    # calls that need a context reject a missing one before touching anything
    assert lib.moe_peers_check(None, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_signal_peers(None, 0, 1, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_wait_peers(None, 0, 1, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_push_counts(None, 1, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_notify_peers(None, 1, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_layout_push(None, 0, None, 0, 0, 1, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_dispatch_cached(None, None, None, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_window_export(None, 16, 1, 0, None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_dispatch_quant_cached(None, None, None, None) == binding.MOE_ERR_INVALID_ARG
    assert binding.status_string(binding.MOE_ERR_STALE_PEERS) != binding.status_string(binding.MOE_ERR_CUDA)
