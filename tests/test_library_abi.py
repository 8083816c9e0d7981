"""CPU-side checks of the boundary: the library builds, loads, exports every symbol the header
declares, and its pure-host entry points behave (no kernel is launched here)."""
import ctypes
import os
import re

import paper_2609_14306_b200 as vp
from paper_2609_14306_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, fn)).read(), flags=re.S)
            names += re.findall(r"\b((?:vp_ce|osadamw)_\w+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    build_library()
    lib = vp.load_library()
    names = declared_functions()
    assert {"vp_ce_forward", "vp_ce_backward", "vp_ce_workspace_bytes", "vp_ce_mean_loss",
            "vp_ce_device_status", "vp_ce_status_string", "vp_ce_meeting_forward", "vp_ce_meeting_backward",
            "osadamw_create", "osadamw_step", "osadamw_wait", "osadamw_update_device"} <= set(names)
    raw = ctypes.CDLL(vp.library_path())
    for n in names:
        assert hasattr(raw, n), n
        assert hasattr(vp, n), f"python binding lacks {n}"


def test_workspace_size_depends_on_neither_V_nor_T():
    # cfg 3 and cfg 5 share (T_chunk, d, block_v), hence the workspace
    a = vp.vp_ce_workspace_bytes(4096, 2880, 8192)
    assert a > 0 and a == vp.vp_ce_workspace_bytes(4096, 2880, 8192)
    g = 4096 * 8192 * 2 + 4096 * 2880 * 4
    assert g <= a <= g + (4 << 20)          # G strip + fp32 dH accumulator + O(T_chunk) state
    assert vp.vp_ce_workspace_bytes(8192, 7168, 8192) > a
    # rejected shapes
    assert vp.vp_ce_workspace_bytes(100, 2880, 8192) == 0      # T_chunk % 128
    assert vp.vp_ce_workspace_bytes(4096, 2881, 8192) == 0     # d % 8
    assert vp.vp_ce_workspace_bytes(4096, 2880, 8000) == 0     # block_v % 256
    assert vp.vp_ce_workspace_bytes(0, 2880, 8192) == 0


def test_status_strings():
    assert vp.vp_ce_status_string(0) == "ok"
    for c in (1, 2, 3, 4):
        assert vp.vp_ce_status_string(c) not in ("ok", "unknown status")
    assert vp.vp_ce_status_string(99) == "unknown status"
    assert vp.vp_ce_launch_count() >= 0


def test_wait_limit_and_test_hook_arguments():
    # pure host state: no kernel is launched
    prev = vp.vp_ce_set_wait_limit_ns(0)                      # query only
    assert prev == 2_000_000_000
    assert vp.vp_ce_set_wait_limit_ns(5) == prev              # clamped up to 1 ms ...
    assert vp.vp_ce_set_wait_limit_ns(10**12) == 1_000_000    # ... and down to 60 s
    assert vp.vp_ce_set_wait_limit_ns(prev) == 60_000_000_000
    assert vp.vp_ce_set_wait_limit_ns(-1) == prev
    import pytest
    for bad in [(4, 0, 1), (0, -1, 1), (0, 0, 0), (0, 0, 4), (0, 70000, 1)]:
        with pytest.raises(vp.VpceError):
            vp.vp_ce_debug_drop_copy(*bad)
    vp.vp_ce_debug_drop_copy(2, 3, 3)
    vp.vp_ce_debug_drop_copy(-1)                              # disarm
    # the tail-split knob: -1 (library's choice) by default; 1, 9 and -2 are ignored
    assert vp.vp_ce_set_tail_parts(3) == -1
    assert vp.vp_ce_set_tail_parts(1) == 3 and vp.vp_ce_set_tail_parts(9) == 3 and vp.vp_ce_set_tail_parts(-2) == 3
    assert vp.vp_ce_set_tail_parts(0) == 3
    assert vp.vp_ce_set_tail_parts(-1) == 0


def test_streamed_adamw_staging_size():
    # pure host arithmetic: 16 bytes per parameter and slot (p, m, v, g in fp32), arrays padded to 256 bytes
    assert vp.osadamw_staging_bytes(1 << 20, 2) == 2 * 4 * (1 << 20) * 4
    assert vp.osadamw_staging_bytes(100, 3) == 3 * 4 * 128 * 4
    assert vp.osadamw_staging_bytes(0, 2) == 0 and vp.osadamw_staging_bytes(100, 0) == 0
