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


def test_tail_choice_of_the_gradient_gemms():
    """Host logic of the K-split tail: which remainder tiles are split, into how many parts."""
    import pytest
    assert vp.vp_ce_set_tail_parts(-1) == -1
    # config 3, weight gradient: 32 x 12 tiles (last column tile 128 wide in the MMA), 2 raster groups, K = 16384 tokens:
    # 384 % 74 = 14 remainder tiles, split (the launch measured 6 % shorter that way)
    n, parts, stagger = vp.vp_ce_tail_choice(32, 12, 6, 128, 256, 74)
    assert n == 14 and parts in (2, 3) and stagger == 15
    # config 4: 32 x 28 whole tiles, K = 8192: 896 % 74 = 8 remainder tiles
    n, parts, stagger = vp.vp_ce_tail_choice(32, 28, 7, 256, 128, 74)
    assert n == 8 and parts in (2, 3)
    # a whole number of rounds: nothing to split
    assert vp.vp_ce_tail_choice(37, 10, 10, 256, 256, 74) == (0, 1, 0)
    # almost a full last round (70 of 74 pairs busy): a split cannot pay
    assert vp.vp_ce_tail_choice(36, 4, 4, 256, 256, 74)[0] == 0
    # a contraction too short for two parts of 8 k-blocks plus the stagger: no split
    assert vp.vp_ce_tail_choice(8, 10, 10, 256, 24, 74) == (0, 1, 0)
    # the knob: 0 forbids, k forces (equal parts when K is too short for staggered ones)
    vp.vp_ce_set_tail_parts(0)
    try:
        assert vp.vp_ce_tail_choice(32, 12, 6, 128, 256, 74) == (0, 1, 0)
        vp.vp_ce_set_tail_parts(4)
        assert vp.vp_ce_tail_choice(32, 12, 6, 128, 256, 74) == (14, 4, 15)
        assert vp.vp_ce_tail_choice(4, 2, 2, 128, 16, 74) == (8, 4, 0)
        assert vp.vp_ce_tail_choice(4, 2, 2, 128, 3, 74) == (0, 1, 0)       # fewer k-blocks than parts
    finally:
        vp.vp_ce_set_tail_parts(-1)
    # never more split tiles than flags in the workspace allow, never more parts than three by the library's own choice
    for rows, cols, kb in [(64, 12, 128), (98, 28, 256), (16, 8, 32), (5, 3, 512), (1, 1, 64), (64, 28, 392)]:
        n, parts, stagger = vp.vp_ce_tail_choice(rows, cols, min(cols, 7), 256, kb, 74)
        assert 0 <= n <= 64 and 1 <= parts <= 3 and (n == 0) == (parts == 1)
        if n:
            assert (kb - stagger * parts * (parts - 1) // 2) // parts >= 8
    with pytest.raises(vp.VpceError):
        vp.vp_ce_tail_choice(0, 1, 1, 256, 64, 74)
