"""The C-ABI shared library loads and exports every entry point include/ue5m3.h declares
(no compute calls: runs without a GPU)."""
import ctypes
import os
import re

import paper_2609_02846_b200.binding as binding
from paper_2609_02846_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ue5m3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ue5m3_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build_library())
    names = _declared()
    assert set(binding.SYMBOLS) <= set(names) and len(names) >= 7
    for n in names:
        assert hasattr(lib, n), n


def test_host_only_entry_points():
    assert binding.status_string(0) == "UE5M3_OK"
    assert "SHAPE" in binding.status_string(2)
    assert binding.scales_bytes(256, 4096, binding.LAYOUT_1D_ROW) == 256 * 256
    assert binding.scales_bytes(256, 4096, binding.LAYOUT_1D_COL) == 4096 * 16
    assert binding.scales_bytes(256, 4096, binding.LAYOUT_2D) == 16 * 256
    assert binding.scales_bytes(200 * 16, 4096, binding.LAYOUT_1D_ROW, binding.SCALES_TILED) == 25 * 16 * 2048
    assert binding.scales_bytes(250, 4096, binding.LAYOUT_1D_ROW) == 0


def test_hold_policy_refreshes_every_interval():
    c = binding.AmaxCache(50)
    hits = []
    for t in range(200):
        if c.refreshes_at(t):
            hits.append(t)
            c.last_refresh = t
    import oracle
    assert hits == [0, 50, 100, 150] == oracle.hold_schedule(200, 50)
