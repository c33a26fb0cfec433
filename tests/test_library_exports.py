"""The C-ABI library loads without a GPU and exports every entry point the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "spatvit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:int32_t|int64_t|uint32_t|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_are_exported():
    import paper_2601_12150_b200 as spv
    from paper_2601_12150_b200 import build
    build.build()
    lib = ctypes.CDLL(spv.LIB_PATH)
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/spatvit.h but not exported"
    assert sorted(spv.EXPORTS) == names


def test_host_only_entry_points():
    import paper_2601_12150_b200 as spv
    assert spv.filter_keep_count(4096, 0.5) == 2048
    assert spv.filter_keep_count(4096, 0.6) == 2458
    assert spv.filter_keep_count(21316, 0.5) == 10658
    for bad in (0.0, 1.01, -1.0):
        with pytest.raises(spv.SpvError):
            spv.filter_keep_count(100, bad)
    assert spv.status_string(0) == "ok"
    assert "wait" in spv.status_string(spv.ERR_TIMEOUT)
    d = spv.FilterDesc(2, 16, 4096, 1, 1024, 0.5, 0, 0)
    need = ctypes.c_size_t(0)
    assert spv.lib().spv_filter_workspace_size(ctypes.byref(d), ctypes.byref(need)) == 0
    assert need.value >= 2 * 2 * 4096 * 4
    d.dim = 1001
    assert spv.lib().spv_filter_workspace_size(ctypes.byref(d), ctypes.byref(need)) == spv.ERR_ALIGNMENT


def test_no_per_process_launch_state_in_the_kernels_sources():
    """Launch configuration (function attributes, resident-CTA counts) is per device and lives in the context:
    no function-level `static` variable may hold it in the CUDA sources (two contexts on two devices of one
    process would share it)."""
    import re
    csrc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2601_12150_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if not name.endswith(".cu"):
            continue
        text = open(os.path.join(csrc, name)).read()
        for m in re.finditer(r"^\s+static\s+(bool|int|int32_t|unsigned)\s+\w+\s*(=|;)", text, re.M):
            raise AssertionError(f"{name}: function-level static `{m.group(0).strip()}`")
