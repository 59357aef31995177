"""The C-ABI library builds, loads without a GPU, and exports every declared symbol."""
import ctypes
import os
import re

from paper_2412_00061_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ctcsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ctcsd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_host_only_entry_points_work_without_a_device():
    lib = binding.load_library()
    assert lib.ctcsd_strerror(0) == b"ok"
    assert lib.ctcsd_strerror(-5) == b"device-side wait timed out"
    cfg = binding.CConfig(1, 4096, 32000, 5, 4, 0, 16, 64, 32, 32, 128, 1, 0, 0)
    n = ctypes.c_size_t(0)
    assert lib.ctcsd_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0
    assert 0 < n.value < (1 << 30)
    assert lib.ctcsd_workspace_bytes(None, ctypes.byref(n)) == -1
    bad = binding.CConfig(1, 4096, 32000, 5, 4, 0, 16, 300, 32, 32, 128, 1, 0, 0)   # too many nodes
    assert lib.ctcsd_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == -1
