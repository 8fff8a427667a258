"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2408_15562_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "fspad.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(fspad_[a-z_]+)\s*\(", src)))


def test_library_builds_and_exports_every_declared_symbol():
    build.build()
    lib = binding.load()
    names = _declared()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_covers_all_codes():
    for code in range(0, -10, -1):
        assert binding.strerror(code) != "unknown error"
    assert binding.strerror(-99) == "unknown error"


def test_host_side_validation_needs_no_device():
    import ctypes
    lib = binding.load()
    h = ctypes.c_void_p()
    bad = binding.FspadConfig(32, 8, 64, 60, 1000, 1, 128, 1, 0.0)      # head_dim 64 is not supported
    assert lib.fspad_create(ctypes.byref(bad), ctypes.byref(h)) == -3 and not h.value
    bad = binding.FspadConfig(32, 8, 128, 257, 1000, 1, 512, 1, 0.0)    # more than 256 nodes
    assert lib.fspad_create(ctypes.byref(bad), ctypes.byref(h)) == -4 and not h.value
    bad = binding.FspadConfig(32, 5, 128, 60, 1000, 1, 128, 1, 0.0)     # Hkv does not divide Hq
    assert lib.fspad_create(ctypes.byref(bad), ctypes.byref(h)) == -3
    assert lib.fspad_create(None, ctypes.byref(h)) == -1
    assert lib.fspad_tree_attn(None, None, None, None, None, None, None, None, 1, 1, None, None) == -1
    assert lib.fspad_kv_compact(None, None, None, None, None, 1, None, None) == -1
