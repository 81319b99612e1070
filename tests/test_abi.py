"""The C-ABI library builds, loads without a GPU, and exports every function include/jot.h declares."""
import ctypes
import os
import re

from paper_2602_11133_b200 import build as jot_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "jot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(jot_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = jot_build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert {"jot_init_model", "jot_denoise_step", "jot_accept_freeze", "jot_generate"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2602_11133_b200 import jot
    assert sorted(jot.EXPORTS) == names


def test_host_side_calls_without_device_work():
    lib = ctypes.CDLL(jot_build.build())
    lib.jot_status_string.restype = ctypes.c_char_p
    assert lib.jot_status_string(0) == b"ok"
    assert b"wait" in lib.jot_status_string(-5)
    assert lib.jot_workspace_bytes(None, 1, 1) == 0
    from paper_2602_11133_b200 import jot
    cfg = jot.ModelConfig(2, 256, 4, 4, 64, 704, 4096, 4095, 10000.0, 1e-5)
    lib.jot_workspace_bytes.restype = ctypes.c_size_t
    lib.jot_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
    n1 = lib.jot_workspace_bytes(ctypes.byref(cfg), 1, 96)
    n2 = lib.jot_workspace_bytes(ctypes.byref(cfg), 2, 96)
    assert 0 < n1 < n2 and n1 % 1024 == 0
    bad = jot.ModelConfig(2, 250, 4, 4, 64, 704, 4096, 4095, 10000.0, 1e-5)
    assert lib.jot_workspace_bytes(ctypes.byref(bad), 1, 96) == 0
    # argument errors are reported before anything touches a device
    assert lib.jot_generate(None, None, 0, None, None, 1, 1, None, None, None, None, None, None) == -1
    assert lib.jot_accept_freeze(None, 0, 0, None, 1, 1, 0, 1, 1, None, None, None, None, None, None, None, 0, None) == -1
