"""The C-ABI library loads and exports every entry point include/topk.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2209_15203_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "topk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tk_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree():
    assert declared_symbols() == sorted(binding.EXPORTS)


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    assert os.path.exists(binding.library_path())
    for name in declared_symbols():
        assert getattr(lib, name) is not None


def test_host_side_argument_checks_need_no_gpu():
    lib = binding.load()
    assert lib.tk_workspace_bytes(0, 1, 1, 1) == 0
    assert lib.tk_workspace_bytes(100, 1, 101, 1) == 0
    assert lib.tk_workspace_bytes(100, 0, 1, 1) == 0
    assert lib.tk_workspace_bytes(2 ** 31, 1, 1, 1) == 0
    assert lib.tk_workspace_bytes(124_000_000, 8, 12_400, 12_400) > 124_000_000 * 4
    assert lib.tk_init(None, 10, 1, 1, 1, None, None, 0, None) == -1
    h = ctypes.c_void_p()
    assert lib.tk_init(ctypes.byref(h), 10, 1, 1, 1, None, None, 0, None) == -1
    assert lib.tk_step(None, None, None, 0.1, 1) == -1
    assert lib.tk_topk(None, None, 1, 10, 1, None, None) == -1
    assert binding.strerror(0) == "ok" and "invalid" in binding.strerror(-1)
    assert lib.tk_launch_count(None) == 0
